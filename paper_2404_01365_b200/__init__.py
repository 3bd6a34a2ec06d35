"""B200-native GRIFFIN feed-forward path (arXiv 2404.01365).

`binding` wraps the C-ABI library (libgriffin_ff.so, hand-written sm_100a
kernels); `synth` draws the seeded synthetic workloads.  Importing the
package loads nothing native; `binding.load()` does, and fails loudly when
the library has not been built.
"""
