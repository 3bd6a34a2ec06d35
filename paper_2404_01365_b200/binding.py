"""ctypes binding of libgriffin_ff.so: argument marshalling only.

Every function here has the name of the C entry point it calls (include/griffin_ff.h) and
takes torch tensors for device buffers; each step of the path runs in the library's CUDA
kernels.  There is no fallback: if the library is missing or a call fails, an exception is
raised.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import build as _build

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(7)
ACT_SWIGLU, ACT_GEGLU_TANH, ACT_REGLU, ACT_GEGLU_ERF = 0, 1, 2, 3
ACT_RELU, ACT_GELU_TANH, ACT_GELU_ERF, ACT_SILU = 4, 5, 6, 7   # blocks without a gate (Eq. 2): w_gate is None
DT_F32, DT_BF16 = 0, 1
DECODE_DEFAULT, DECODE_OVERLAP_WEIGHT_PREFETCH, DECODE_TCGEN05, DECODE_RING, DECODE_STREAM = 0, 1, 2, 4, 8
MAX_BATCH = 32

ACT_BY_NAME = {"swiglu": ACT_SWIGLU, "geglu_tanh": ACT_GEGLU_TANH, "reglu": ACT_REGLU, "geglu_erf": ACT_GEGLU_ERF,
               "relu": ACT_RELU, "gelu_tanh": ACT_GELU_TANH, "gelu_erf": ACT_GELU_ERF, "silu": ACT_SILU}


def act_is_gated(act):
    act = ACT_BY_NAME[act] if isinstance(act, str) else int(act)
    return ACT_SWIGLU <= act <= ACT_GEGLU_ERF
DTYPE_BY_NAME = {"f32": DT_F32, "bf16": DT_BF16}

EXPORTS = (
    "griffin_status_string", "griffin_version", "griffin_k_from_keep_ratio", "griffin_compact_ldk",
    "griffin_workspace_bytes", "griffin_workspace_init", "griffin_ff_prefill_score", "griffin_select_topk",
    "griffin_combine_scores", "griffin_compact_experts", "griffin_ff_decode", "griffin_check_device_status",
    "griffin_ff_decode_static", "griffin_ff_decode_indexed", "griffin_ff_prefill_score_chunk",
    "griffin_kernel_launches", "griffin_ff_decode_static_status", "griffin_compact_experts_nm",
)


class GriffinError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        super().__init__(f"{what}: status {status} ({status_string(status)})")


class FFDesc(C.Structure):
    _fields_ = [("d", C.c_int32), ("d_ff", C.c_int32), ("act", C.c_int32), ("dtype", C.c_int32)]


class FFWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("w_gate", "w_up", "w_down", "b_gate", "b_up", "b_down")]


class FFWeightsNM(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("w_gate", "w_up", "w_down_t", "b_gate", "b_up", "b_down")]


class FFCompact(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("w_gate_c", "w_up_c", "w_down_c", "b_gate_c", "b_up_c")] + \
               [("k", C.c_int32), ("ldk", C.c_int32)]


_lib = None


def load(path=None):
    """Loads the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    path = path or os.environ.get("GRIFFIN_FF_LIB") or _build.LIB_PATH
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_2404_01365_b200.build` "
                           "(there is no fallback path)")
    lib = C.CDLL(path)
    vp, i32, u32, sz = C.c_void_p, C.c_int32, C.c_uint32, C.c_size_t
    lib.griffin_status_string.restype = C.c_char_p
    lib.griffin_status_string.argtypes = [C.c_int]
    lib.griffin_version.restype = i32
    lib.griffin_version.argtypes = []
    lib.griffin_kernel_launches.restype = C.c_uint64
    lib.griffin_kernel_launches.argtypes = []
    lib.griffin_k_from_keep_ratio.restype = i32
    lib.griffin_k_from_keep_ratio.argtypes = [i32, C.c_double]
    lib.griffin_compact_ldk.restype = i32
    lib.griffin_compact_ldk.argtypes = [i32]
    lib.griffin_workspace_bytes.restype = sz
    lib.griffin_workspace_bytes.argtypes = [C.POINTER(FFDesc), i32, i32]
    lib.griffin_workspace_init.restype = C.c_int
    lib.griffin_workspace_init.argtypes = [vp, sz, vp]
    lib.griffin_ff_prefill_score.restype = C.c_int
    lib.griffin_ff_prefill_score.argtypes = [C.POINTER(FFDesc), C.POINTER(FFWeights), vp, i32, vp, vp, vp, sz, vp]
    lib.griffin_ff_prefill_score_chunk.restype = C.c_int
    lib.griffin_ff_prefill_score_chunk.argtypes = [C.POINTER(FFDesc), C.POINTER(FFWeights), vp, i32, vp, vp, vp, i32, vp,
                                                   sz, vp]
    lib.griffin_select_topk.restype = C.c_int
    lib.griffin_select_topk.argtypes = [vp, i32, i32, i32, vp, vp]
    lib.griffin_combine_scores.restype = C.c_int
    lib.griffin_combine_scores.argtypes = [vp, C.POINTER(i32), i32, i32, vp, vp]
    lib.griffin_compact_experts.restype = C.c_int
    lib.griffin_compact_experts.argtypes = [C.POINTER(FFDesc), C.POINTER(FFWeights), vp, C.POINTER(FFCompact), vp, vp]
    lib.griffin_compact_experts_nm.restype = C.c_int
    lib.griffin_compact_experts_nm.argtypes = [C.POINTER(FFDesc), C.POINTER(FFWeightsNM), vp, C.POINTER(FFCompact), vp, vp]
    lib.griffin_ff_decode.restype = C.c_int
    lib.griffin_ff_decode.argtypes = [C.POINTER(FFDesc), i32, C.POINTER(FFCompact), vp, vp, vp, vp, sz, u32, vp]
    lib.griffin_ff_decode_indexed.restype = C.c_int
    lib.griffin_ff_decode_indexed.argtypes = [C.POINTER(FFDesc), i32, C.POINTER(FFWeightsNM), vp, i32, vp, vp, vp, sz, u32, vp]
    lib.griffin_ff_decode_static.restype = C.c_int
    lib.griffin_ff_decode_static.argtypes = [C.POINTER(FFDesc), i32, C.POINTER(FFCompact), vp, vp, vp, u32, vp]
    lib.griffin_ff_decode_static_status.restype = C.c_int
    lib.griffin_ff_decode_static_status.argtypes = [vp]
    lib.griffin_check_device_status.restype = C.c_int
    lib.griffin_check_device_status.argtypes = [vp, vp]
    _lib = lib
    return lib


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _check(st, what):
    if st != OK:
        raise GriffinError(st, what)


def status_string(st):
    return load().griffin_status_string(int(st)).decode()


def griffin_version():
    return load().griffin_version()


def griffin_kernel_launches():
    """Kernels launched by the library in this process so far."""
    return int(load().griffin_kernel_launches())


def griffin_k_from_keep_ratio(d_ff, keep):
    return load().griffin_k_from_keep_ratio(int(d_ff), float(keep))


def griffin_compact_ldk(k):
    return load().griffin_compact_ldk(int(k))


def make_desc(d, d_ff, act, dtype):
    act = ACT_BY_NAME[act] if isinstance(act, str) else int(act)
    dtype = DTYPE_BY_NAME[dtype] if isinstance(dtype, str) else int(dtype)
    return FFDesc(int(d), int(d_ff), act, dtype)


def make_weights(w_gate, w_up, w_down, b_gate=None, b_up=None, b_down=None):
    w = FFWeights(_ptr(w_gate), _ptr(w_up), _ptr(w_down), _ptr(b_gate), _ptr(b_up), _ptr(b_down))
    w._keep = (w_gate, w_up, w_down, b_gate, b_up, b_down)  # keep the tensors alive
    return w


def make_weights_nm(w_gate, w_up, w_down_t, b_gate=None, b_up=None, b_down=None):
    """Neuron-major full weights for griffin_ff_decode_indexed: w_down_t is W_2 transposed, [d_ff, d]."""
    w = FFWeightsNM(_ptr(w_gate), _ptr(w_up), _ptr(w_down_t), _ptr(b_gate), _ptr(b_up), _ptr(b_down))
    w._keep = (w_gate, w_up, w_down_t, b_gate, b_up, b_down)
    return w


def make_compact(w_gate_c, w_up_c, w_down_c, k, ldk, b_gate_c=None, b_up_c=None):
    c = FFCompact(_ptr(w_gate_c), _ptr(w_up_c), _ptr(w_down_c), _ptr(b_gate_c), _ptr(b_up_c), int(k), int(ldk))
    c._keep = (w_gate_c, w_up_c, w_down_c, b_gate_c, b_up_c)
    return c


def alloc_compact(desc, k, device, torch_dtype, with_bias=False):
    """Allocates the buffers of one compact expert set (torch owns the memory)."""
    ldk = griffin_compact_ldk(k)
    gated = act_is_gated(desc.act)   # a block without a gate has no W_g_hat
    g = torch.empty((k, desc.d), device=device, dtype=torch_dtype) if gated else None
    u = torch.empty((k, desc.d), device=device, dtype=torch_dtype)
    dn = torch.empty((desc.d, ldk), device=device, dtype=torch_dtype)
    bg = torch.empty((k,), device=device, dtype=torch_dtype) if with_bias and gated else None
    bu = torch.empty((k,), device=device, dtype=torch_dtype) if with_bias else None
    return make_compact(g, u, dn, k, ldk, bg, bu)


def griffin_workspace_bytes(desc, S_max, n_seq_max):
    return load().griffin_workspace_bytes(C.byref(desc), int(S_max), int(n_seq_max))


def alloc_workspace(desc, S_max, n_seq_max, device, stream=None):
    """Allocates and initialises a workspace tensor (uint8) large enough for any call."""
    n = griffin_workspace_bytes(desc, S_max, n_seq_max)
    if n == 0:
        raise GriffinError(ERR_INVALID_ARG, "griffin_workspace_bytes")
    ws = torch.empty((n,), device=device, dtype=torch.uint8)
    griffin_workspace_init(ws, stream)
    return ws


def griffin_workspace_init(ws, stream=None):
    _check(load().griffin_workspace_init(_ptr(ws), ws.numel(), _stream(stream)), "griffin_workspace_init")


def griffin_ff_prefill_score(desc, weights, x, y, score, ws, stream=None):
    S = x.shape[0]
    _check(load().griffin_ff_prefill_score(C.byref(desc), C.byref(weights), _ptr(x), S, _ptr(y), _ptr(score),
                                           _ptr(ws), ws.numel(), _stream(stream)), "griffin_ff_prefill_score")


def griffin_ff_prefill_score_chunk(desc, weights, x, y, sumsq, score, first, ws, stream=None):
    """One piece of a prompt that is fed piece by piece: sumsq carries the statistic's squares."""
    S = x.shape[0]
    _check(load().griffin_ff_prefill_score_chunk(C.byref(desc), C.byref(weights), _ptr(x), S, _ptr(y), _ptr(sumsq),
                                                 _ptr(score), 1 if first else 0, _ptr(ws), ws.numel(), _stream(stream)),
           "griffin_ff_prefill_score_chunk")


def griffin_select_topk(score, k, idx, stream=None):
    n_seq, d_ff = (1, score.shape[0]) if score.dim() == 1 else score.shape
    _check(load().griffin_select_topk(_ptr(score), int(n_seq), int(d_ff), int(k), _ptr(idx), _stream(stream)),
           "griffin_select_topk")


def griffin_combine_scores(score, prompt_len, out, stream=None):
    n_seq, d_ff = score.shape
    arr = (C.c_int32 * n_seq)(*[int(v) for v in prompt_len])
    _check(load().griffin_combine_scores(_ptr(score), arr, int(n_seq), int(d_ff), _ptr(out), _stream(stream)),
           "griffin_combine_scores")


def griffin_compact_experts(desc, weights, idx, out, ws=None, stream=None):
    _check(load().griffin_compact_experts(C.byref(desc), C.byref(weights), _ptr(idx), C.byref(out), _ptr(ws),
                                          _stream(stream)), "griffin_compact_experts")


def griffin_compact_experts_nm(desc, weights_nm, idx, out, ws=None, stream=None):
    """The same compact set from neuron-major full weights (w_down_t = W_2 transposed)."""
    _check(load().griffin_compact_experts_nm(C.byref(desc), C.byref(weights_nm), _ptr(idx), C.byref(out), _ptr(ws),
                                             _stream(stream)), "griffin_compact_experts_nm")


def compact_array(sets):
    """A C array of compact-set structs for griffin_ff_decode (build once, reuse per step)."""
    arr = (FFCompact * len(sets))()
    for i, s in enumerate(sets):
        C.memmove(C.byref(arr[i]), C.byref(s), C.sizeof(FFCompact))
    arr._keep = list(sets)
    return arr


def griffin_ff_decode(desc, sets, b_down, x, y, ws, flags=DECODE_DEFAULT, stream=None):
    arr = sets if isinstance(sets, C.Array) else compact_array(sets)
    _check(load().griffin_ff_decode(C.byref(desc), len(arr), arr, _ptr(b_down), _ptr(x), _ptr(y), _ptr(ws),
                                    ws.numel(), int(flags), _stream(stream)), "griffin_ff_decode")


def griffin_ff_decode_indexed(desc, weights_nm, idx, x, y, ws, flags=DECODE_DEFAULT, stream=None):
    """Pruned FF straight from the full neuron-major weights; idx [B, k] int32 on the device."""
    B, k = (1, idx.shape[0]) if idx.dim() == 1 else idx.shape
    _check(load().griffin_ff_decode_indexed(C.byref(desc), int(B), C.byref(weights_nm), _ptr(idx), int(k), _ptr(x),
                                            _ptr(y), _ptr(ws), ws.numel(), int(flags), _stream(stream)),
           "griffin_ff_decode_indexed")


STATIC_SCRATCH_BYTES = 1 << 20


def griffin_ff_decode_static(desc, sets, b_down, x, y, flags=DECODE_DEFAULT, stream=None):
    """griffin_ff_decode for callers that cannot allocate a workspace: the scratch is a fixed
    array inside the library (see include/griffin_ff.h for its limit and sharing rules)."""
    arr = sets if isinstance(sets, C.Array) else compact_array(sets)
    _check(load().griffin_ff_decode_static(C.byref(desc), len(arr), arr, _ptr(b_down), _ptr(x), _ptr(y), int(flags),
                                           _stream(stream)), "griffin_ff_decode_static")


def griffin_ff_decode_static_status(stream=None):
    """Status of the static-scratch decode calls on the current device (synchronises the stream)."""
    return load().griffin_ff_decode_static_status(_stream(stream))


def griffin_check_device_status(ws, stream=None):
    return load().griffin_check_device_status(_ptr(ws), _stream(stream))
