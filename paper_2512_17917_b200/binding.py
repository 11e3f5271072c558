"""Thin ctypes binding of libkvr.so: same names as the C ABI in include/kvr.h, argument
marshalling only.  torch provides device memory and the current stream; every step of the path
runs in the library's CUDA kernels.  There is no fallback: if libkvr.so is missing or does not
load, every call raises.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libkvr.so")

KVR_OK = 0
KVR_ERR_SHAPE = 3
KVR_F16, KVR_BF16 = 0, 1
KVR_ALL_LAYERS = -1
KVR_MAX_B = 8192
KVR_DECODE_AUTO, KVR_DECODE_SPLIT, KVR_DECODE_STAGED = 0, 1, 2
KVR_SCORE_AUTO, KVR_SCORE_MMA_SYNC, KVR_SCORE_TCGEN05 = 0, 1, 2
KVR_COMBINE_MEDIAN, KVR_COMBINE_MEAN = 0, 1

# every symbol include/kvr.h declares
EXPORTS = (
    "kvr_sketch_create", "kvr_sketch_reset", "kvr_sketch_destroy", "kvr_sketch_device_bytes",
    "kvr_compress", "kvr_decode_attention", "kvr_compress_host", "kvr_decode_attention_host",
    "kvr_get_scores", "kvr_get_assignment", "kvr_get_cells", "kvr_reconstruct", "kvr_layer_shape",
    "kvr_launch_count", "kvr_status_string", "kvr_decode_attention_static",
    "kvr_sketch_set_decode_kernel", "kvr_last_decode_kernel", "kvr_sketch_device_status",
    "kvr_accumulate_scores", "kvr_demote", "kvr_sketch_set_score_kernel", "kvr_last_score_kernel",
    "kvr_accumulate_vague_scores", "kvr_swap", "kvr_sketch_set_obs_window_causal", "kvr_paper_storage_split", "kvr_layer_budgets", "kvr_sketch_set_combine",
    "kvr_measure_pipe_peaks", "kvr_append", "kvr_append_sizes", "kvr_decode_attention_mq", "kvr_sketch_set_wait_test", "kvr_decode_attention_scored",
)


i32_t = ctypes.c_int32


class KvrError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (kvr_status_t {status})")


class SketchDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "r", "b", "head_dim", "n_kv_heads", "n_q_heads", "batch", "n_layers", "max_context",
        "kv_dtype", "index_mix", "seeds_per_head")]


_lib = None


def lib() -> ctypes.CDLL:
    """Load libkvr.so (built by `python -m paper_2512_17917_b200.build`); raise if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2512_17917_b200.build` "
                               "(there is no CPU or PyTorch fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_float
        L.kvr_sketch_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(SketchDesc), vp, vp]
        L.kvr_sketch_reset.argtypes = [vp, i32, vp]
        L.kvr_sketch_destroy.argtypes = [vp]
        L.kvr_sketch_device_bytes.argtypes = [vp]
        L.kvr_sketch_device_bytes.restype = ctypes.c_size_t
        L.kvr_compress.argtypes = [vp, i32, vp, vp, vp, i32, i32, i32, i32, vp, vp, vp, vp]
        L.kvr_decode_attention.argtypes = [vp, i32, vp, vp, vp, vp, i32, f32, vp, vp]
        L.kvr_decode_attention_static.argtypes = [vp, i32, vp, vp, vp, vp, i32, f32, vp, vp]
        L.kvr_decode_attention_scored.argtypes = [vp, i32, vp, vp, vp, vp, i32, f32, vp, vp, vp]
        L.kvr_compress_host.argtypes = [vp, i32, vp, vp, vp, i32, i32, i32, i32, vp]
        L.kvr_decode_attention_host.argtypes = [vp, i32, vp, f32, vp, vp]
        L.kvr_get_scores.argtypes = [vp, i32, vp, vp]
        L.kvr_get_assignment.argtypes = [vp, i32, vp, vp, vp, vp]
        L.kvr_get_cells.argtypes = [vp, i32, vp, vp]
        L.kvr_reconstruct.argtypes = [vp, i32, vp, vp, vp]
        L.kvr_layer_shape.argtypes = [vp, i32, ctypes.POINTER(i32), ctypes.POINTER(i32)]
        L.kvr_launch_count.argtypes = [vp]
        L.kvr_launch_count.restype = ctypes.c_int64
        L.kvr_sketch_set_decode_kernel.argtypes = [vp, i32]
        L.kvr_sketch_device_status.argtypes = [vp, ctypes.POINTER(i32), vp]
        L.kvr_accumulate_scores.argtypes = [vp, i32, vp, vp, i32, f32, vp, vp]
        L.kvr_demote.argtypes = [vp, i32, vp, vp, vp, vp, i32, i32, i32, i32, vp, vp, vp, vp, vp]
        L.kvr_sketch_set_score_kernel.argtypes = [vp, i32]
        L.kvr_sketch_set_obs_window_causal.argtypes = [vp, i32]
        L.kvr_sketch_set_combine.argtypes = [vp, i32]
        L.kvr_layer_budgets.argtypes = [ctypes.POINTER(ctypes.c_double), i32, i32, f32, ctypes.POINTER(i32)]
        L.kvr_paper_storage_split.argtypes = [i32, f32, ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(i32)]
        L.kvr_accumulate_vague_scores.argtypes = [vp, i32, vp, f32, vp]
        L.kvr_swap.argtypes = [vp, i32, vp, vp, vp, vp, i32, i32, f32, i32, vp, vp]
        L.kvr_last_score_kernel.argtypes = [vp]
        L.kvr_last_score_kernel.restype = i32
        L.kvr_last_decode_kernel.argtypes = [vp]
        L.kvr_last_decode_kernel.restype = i32
        L.kvr_decode_attention_mq.argtypes = [vp, i32, vp, vp, vp, vp, i32, i32, i32, f32, vp, vp]
        L.kvr_sketch_set_wait_test.argtypes = [vp, ctypes.c_int64, i32]
        L.kvr_append_sizes.argtypes = [i32, i32, i32, i32, i32, i32, ctypes.POINTER(i32)]
        L.kvr_append_sizes.restype = i32
        L.kvr_append.argtypes = [vp, i32, vp, vp, vp, vp, i32, i32, vp, vp, i32, i32, i32, i32, f32, i32, vp, vp, vp, vp, vp, vp]
        L.kvr_measure_pipe_peaks.argtypes = [ctypes.POINTER(ctypes.c_double), vp]
        L.kvr_status_string.argtypes = [i32]
        L.kvr_status_string.restype = ctypes.c_char_p
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().kvr_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != KVR_OK:
        raise KvrError(status, where)


def _stream(stream=None) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _ptr(t) -> ctypes.c_void_p:
    if t is None:
        return ctypes.c_void_p(0)
    assert t.is_contiguous(), "kvr tensors must be contiguous"
    return ctypes.c_void_p(t.data_ptr())


def _dtype_code(dtype: torch.dtype) -> int:
    if dtype == torch.float16:
        return KVR_F16
    if dtype == torch.bfloat16:
        return KVR_BF16
    raise ValueError(f"kv dtype must be float16 or bfloat16, got {dtype}")


class Sketch:
    """Owner of one kvr_sketch_t*; destroyed with the object."""

    def __init__(self, handle: int, desc: SketchDesc, device):
        self.handle = ctypes.c_void_p(handle)
        self.desc = desc
        self.device = device

    @property
    def torch_dtype(self):
        return torch.float16 if self.desc.kv_dtype == KVR_F16 else torch.bfloat16

    def close(self):
        if self.handle:
            lib().kvr_sketch_destroy(self.handle)
            self.handle = ctypes.c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def kvr_sketch_create(*, b: int, batch: int, n_layers: int, n_kv_heads: int, n_q_heads: int,
                      max_context: int, kv_dtype: torch.dtype, hash_seeds, r: int = 3, head_dim: int = 128,
                      index_mix: bool = True, device="cuda", stream=None) -> Sketch:
    """kvr_sketch_create: hash_seeds is an [r, 4] array of uint32 (A, C, A', C' per row), or
    [n_kv_heads, r, 4] for one set of seeds per kv head."""
    seeds = np.ascontiguousarray(hash_seeds, dtype=np.uint32)
    if seeds.shape not in ((r, 4), (n_kv_heads, r, 4)):
        raise ValueError("hash_seeds must have shape [r, 4] or [n_kv_heads, r, 4]")
    desc = SketchDesc(r, b, head_dim, n_kv_heads, n_q_heads, batch, n_layers, max_context,
                      _dtype_code(kv_dtype), int(bool(index_mix)), int(seeds.ndim == 3))
    dev = torch.device(device)
    out = ctypes.c_void_p(0)
    with torch.cuda.device(dev):
        st = lib().kvr_sketch_create(ctypes.byref(out), ctypes.byref(desc),
                                     seeds.ctypes.data_as(ctypes.c_void_p), _stream(stream))
    _check(st, "kvr_sketch_create")
    return Sketch(out.value, desc, dev)


def kvr_sketch_reset(sk: Sketch, layer: int = KVR_ALL_LAYERS, stream=None):
    _check(lib().kvr_sketch_reset(sk.handle, layer, _stream(stream)), "kvr_sketch_reset")


def kvr_sketch_destroy(sk: Sketch):
    sk.close()


def kvr_sketch_device_bytes(sk: Sketch) -> int:
    return int(lib().kvr_sketch_device_bytes(sk.handle))


def kvr_sketch_set_decode_kernel(sk: Sketch, which: int):
    _check(lib().kvr_sketch_set_decode_kernel(sk.handle, int(which)), "kvr_sketch_set_decode_kernel")


def kvr_sketch_device_status(sk: Sketch, stream=None) -> int:
    """Synchronises the stream; 0 = every decode kernel of the handle completed normally."""
    out = ctypes.c_int32(-1)
    with torch.cuda.device(sk.device):
        _check(lib().kvr_sketch_device_status(sk.handle, ctypes.byref(out), _stream(stream)), "kvr_sketch_device_status")
    return out.value


def kvr_last_decode_kernel(sk: Sketch) -> int:
    return int(lib().kvr_last_decode_kernel(sk.handle))


def kvr_sketch_set_score_kernel(sk: Sketch, which: int):
    _check(lib().kvr_sketch_set_score_kernel(sk.handle, int(which)), "kvr_sketch_set_score_kernel")


def kvr_paper_storage_split(context: int, ratio: float):
    """kvr_paper_storage_split: (exact_rows, n_recent, b) of the paper's 0.45 / 0.45 / 0.10 split."""
    e, n, b = ctypes.c_int32(0), ctypes.c_int32(0), ctypes.c_int32(0)
    _check(lib().kvr_paper_storage_split(int(context), float(ratio), ctypes.byref(e), ctypes.byref(n), ctypes.byref(b)),
           "kvr_paper_storage_split")
    return e.value, n.value, b.value


def kvr_layer_budgets(weights, context: int, ratio: float):
    """kvr_layer_budgets: per-layer budgets (list of int) proportional to the per-layer weights."""
    n = len(weights)
    w = (ctypes.c_double * n)(*[float(x) for x in weights])
    out = (i32_t * n)()
    _check(lib().kvr_layer_budgets(w, n, int(context), float(ratio), out), "kvr_layer_budgets")
    return [int(x) for x in out]


def kvr_sketch_set_combine(sk: Sketch, which: int):
    _check(lib().kvr_sketch_set_combine(sk.handle, int(which)), "kvr_sketch_set_combine")


def kvr_sketch_set_obs_window_causal(sk: Sketch, on: bool):
    _check(lib().kvr_sketch_set_obs_window_causal(sk.handle, int(bool(on))), "kvr_sketch_set_obs_window_causal")


def kvr_last_score_kernel(sk: Sketch) -> int:
    return int(lib().kvr_last_score_kernel(sk.handle))


def kvr_measure_pipe_peaks(stream=None):
    """(fp32 min/max lane-ops per second, shared-memory bytes read per second) measured on the current device."""
    out = (ctypes.c_double * 2)()
    _check(lib().kvr_measure_pipe_peaks(out, _stream(stream)), "kvr_measure_pipe_peaks")
    return float(out[0]), float(out[1])


def kvr_sketch_set_wait_test(sk: Sketch, wait_limit_ns: int, unannounced_bytes: int):
    _check(lib().kvr_sketch_set_wait_test(sk.handle, int(wait_limit_ns), int(unannounced_bytes)), "kvr_sketch_set_wait_test")


def kvr_launch_count(sk: Sketch) -> int:
    return int(lib().kvr_launch_count(sk.handle))


def _lead(sk: Sketch, layer: int):
    d = sk.desc
    return (d.n_layers, d.batch) if layer == KVR_ALL_LAYERS else (d.batch,)


def kvr_compress(sk: Sketch, layer: int, K, V, Qobs, budget: int, n_recent: int = 0, *, Kr=None, Vr=None,
                 ret_idx=None, stream=None):
    """kvr_compress.  K, V [.., H, N, D], Qobs [.., Hq, W, D] on the device; returns (Kr, Vr, ret_idx)
    (allocated here with torch unless given)."""
    d = sk.desc
    lead = _lead(sk, layer)
    N, W = K.shape[-2], Qobs.shape[-2]
    assert tuple(K.shape) == lead + (d.n_kv_heads, N, d.head_dim) and V.shape == K.shape, "K/V shape"
    assert tuple(Qobs.shape) == lead + (d.n_q_heads, W, d.head_dim), "Qobs shape"
    assert K.dtype == sk.torch_dtype and V.dtype == K.dtype and Qobs.dtype == K.dtype, "dtype"
    R = min(int(budget), N)
    if Kr is None:
        Kr = torch.empty(lead + (d.n_kv_heads, R, d.head_dim), dtype=K.dtype, device=K.device)
    if Vr is None:
        Vr = torch.empty_like(Kr)
    if ret_idx is None:
        ret_idx = torch.empty(lead + (d.n_kv_heads, R), dtype=torch.int32, device=K.device)
    st = lib().kvr_compress(sk.handle, layer, _ptr(K), _ptr(V), _ptr(Qobs), N, W, int(budget), int(n_recent),
                            _ptr(Kr) if R else None, _ptr(Vr) if R else None, _ptr(ret_idx) if R else None,
                            _stream(stream))
    _check(st, "kvr_compress")
    return Kr, Vr, ret_idx


def kvr_decode_attention(sk: Sketch, layer: int, q, Kr, Vr, ret_idx, *, softmax_scale: float = 0.0, out=None,
                         stream=None):
    """kvr_decode_attention.  q [.., Hq, D]; returns out [.., Hq, D] float32."""
    d = sk.desc
    lead = _lead(sk, layer)
    assert tuple(q.shape) == lead + (d.n_q_heads, d.head_dim) and q.dtype == sk.torch_dtype, "q shape/dtype"
    R = Kr.shape[-2]
    if out is None:
        out = torch.empty(lead + (d.n_q_heads, d.head_dim), dtype=torch.float32, device=q.device)
    st = lib().kvr_decode_attention(sk.handle, layer, _ptr(q), _ptr(Kr) if R else None, _ptr(Vr) if R else None,
                                    _ptr(ret_idx) if R else None, R, float(softmax_scale), _ptr(out),
                                    _stream(stream))
    _check(st, "kvr_decode_attention")
    return out


def kvr_decode_attention_scored(sk: Sketch, layer: int, q, Kr, Vr, ret_idx, score_acc, *, softmax_scale: float = 0.0,
                                out=None, stream=None):
    """kvr_decode_attention_scored: the decode call that also adds the step's attention mass to score_acc
    [.., H, n_rows] (float32, in place) and to the handle's per-token scores of the vague tokens."""
    d = sk.desc
    lead = _lead(sk, layer)
    assert tuple(q.shape) == lead + (d.n_q_heads, d.head_dim) and q.dtype == sk.torch_dtype, "q shape/dtype"
    R = Kr.shape[-2]
    assert score_acc.dtype == torch.float32 and score_acc.shape[-1] == R and score_acc.is_contiguous()
    if out is None:
        out = torch.empty(lead + (d.n_q_heads, d.head_dim), dtype=torch.float32, device=q.device)
    with torch.cuda.device(sk.device):
        st = lib().kvr_decode_attention_scored(sk.handle, layer, _ptr(q), _ptr(Kr) if R else None, _ptr(Vr) if R else None,
                                               _ptr(ret_idx) if R else None, R, float(softmax_scale), _ptr(out),
                                               _ptr(score_acc), _stream(stream))
    _check(st, "kvr_decode_attention_scored")
    return out


def kvr_decode_attention_mq(sk: Sketch, layer: int, q, Kr, Vr, ret_idx, *, causal: bool = True, softmax_scale: float = 0.0,
                            out=None, stream=None):
    """kvr_decode_attention_mq: q [.., n_q_heads, n_queries, head_dim] -> out of the same shape (float32)."""
    d = sk.desc
    lead = _lead(sk, layer)
    Qn = q.shape[-2]
    assert tuple(q.shape) == lead + (d.n_q_heads, Qn, d.head_dim) and q.dtype == sk.torch_dtype, "q shape/dtype"
    R = Kr.shape[-2]
    if out is None:
        out = torch.empty(lead + (d.n_q_heads, Qn, d.head_dim), dtype=torch.float32, device=q.device)
    with torch.cuda.device(sk.device):
        st = lib().kvr_decode_attention_mq(sk.handle, layer, _ptr(q), _ptr(Kr) if R else None, _ptr(Vr) if R else None,
                                           _ptr(ret_idx) if R else None, R, int(Qn), int(bool(causal)),
                                           float(softmax_scale), _ptr(out), _stream(stream))
    _check(st, "kvr_decode_attention_mq")
    return out


def kvr_decode_attention_static(sk: Sketch, layer: int, q, Kr, Vr, ret_idx, *, softmax_scale: float = 0.0,
                                out=None, stream=None):
    """kvr_decode_attention_static: the decode call that never allocates device memory (its scratch is
    a fixed array inside the library).  `out` should be passed in by callers that must not allocate;
    it is created with torch here only when omitted."""
    d = sk.desc
    lead = _lead(sk, layer)
    assert tuple(q.shape) == lead + (d.n_q_heads, d.head_dim) and q.dtype == sk.torch_dtype, "q shape/dtype"
    R = Kr.shape[-2]
    if out is None:
        out = torch.empty(lead + (d.n_q_heads, d.head_dim), dtype=torch.float32, device=q.device)
    st = lib().kvr_decode_attention_static(sk.handle, layer, _ptr(q), _ptr(Kr) if R else None,
                                           _ptr(Vr) if R else None, _ptr(ret_idx) if R else None, R,
                                           float(softmax_scale), _ptr(out), _stream(stream))
    _check(st, "kvr_decode_attention_static")
    return out


def kvr_accumulate_scores(sk: Sketch, layer: int, q, Kr, score_acc, *, softmax_scale: float = 0.0, stream=None):
    """kvr_accumulate_scores: adds the attention mass of the rows of Kr in the layer's last decode to
    score_acc [.., H, n_rows] (float32, in place)."""
    n_rows = Kr.shape[-2]
    assert score_acc.dtype == torch.float32 and score_acc.shape[-1] == n_rows
    st = lib().kvr_accumulate_scores(sk.handle, layer, _ptr(q), _ptr(Kr) if n_rows else None, n_rows,
                                     float(softmax_scale), _ptr(score_acc), _stream(stream))
    _check(st, "kvr_accumulate_scores")
    return score_acc


def kvr_demote(sk: Sketch, layer: int, Kr, Vr, ret_idx, row_scores, new_context: int, budget: int,
               n_recent: int = 0, stream=None):
    """kvr_demote: returns (Kr_out, Vr_out, ret_idx_out, row_scores_out) with `budget` rows."""
    n_rows = Kr.shape[-2]
    lead = tuple(Kr.shape[:-2])
    Kr_out = torch.empty(lead + (budget, Kr.shape[-1]), dtype=Kr.dtype, device=Kr.device)
    Vr_out = torch.empty_like(Kr_out)
    ret_out = torch.empty(lead + (budget,), dtype=torch.int32, device=Kr.device)
    sc_out = torch.empty(lead + (budget,), dtype=torch.float32, device=Kr.device)
    st = lib().kvr_demote(sk.handle, layer, _ptr(Kr), _ptr(Vr), _ptr(ret_idx), _ptr(row_scores), n_rows,
                          int(new_context), int(budget), int(n_recent), _ptr(Kr_out) if budget else None,
                          _ptr(Vr_out) if budget else None, _ptr(ret_out) if budget else None,
                          _ptr(sc_out) if budget else None, _stream(stream))
    _check(st, "kvr_demote")
    return Kr_out, Vr_out, ret_out, sc_out


def kvr_accumulate_vague_scores(sk: Sketch, layer: int, q, *, softmax_scale: float = 0.0, stream=None):
    """kvr_accumulate_vague_scores: adds the last decode's attention mass of the vague tokens to the
    handle's per-token scores (kvr_get_scores)."""
    with torch.cuda.device(sk.device):
        _check(lib().kvr_accumulate_vague_scores(sk.handle, layer, _ptr(q), float(softmax_scale), _stream(stream)),
               "kvr_accumulate_vague_scores")


def kvr_swap(sk: Sketch, layer: int, Kr, Vr, ret_idx, row_scores, n_recent: int = 0, replace_rate: float = 1.1,
             max_swaps: int = 1 << 30, stream=None):
    """kvr_swap: in place on Kr, Vr, ret_idx, row_scores; returns the swaps made per head-instance
    (int32 tensor shaped like ret_idx without its last axis)."""
    assert Kr.is_cuda and Kr.is_contiguous() and Vr.is_contiguous() and ret_idx.is_contiguous()
    assert row_scores.dtype == torch.float32 and row_scores.is_contiguous() and ret_idx.dtype == torch.int32
    n = torch.zeros(tuple(ret_idx.shape[:-1]), dtype=torch.int32, device=Kr.device)
    with torch.cuda.device(sk.device):
        st = lib().kvr_swap(sk.handle, layer, _ptr(Kr), _ptr(Vr), _ptr(ret_idx), _ptr(row_scores), Kr.shape[-2],
                            int(n_recent), float(replace_rate), int(min(max_swaps, 2 ** 31 - 1)), _ptr(n),
                            _stream(stream))
    _check(st, "kvr_swap")
    return n


def kvr_append_sizes(n_rows: int, n_recent: int, n_new: int, r_budget: int, c_budget: int, slack: int):
    """(rows_after, n_recent_after) of kvr_append, from the counts alone."""
    rec = ctypes.c_int32(0)
    n = lib().kvr_append_sizes(int(n_rows), int(n_recent), int(n_new), int(r_budget), int(c_budget), int(slack),
                               ctypes.byref(rec))
    if n < 0:
        raise KvrError(KVR_ERR_SHAPE, "kvr_append_sizes")
    return int(n), int(rec.value)


def kvr_append(sk: Sketch, layer: int, Kr, Vr, ret_idx, row_scores, n_recent: int, K_new, V_new, r_budget: int,
               c_budget: int, slack: int, replace_rate: float = 1.1, max_swaps: int = 1 << 30, stream=None):
    """kvr_append: Algorithm 3 for the new rows K_new, V_new.  Returns
    (Kr_out, Vr_out, ret_idx_out, row_scores_out, n_recent_after, n_swapped)."""
    n_rows, n_new = Kr.shape[-2], K_new.shape[-2]
    rows_after, rec_after = kvr_append_sizes(n_rows, n_recent, n_new, r_budget, c_budget, slack)
    lead = tuple(K_new.shape[:-2])
    Ko = torch.empty(lead + (rows_after, K_new.shape[-1]), dtype=K_new.dtype, device=K_new.device)
    Vo = torch.empty_like(Ko)
    ro = torch.empty(lead + (rows_after,), dtype=torch.int32, device=K_new.device)
    so = torch.empty(lead + (rows_after,), dtype=torch.float32, device=K_new.device)
    n = torch.zeros(lead, dtype=torch.int32, device=K_new.device)
    with torch.cuda.device(sk.device):
        st = lib().kvr_append(sk.handle, layer, _ptr(Kr) if n_rows else None, _ptr(Vr) if n_rows else None,
                              _ptr(ret_idx) if n_rows else None, _ptr(row_scores) if n_rows else None, n_rows,
                              int(n_recent), _ptr(K_new) if n_new else None, _ptr(V_new) if n_new else None, n_new,
                              int(r_budget), int(c_budget), int(slack), float(replace_rate),
                              int(min(max_swaps, 2 ** 31 - 1)), _ptr(Ko), _ptr(Vo), _ptr(ro), _ptr(so), _ptr(n),
                              _stream(stream))
    _check(st, "kvr_append")
    return Ko, Vo, ro, so, rec_after, n


def kvr_compress_host(sk: Sketch, layer: int, K, V, Qobs, budget: int, n_recent: int = 0, stream=None):
    """kvr_compress_host: K, V, Qobs are HOST tensors (pinned for full copy speed)."""
    assert not K.is_cuda and not V.is_cuda and not Qobs.is_cuda
    N, W = K.shape[-2], Qobs.shape[-2]
    with torch.cuda.device(sk.device):
        st = lib().kvr_compress_host(sk.handle, layer, _ptr(K), _ptr(V), _ptr(Qobs), N, W, int(budget),
                                     int(n_recent), _stream(stream))
    _check(st, "kvr_compress_host")


def kvr_decode_attention_host(sk: Sketch, layer: int, q, out, *, softmax_scale: float = 0.0, stream=None):
    """kvr_decode_attention_host: q and out are HOST tensors; returns out (filled on return)."""
    assert not q.is_cuda and not out.is_cuda and out.dtype == torch.float32
    with torch.cuda.device(sk.device):
        st = lib().kvr_decode_attention_host(sk.handle, layer, _ptr(q), float(softmax_scale), _ptr(out),
                                             _stream(stream))
    _check(st, "kvr_decode_attention_host")
    return out


def kvr_layer_shape(sk: Sketch, layer: int):
    N, R = ctypes.c_int32(0), ctypes.c_int32(0)
    _check(lib().kvr_layer_shape(sk.handle, layer, ctypes.byref(N), ctypes.byref(R)), "kvr_layer_shape")
    return N.value, R.value


def _layer_NR(sk: Sketch, layer: int):
    return kvr_layer_shape(sk, 0 if layer == KVR_ALL_LAYERS else layer)


def kvr_get_scores(sk: Sketch, layer: int, stream=None):
    d = sk.desc
    N, _ = _layer_NR(sk, layer)
    s = torch.empty(_lead(sk, layer) + (d.n_kv_heads, N), dtype=torch.float32, device=sk.device)
    _check(lib().kvr_get_scores(sk.handle, layer, _ptr(s), _stream(stream)), "kvr_get_scores")
    return s


def kvr_get_assignment(sk: Sketch, layer: int, stream=None):
    d = sk.desc
    N, R = _layer_NR(sk, layer)
    a = N - R
    lead = _lead(sk, layer) + (d.n_kv_heads,)
    cmp_idx = torch.empty(lead + (a,), dtype=torch.int32, device=sk.device)
    bucket = torch.empty(lead + (d.r, a), dtype=torch.int32, device=sk.device)
    sign = torch.empty(lead + (d.r, a), dtype=torch.int8, device=sk.device)
    _check(lib().kvr_get_assignment(sk.handle, layer, _ptr(cmp_idx), _ptr(bucket), _ptr(sign), _stream(stream)),
           "kvr_get_assignment")
    return cmp_idx, bucket, sign


def kvr_get_cells(sk: Sketch, layer: int, stream=None):
    d = sk.desc
    cells = torch.empty(_lead(sk, layer) + (d.n_kv_heads, 2, d.r, d.b, d.head_dim), dtype=torch.float32,
                        device=sk.device)
    _check(lib().kvr_get_cells(sk.handle, layer, _ptr(cells), _stream(stream)), "kvr_get_cells")
    return cells


def kvr_reconstruct(sk: Sketch, layer: int, stream=None):
    d = sk.desc
    N, R = _layer_NR(sk, layer)
    shape = _lead(sk, layer) + (d.n_kv_heads, N - R, d.head_dim)
    Kt = torch.empty(shape, dtype=torch.float32, device=sk.device)
    Vt = torch.empty(shape, dtype=torch.float32, device=sk.device)
    _check(lib().kvr_reconstruct(sk.handle, layer, _ptr(Kt), _ptr(Vt), _stream(stream)), "kvr_reconstruct")
    return Kt, Vt
