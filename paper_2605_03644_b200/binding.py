"""ctypes binding of libadapshot.so: same names as the C ABI, marshalling only.

Every step of the path runs inside the CUDA library.  Importing this module
raises if the library has not been built: there is no CPU fallback.
Tensors are torch CUDA tensors used as device memory; the current torch CUDA
stream is passed to every call.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libadapshot.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError(
        f"{_LIB_PATH} is missing: build it with `python -m paper_2605_03644_b200.build` "
        "(the CUDA library is the only implementation; there is no fallback)")
lib = C.CDLL(_LIB_PATH)

OK, EINVAL, ESHAPE, EALIGN, ECAPACITY, EUNSUPPORTED, ECUDA, EINDEX, ETIMEOUT = 0, -1, -2, -3, -4, -5, -6, -7, -8
F32, BF16 = 0, 1
ASSEMBLE_KEEP_PLAN = 1
ASSEMBLE_K_ONLY = 2

EXPORTS = [
    "adapshot_select_workspace_bytes", "adapshot_select", "adapshot_select_attn_workspace_bytes",
    "adapshot_select_attn", "adapshot_assemble_kv", "adapshot_assemble_kv_from",
    "adapshot_attn_workspace_bytes", "adapshot_query_attn",
    "adapshot_attn_fused_workspace_bytes", "adapshot_query_attn_fused",
    "adapshot_attn_vpool_workspace_bytes", "adapshot_query_attn_vpool",
    "adapshot_tree_layout", "adapshot_tree_attn", "adapshot_decode_workspace_bytes", "adapshot_decode_attn",
    "adapshot_entropy_workspace_bytes", "adapshot_entropy", "adapshot_entropy_subset",
    "adapshot_entropy_static",
    "adapshot_profile", "adapshot_profile_attn_main_ms", "adapshot_selftest_wait_timeout",
    "adapshot_strerror", "adapshot_version",
]


class ModelT(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("dtype", C.c_int32), ("k_pos_mode", C.c_int32),
                ("rope_base", C.c_double), ("softmax_scale", C.c_float), ("reserved", C.c_int32)]


class PoolT(C.Structure):
    _fields_ = [("n_shots", C.c_int32), ("emb_dim", C.c_int32), ("pool_tokens", C.c_int64),
                ("shot_off", C.c_void_p), ("k", C.c_void_p), ("v", C.c_void_p), ("emb", C.c_void_p)]


def _sig(name, restype, argtypes):
    fn = getattr(lib, name)
    fn.restype = restype
    fn.argtypes = argtypes
    return fn


_vp, _i32, _i64, _sz, _u32, _f = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t, C.c_uint32, C.c_float
_select_ws = _sig("adapshot_select_workspace_bytes", _sz, [_i32, _i32, _i32])
_select = _sig("adapshot_select", C.c_int, [C.POINTER(PoolT), _vp, _i32, _i32, _vp, _vp, _vp, _sz, _vp, _vp])
_select_attn_ws = _sig("adapshot_select_attn_workspace_bytes", _sz,
                       [C.POINTER(ModelT), C.POINTER(PoolT), _i32, _i32, _i32])
_select_attn = _sig("adapshot_select_attn", C.c_int,
                    [C.POINTER(ModelT), C.POINTER(PoolT), _i32, _vp, _i32, _i32, _i32, _u32, _vp, _vp, _vp, _sz,
                     _vp, _vp])
RELEVANCE_PER_TOKEN = 1
_assemble = _sig("adapshot_assemble_kv", C.c_int,
                 [C.POINTER(ModelT), C.POINTER(PoolT), _vp, _i32, _i32, _i32, _i32, _vp, _vp, _i64,
                  _vp, _u32, _vp, _vp])
_assemble_from = _sig("adapshot_assemble_kv_from", C.c_int,
                      [C.POINTER(ModelT), C.POINTER(PoolT), _vp, _i32, _i32, _i32, _i32, _i32, _vp, _vp, _i64,
                       _vp, _u32, _vp, _vp])
_entropy_ws = _sig("adapshot_entropy_workspace_bytes", _sz, [_i32, _i32])
_entropy = _sig("adapshot_entropy", C.c_int,
                [_vp, _i32, _i32, _i32, _i64, _vp, _f, _i32, _vp, _vp, _sz, _vp, _vp])
_entropy_subset = _sig("adapshot_entropy_subset", C.c_int,
                       [_vp, _i32, _i32, _i32, _i64, _vp, _i32, _u32, _vp, _f, _i32, _vp, _vp, _sz, _vp, _vp])
_entropy_static = _sig("adapshot_entropy_static", C.c_int,
                       [_vp, _i32, _i32, _i32, _i64, _vp, _f, _i32, _vp, _vp, _vp])
_strerror = _sig("adapshot_strerror", C.c_char_p, [C.c_int])
_version = _sig("adapshot_version", C.c_int, [])
_attn_ws = _sig("adapshot_attn_workspace_bytes", _sz, [C.POINTER(ModelT), _i32, _i32, _i32, _i32, _i64])
_attn = _sig("adapshot_query_attn", C.c_int,
             [C.POINTER(ModelT), _vp, _vp, _i64, _vp, _i32, _i32, C.POINTER(_i32), _i32,
              _vp, _vp, _vp, _i32, _i32, _i32, _vp, _vp, _u32, _vp, _sz, _vp, _vp])


_attn_fused_ws = _sig("adapshot_attn_fused_workspace_bytes", _sz,
                      [C.POINTER(ModelT), _i32, _i32, _i32, _i32, _i64])
_attn_fused = _sig("adapshot_query_attn_fused", C.c_int,
                   [C.POINTER(ModelT), C.POINTER(PoolT), _vp, _vp, _i64, _i32, _i32, C.POINTER(_i32), _i32,
                    _vp, _vp, _vp, _i32, _i32, _i32, _vp, _vp, _u32, _vp, _sz, _vp, _vp])


_attn_vpool_ws = _sig("adapshot_attn_vpool_workspace_bytes", _sz,
                      [C.POINTER(ModelT), _i32, _i32, _i32, _i32, _i64])
_attn_vpool = _sig("adapshot_query_attn_vpool", C.c_int,
                   [C.POINTER(ModelT), C.POINTER(PoolT), _vp, _vp, _i64, _vp, _i32, _i32, C.POINTER(_i32), _i32,
                    _vp, _vp, _vp, _i32, _i32, _i32, _vp, _vp, _u32, _vp, _sz, _vp, _vp])


_tree_layout = _sig("adapshot_tree_layout", C.c_int,
                    [C.POINTER(_i32), C.POINTER(_i32), _i32, _i32, C.POINTER(_i32), C.POINTER(_i32), C.POINTER(_i32)])
_tree_attn = _sig("adapshot_tree_attn", C.c_int,
                  [C.POINTER(ModelT), _vp, _vp, _i64, _vp, _i32, _i32, C.POINTER(_i32), C.POINTER(_i32), _i32,
                   _vp, _vp, _vp, _i32, _i32, _vp, _vp, _vp, _u32, _vp, _sz, _vp, _vp])
_decode_ws = _sig("adapshot_decode_workspace_bytes", _sz, [C.POINTER(ModelT), _i32, _i32, _i32, _i32])
_decode = _sig("adapshot_decode_attn", C.c_int,
               [C.POINTER(ModelT), _vp, _vp, _i64, _vp, _i32, _i32, _vp, _vp, _vp, _vp, _i32, _i32, _i32, _i32,
                _vp, _vp, _u32, _vp, _sz, _vp, _vp])
SEG_SHOTS, SEG_PROBE = 0, 1


_profile = _sig("adapshot_profile", C.c_int, [C.c_int])
_profile_ms = _sig("adapshot_profile_attn_main_ms", C.c_float, [])


def adapshot_profile(enable: bool):
    _check(_profile(1 if enable else 0))


def adapshot_profile_attn_main_ms() -> float:
    return float(_profile_ms())


_selftest = _sig("adapshot_selftest_wait_timeout", C.c_int, [_vp, _vp, _vp])


def adapshot_selftest_wait_timeout(status: torch.Tensor, cycles: torch.Tensor):
    _check(_selftest(_ptr(status), _ptr(cycles), _stream()))


class AdapshotError(RuntimeError):
    def __init__(self, code: int):
        self.code = code
        super().__init__(f"adapshot error {code}: {adapshot_strerror(code)}")


def adapshot_strerror(code: int) -> str:
    return _strerror(code).decode()


def adapshot_version() -> int:
    return _version()


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(rc: int):
    if rc != OK:
        raise AdapshotError(rc)


def make_model(n_layers, n_q_heads, n_kv_heads, head_dim, dtype, rope_base, k_pos_mode=0,
               softmax_scale=0.0) -> ModelT:
    dt = {torch.float32: F32, torch.bfloat16: BF16, "fp32": F32, "bf16": BF16}[dtype]
    return ModelT(n_layers, n_q_heads, n_kv_heads, head_dim, dt, k_pos_mode, float(rope_base),
                  float(softmax_scale), 0)


class Pool:
    """Holds the device tensors of a pool and the C struct that points at them."""

    def __init__(self, shot_off: torch.Tensor, k: Optional[torch.Tensor], v: Optional[torch.Tensor],
                 emb: Optional[torch.Tensor]):
        self.shot_off, self.k, self.v, self.emb = shot_off, k, v, emb
        n_shots = shot_off.numel() - 1
        tokens = int(k.shape[1]) if k is not None else 0
        self.c = PoolT(n_shots, int(emb.shape[1]) if emb is not None else 0, tokens,
                       _ptr(shot_off), _ptr(k), _ptr(v), _ptr(emb))


def adapshot_select_workspace_bytes(n_shots: int, B: int, k: int) -> int:
    return _select_ws(n_shots, B, k)


def adapshot_select(pool: Pool, q_emb: torch.Tensor, k: int, sel_idx: torch.Tensor,
                    sel_score: Optional[torch.Tensor], ws: torch.Tensor, status: torch.Tensor):
    B = q_emb.shape[0]
    _check(_select(C.byref(pool.c), _ptr(q_emb), B, k, _ptr(sel_idx), _ptr(sel_score),
                   _ptr(ws), ws.numel() * ws.element_size(), _ptr(status), _stream()))


def adapshot_select_attn_workspace_bytes(model: ModelT, pool: Pool, B: int, Tq: int, k: int) -> int:
    return _select_attn_ws(C.byref(model), C.byref(pool.c), B, Tq, k)


def adapshot_select_attn(model: ModelT, pool: Pool, layer: int, q: torch.Tensor, k: int, sel_idx: torch.Tensor,
                         sel_score: Optional[torch.Tensor], ws: torch.Tensor, status: torch.Tensor,
                         per_token: bool = False):
    """Top-k by attention mass (Sec. 4.2): q [B][T_q][Hq][d] bf16 against the pool's K at `layer`."""
    B, Tq = q.shape[0], q.shape[1]
    _check(_select_attn(C.byref(model), C.byref(pool.c), layer, _ptr(q), B, Tq, k,
                        RELEVANCE_PER_TOKEN if per_token else 0, _ptr(sel_idx), _ptr(sel_score), _ptr(ws),
                        ws.numel() * ws.element_size(), _ptr(status), _stream()))


def adapshot_assemble_kv(model: ModelT, pool: Pool, sel_idx: torch.Tensor, layer_begin: int,
                         layer_end: int, k_ctx: Optional[torch.Tensor], v_ctx: Optional[torch.Tensor],
                         ctx_cap: int, ctx_off: torch.Tensor, status: torch.Tensor, flags: int = 0):
    B, k = sel_idx.shape
    _check(_assemble(C.byref(model), C.byref(pool.c), _ptr(sel_idx), B, k, layer_begin, layer_end,
                     _ptr(k_ctx), _ptr(v_ctx), ctx_cap, _ptr(ctx_off), flags, _ptr(status), _stream()))


def adapshot_assemble_kv_from(model: ModelT, pool: Pool, sel_idx: torch.Tensor, shot_begin: int,
                              layer_begin: int, layer_end: int, k_ctx: torch.Tensor, v_ctx: torch.Tensor,
                              ctx_cap: int, ctx_off: torch.Tensor, status: torch.Tensor, flags: int = 0):
    B, k = sel_idx.shape
    _check(_assemble_from(C.byref(model), C.byref(pool.c), _ptr(sel_idx), B, k, shot_begin, layer_begin,
                          layer_end, _ptr(k_ctx), _ptr(v_ctx), ctx_cap, _ptr(ctx_off), flags, _ptr(status),
                          _stream()))


def adapshot_attn_workspace_bytes(model: ModelT, B: int, P: int, Tq: int, n_layers_in_call: int,
                                  ctx_cap: int) -> int:
    return _attn_ws(C.byref(model), B, P, Tq, n_layers_in_call, ctx_cap)


def adapshot_query_attn(model: ModelT, k_ctx: torch.Tensor, v_ctx: torch.Tensor, ctx_cap: int,
                        ctx_off: torch.Tensor, k: int, probe_nshots: Sequence[int],
                        q: torch.Tensor, kq: torch.Tensor, vq: torch.Tensor,
                        layer_begin: int, layer_end: int, out: torch.Tensor,
                        lse: Optional[torch.Tensor], ws: torch.Tensor, status: torch.Tensor,
                        flags: int = 0):
    B = q.shape[0]
    P = len(probe_nshots)
    Tq = q.shape[3]
    arr = (_i32 * P)(*[int(x) for x in probe_nshots])
    _check(_attn(C.byref(model), _ptr(k_ctx), _ptr(v_ctx), ctx_cap, _ptr(ctx_off), B, k, arr, P,
                 _ptr(q), _ptr(kq), _ptr(vq), Tq, layer_begin, layer_end, _ptr(out), _ptr(lse),
                 flags, _ptr(ws), ws.numel() * ws.element_size(), _ptr(status), _stream()))


def adapshot_attn_fused_workspace_bytes(model: ModelT, B: int, P: int, Tq: int, n_layers_in_call: int,
                                        ctx_cap: int) -> int:
    return _attn_fused_ws(C.byref(model), B, P, Tq, n_layers_in_call, ctx_cap)


def adapshot_query_attn_fused(model: ModelT, pool: Pool, sel_idx: torch.Tensor, ctx_off: torch.Tensor,
                              ctx_cap: int, probe_nshots: Sequence[int], q: torch.Tensor, kq: torch.Tensor,
                              vq: torch.Tensor, layer_begin: int, layer_end: int, out: torch.Tensor,
                              lse: Optional[torch.Tensor], ws: torch.Tensor, status: torch.Tensor,
                              flags: int = 0):
    B, k = sel_idx.shape
    P = len(probe_nshots)
    Tq = q.shape[3]
    arr = (_i32 * P)(*[int(x) for x in probe_nshots])
    _check(_attn_fused(C.byref(model), C.byref(pool.c), _ptr(sel_idx), _ptr(ctx_off), ctx_cap, B, k, arr, P,
                       _ptr(q), _ptr(kq), _ptr(vq), Tq, layer_begin, layer_end, _ptr(out), _ptr(lse),
                       flags, _ptr(ws), ws.numel() * ws.element_size(), _ptr(status), _stream()))


def adapshot_attn_vpool_workspace_bytes(model: ModelT, B: int, P: int, Tq: int, n_layers_in_call: int,
                                        ctx_cap: int) -> int:
    return _attn_vpool_ws(C.byref(model), B, P, Tq, n_layers_in_call, ctx_cap)


def adapshot_query_attn_vpool(model: ModelT, pool: Pool, sel_idx: torch.Tensor, k_ctx: torch.Tensor,
                              ctx_cap: int, ctx_off: torch.Tensor, probe_nshots: Sequence[int],
                              q: torch.Tensor, kq: torch.Tensor, vq: torch.Tensor, layer_begin: int,
                              layer_end: int, out: torch.Tensor, lse: Optional[torch.Tensor], ws: torch.Tensor,
                              status: torch.Tensor, flags: int = 0):
    B, k = sel_idx.shape
    P = len(probe_nshots)
    Tq = q.shape[3]
    arr = (_i32 * P)(*[int(x) for x in probe_nshots])
    _check(_attn_vpool(C.byref(model), C.byref(pool.c), _ptr(sel_idx), _ptr(k_ctx), ctx_cap, _ptr(ctx_off), B, k,
                       arr, P, _ptr(q), _ptr(kq), _ptr(vq), Tq, layer_begin, layer_end, _ptr(out), _ptr(lse),
                       flags, _ptr(ws), ws.numel() * ws.element_size(), _ptr(status), _stream()))


def _seg_arrays(segments):
    n = len(segments)
    kinds = (_i32 * n)(*[int(kd) for kd, _ in segments])
    lens = (_i32 * n)(*[int(ln) for _, ln in segments])
    return kinds, lens, n


def adapshot_tree_layout(segments, k: int):
    """Parses a segment table [(SEG_SHOTS, n shots) | (SEG_PROBE, tokens), ...] of the interleaved
    sequence; returns (probe shot counts, tokens per probe)."""
    kinds, lens, n = _seg_arrays(segments)
    probes = (_i32 * 16)()
    P, Tq = _i32(0), _i32(0)
    _check(_tree_layout(kinds, lens, n, k, probes, C.byref(P), C.byref(Tq)))
    return [int(probes[i]) for i in range(P.value)], int(Tq.value)


def adapshot_tree_attn(model: ModelT, k_ctx: torch.Tensor, v_ctx: torch.Tensor, ctx_cap: int,
                       ctx_off: torch.Tensor, k: int, segments, q_seq: torch.Tensor, kq_seq: torch.Tensor,
                       vq_seq: torch.Tensor, layer_begin: int, layer_end: int, out_seq: torch.Tensor,
                       lse: Optional[torch.Tensor], pos_seq: Optional[torch.Tensor], ws: torch.Tensor,
                       status: torch.Tensor, flags: int = 0):
    B = q_seq.shape[0]
    kinds, lens, n = _seg_arrays(segments)
    _check(_tree_attn(C.byref(model), _ptr(k_ctx), _ptr(v_ctx), ctx_cap, _ptr(ctx_off), B, k, kinds, lens, n,
                      _ptr(q_seq), _ptr(kq_seq), _ptr(vq_seq), layer_begin, layer_end, _ptr(out_seq), _ptr(lse),
                      _ptr(pos_seq), flags, _ptr(ws), ws.numel() * ws.element_size(), _ptr(status), _stream()))


def adapshot_decode_workspace_bytes(model: ModelT, B: int, T_new: int, T_own: int, n_layers_in_call: int) -> int:
    return _decode_ws(C.byref(model), B, T_new, T_own, n_layers_in_call)


def adapshot_decode_attn(model: ModelT, k_ctx: torch.Tensor, v_ctx: torch.Tensor, ctx_cap: int,
                         ctx_off: torch.Tensor, k: int, n_shots: torch.Tensor, q_new: torch.Tensor,
                         k_own: torch.Tensor, v_own: torch.Tensor, layer_begin: int, layer_end: int,
                         out: torch.Tensor, lse: Optional[torch.Tensor], ws: torch.Tensor, status: torch.Tensor,
                         flags: int = 0):
    B, T_new, T_own = q_new.shape[0], q_new.shape[2], k_own.shape[2]
    if n_shots.dtype != torch.int32:
        raise ValueError("n_shots must be int32")
    _check(_decode(C.byref(model), _ptr(k_ctx), _ptr(v_ctx), ctx_cap, _ptr(ctx_off), B, k, _ptr(n_shots),
                   _ptr(q_new), _ptr(k_own), _ptr(v_own), T_new, T_own, layer_begin, layer_end, _ptr(out),
                   _ptr(lse), flags, _ptr(ws), ws.numel() * ws.element_size(), _ptr(status), _stream()))


def adapshot_entropy_workspace_bytes(R: int, V: int) -> int:
    return _entropy_ws(R, V)


def adapshot_entropy(logits: torch.Tensor, H: torch.Tensor, tau: float, rows_per_group: int,
                     first_ok: Optional[torch.Tensor], ws: torch.Tensor, status: torch.Tensor):
    R, V = logits.shape
    dt = F32 if logits.dtype == torch.float32 else BF16
    if logits.stride(1) != 1:
        raise ValueError("logit rows must be contiguous")
    _check(_entropy(logits.data_ptr(), dt, R, V, logits.stride(0), _ptr(H), tau, rows_per_group,
                    _ptr(first_ok), _ptr(ws), ws.numel() * ws.element_size(), _ptr(status), _stream()))


def adapshot_entropy_subset(logits: torch.Tensor, subset_ids: torch.Tensor, H: torch.Tensor, tau: float,
                            rows_per_group: int, first_ok: Optional[torch.Tensor], ws: torch.Tensor,
                            status: torch.Tensor, renorm: bool = False):
    R, V = logits.shape
    dt = F32 if logits.dtype == torch.float32 else BF16
    if logits.stride(1) != 1 or subset_ids.dtype != torch.int32:
        raise ValueError("logit rows must be contiguous and subset_ids int32")
    _check(_entropy_subset(logits.data_ptr(), dt, R, V, logits.stride(0), _ptr(subset_ids), subset_ids.numel(),
                           1 if renorm else 0, _ptr(H), tau, rows_per_group, _ptr(first_ok), _ptr(ws),
                           ws.numel() * ws.element_size(), _ptr(status), _stream()))


def adapshot_entropy_static(logits: torch.Tensor, H: torch.Tensor, tau: float, rows_per_group: int,
                            first_ok: Optional[torch.Tensor], status: torch.Tensor):
    """adapshot_entropy for callers that may not allocate or pass scratch memory (for
    instance code inside a server whose allocator owns all device memory): the scratch
    is a fixed array inside the library.  Raises AdapshotError(ECAPACITY) beyond its
    size.  Calls share that array, so do not let two of them overlap on the GPU."""
    R, V = logits.shape
    dt = F32 if logits.dtype == torch.float32 else BF16
    if logits.stride(1) != 1:
        raise ValueError("logit rows must be contiguous")
    _check(_entropy_static(logits.data_ptr(), dt, R, V, logits.stride(0), _ptr(H), tau, rows_per_group,
                           _ptr(first_ok), _ptr(status), _stream()))
