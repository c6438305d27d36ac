"""ctypes binding of libsagekv.so (include/sagekv.h).

Argument marshalling only: every function below has the name and the meaning of
the C entry point it calls, takes torch CUDA tensors for the device buffers and
passes their pointers, strides and the current CUDA stream through.  Nothing is
computed here, and there is no fallback: importing this module raises if the
library has not been built (`python -m paper_2503_08879_b200.build`), and every
call raises `SagekvError` on a non-zero return code.
"""

from __future__ import annotations

import ctypes as C
import os

import torch

# SAGEKV_LIB selects another build of the same interface (the checked build, libsagekv_checked.so)
_LIB_PATH = os.environ.get("SAGEKV_LIB") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "libsagekv.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError(
        f"{_LIB_PATH} is missing: build it with `python -m paper_2503_08879_b200.build` "
        "(nvcc, sm_100a). There is no CPU or PyTorch fallback.")
lib = C.CDLL(_LIB_PATH)

OK, ERR_INVALID, ERR_ALIGN, ERR_UNSUPPORTED, ERR_CUDA, ERR_NOMEM = 0, -1, -2, -3, -4, -5
ERR_TOO_LARGE, ERR_TIMEOUT, ERR_BOUNDS, ERR_DEVICE = -6, -7, -8, -9


class Shape(C.Structure):
    _fields_ = [("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("batch", C.c_int32), ("softmax_scale", C.c_float)]


class Strides(C.Structure):
    _fields_ = [("batch_stride", C.c_int64), ("head_stride", C.c_int64), ("token_stride", C.c_int64)]


class CacheState(C.Structure):
    _fields_ = [("n_init", C.c_int32), ("k_q", C.c_int32), ("n_sel", C.c_int32), ("n_recent", C.c_int32),
                ("ring_len", C.c_int32), ("len", C.c_int32), ("d_step", C.c_void_p)]


_vp, _i32, _i64 = C.c_void_p, C.c_int32, C.c_int64
lib.sagekv_create.argtypes = [C.POINTER(_vp), C.POINTER(Shape), _i64, _i32]
lib.sagekv_destroy.argtypes = [_vp]
lib.sagekv_budget_split.argtypes = [_i32, _i32, C.POINTER(_i32), C.POINTER(_i32), C.POINTER(_i32)]
lib.sagekv_score.argtypes = [_vp, _vp, _vp, Strides, _i64, _i32, _i32, _vp, _i64, _vp]
lib.sagekv_select_compact.argtypes = [_vp, _vp, _i64, _vp, _vp, Strides, _i64, _i32, _i32, _i32,
                                      _vp, _vp, _vp, Strides, C.POINTER(CacheState), _vp]
lib.sagekv_decode_attn.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, Strides, C.POINTER(CacheState), _vp, _vp, _vp]
lib.sagekv_score_static.argtypes = [C.POINTER(Shape), _vp, _vp, Strides, _i64, _i32, _i32, _vp, _i64, _vp]
lib.sagekv_score_static.restype = C.c_int
lib.sagekv_set_overlap.argtypes = [_vp, C.c_int]
lib.sagekv_set_overlap.restype = C.c_int
lib.sagekv_set_decode_variant.argtypes = [_vp, C.c_int]
lib.sagekv_set_decode_variant.restype = C.c_int
lib.sagekv_set_select_overlap.argtypes = [_vp, C.c_int]
lib.sagekv_set_select_overlap.restype = C.c_int
lib.sagekv_set_select_hint.argtypes = [_vp, C.c_int, _i32]
lib.sagekv_set_select_hint.restype = C.c_int
lib.sagekv_scores_row_stride.argtypes = [_vp, _i64, _i32, _i32]
lib.sagekv_scores_row_stride.restype = _i64
lib.sagekv_set_group_mode.argtypes = [_vp, C.c_int]
lib.sagekv_set_group_mode.restype = C.c_int
lib.sagekv_pool_scores.argtypes = [_vp, _vp, _i64, _i64, _i32, _i32, _vp, _i64, _vp]
lib.sagekv_pool_scores.restype = C.c_int
lib.sagekv_compact_window_rope.argtypes = [_vp, _vp, _vp, Strides, _i64, _i32, _i32, C.c_float, _vp, _vp, Strides,
                                           C.POINTER(CacheState), _vp]
lib.sagekv_compact_window_rope.restype = C.c_int
lib.sagekv_quest_build.argtypes = [_vp, _vp, Strides, _i64, _i32, _i32, _vp, _vp, _vp]
lib.sagekv_quest_build.restype = C.c_int
lib.sagekv_quest_bounds.argtypes = [_vp, _vp, _vp, _vp, _i64, _vp, _i64, _vp]
lib.sagekv_quest_bounds.restype = C.c_int
lib.sagekv_select_topk.argtypes = [_vp, _vp, _i64, _i64, _i32, _vp, _vp]
lib.sagekv_select_topk.restype = C.c_int
lib.sagekv_status.argtypes = [_vp, C.POINTER(_i32)]
lib.sagekv_status.restype = C.c_int
lib.sagekv_status_code.argtypes = [_i32]
lib.sagekv_status_code.restype = C.c_int
lib.sagekv_checked_build.argtypes = []
lib.sagekv_checked_build.restype = C.c_int
lib.sagekv_strerror.argtypes = [C.c_int]
lib.sagekv_strerror.restype = C.c_char_p
lib.sagekv_last_cuda_error.argtypes = [_vp]
for _f in (lib.sagekv_create, lib.sagekv_destroy, lib.sagekv_budget_split, lib.sagekv_score,
           lib.sagekv_select_compact, lib.sagekv_decode_attn, lib.sagekv_last_cuda_error):
    _f.restype = C.c_int


class SagekvError(RuntimeError):
    def __init__(self, code: int, where: str, cuda_error: int = 0):
        self.code = code
        msg = f"{where}: {lib.sagekv_strerror(code).decode()} ({code})"
        if cuda_error:
            msg += f", cudaError {cuda_error}"
        super().__init__(msg)


def _check(code: int, where: str, ctx=None):
    if code != OK:
        raise SagekvError(code, where, lib.sagekv_last_cuda_error(ctx) if ctx else 0)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _kv_strides(t: torch.Tensor) -> Strides:
    """Strides of a [B, H_kv, tokens, 128] tensor whose last dimension is contiguous."""
    if t.dim() != 4 or t.stride(3) != 1:
        raise ValueError("expected a [B, H_kv, tokens, head_dim] tensor with contiguous head_dim")
    return Strides(t.stride(0), t.stride(1), t.stride(2))


def sagekv_budget_split(B: int, G: int):
    a, b, c = _i32(), _i32(), _i32()
    _check(lib.sagekv_budget_split(B, G, C.byref(a), C.byref(b), C.byref(c)), "sagekv_budget_split")
    return a.value, b.value, c.value


def sagekv_create(n_q_heads: int, n_kv_heads: int, head_dim: int, batch: int, max_ctx: int, max_len: int,
                  softmax_scale: float = 0.0):
    h = _vp()
    shape = Shape(n_q_heads, n_kv_heads, head_dim, batch, softmax_scale)
    _check(lib.sagekv_create(C.byref(h), C.byref(shape), max_ctx, max_len), "sagekv_create")
    return h


def sagekv_destroy(ctx):
    _check(lib.sagekv_destroy(ctx), "sagekv_destroy")


def sagekv_score(ctx, q_last, K, n_ctx: int, n_init: int, n_recent: int, scores, scores_row_stride: int):
    _check(lib.sagekv_score(ctx, _ptr(q_last), _ptr(K), _kv_strides(K), n_ctx, n_init, n_recent, _ptr(scores),
                            scores_row_stride, _stream()), "sagekv_score", ctx)


def sagekv_set_overlap(ctx, mode: int):
    _check(lib.sagekv_set_overlap(ctx, mode), "sagekv_set_overlap", ctx)


def sagekv_set_decode_variant(ctx, variant: int):
    _check(lib.sagekv_set_decode_variant(ctx, variant), "sagekv_set_decode_variant", ctx)


def sagekv_set_select_overlap(ctx, mode: int):
    _check(lib.sagekv_set_select_overlap(ctx, mode), "sagekv_set_select_overlap", ctx)


def sagekv_set_select_hint(ctx, mode: int, k: int = 0):
    _check(lib.sagekv_set_select_hint(ctx, mode, k), "sagekv_set_select_hint", ctx)


def sagekv_scores_row_stride(ctx, n_ctx: int, n_init: int, n_recent: int) -> int:
    r = lib.sagekv_scores_row_stride(ctx, n_ctx, n_init, n_recent)
    if r < 0:
        _check(int(r), "sagekv_scores_row_stride", ctx)
    return int(r)


def sagekv_set_group_mode(ctx, mode: int):
    _check(lib.sagekv_set_group_mode(ctx, mode), "sagekv_set_group_mode", ctx)


def sagekv_pool_scores(ctx, scores, scores_row_stride: int, n_ctx: int, n_init: int, n_recent: int, pooled,
                       pooled_row_stride: int):
    _check(lib.sagekv_pool_scores(ctx, _ptr(scores), scores_row_stride, n_ctx, n_init, n_recent, _ptr(pooled),
                                  pooled_row_stride, _stream()), "sagekv_pool_scores", ctx)


def sagekv_compact_window_rope(ctx, K_pre, V, n_ctx: int, n_init: int, n_recent: int, rope_theta: float, Kc, Vc,
                               state: CacheState):
    _check(lib.sagekv_compact_window_rope(ctx, _ptr(K_pre), _ptr(V), _kv_strides(K_pre), n_ctx, n_init, n_recent,
                                          rope_theta, _ptr(Kc), _ptr(Vc), _kv_strides(Kc), C.byref(state), _stream()),
           "sagekv_compact_window_rope", ctx)


def sagekv_quest_build(ctx, K, n_ctx: int, n_init: int, n_recent: int, kmin, kmax):
    _check(lib.sagekv_quest_build(ctx, _ptr(K), _kv_strides(K), n_ctx, n_init, n_recent, _ptr(kmin), _ptr(kmax), _stream()),
           "sagekv_quest_build", ctx)


def sagekv_quest_bounds(ctx, q, kmin, kmax, n_blocks: int, bounds, bounds_row_stride: int):
    _check(lib.sagekv_quest_bounds(ctx, _ptr(q), _ptr(kmin), _ptr(kmax), n_blocks, _ptr(bounds), bounds_row_stride,
                                   _stream()), "sagekv_quest_bounds", ctx)


def sagekv_select_topk(ctx, scores, scores_row_stride: int, n: int, k_q: int, idx):
    _check(lib.sagekv_select_topk(ctx, _ptr(scores), scores_row_stride, n, k_q, _ptr(idx), _stream()),
           "sagekv_select_topk", ctx)


def sagekv_status(ctx) -> int:
    """The context's device status word (0 = clean); raises SagekvError if any bit is set."""
    bits = _i32(0)
    code = lib.sagekv_status(ctx, C.byref(bits))
    if code != OK:
        e = SagekvError(code, "sagekv_status (word %d)" % bits.value, lib.sagekv_last_cuda_error(ctx))
        e.bits = bits.value
        raise e
    return bits.value


def sagekv_score_static(shape: Shape, q_last, K, n_ctx: int, n_init: int, n_recent: int, scores,
                        scores_row_stride: int):
    """sagekv_score without a context or any allocation: the partials live in the library's fixed array."""
    _check(lib.sagekv_score_static(C.byref(shape), _ptr(q_last), _ptr(K), _kv_strides(K), n_ctx, n_init, n_recent,
                                   _ptr(scores), scores_row_stride, _stream()), "sagekv_score_static")


def sagekv_select_compact(ctx, scores, scores_row_stride: int, K, V, n_ctx: int, n_init: int, n_recent: int, k: int,
                          idx, Kc, Vc, state: CacheState):
    _check(lib.sagekv_select_compact(ctx, _ptr(scores), scores_row_stride, _ptr(K), _ptr(V), _kv_strides(K), n_ctx,
                                     n_init, n_recent, k, _ptr(idx), _ptr(Kc), _ptr(Vc), _kv_strides(Kc),
                                     C.byref(state), _stream()), "sagekv_select_compact", ctx)


def sagekv_decode_attn(ctx, q, k_new, v_new, Kc, Vc, state: CacheState, out, lse=None):
    _check(lib.sagekv_decode_attn(ctx, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(Kc), _ptr(Vc), _kv_strides(Kc),
                                  C.byref(state), _ptr(out), _ptr(lse), _stream()), "sagekv_decode_attn", ctx)


class Layer:
    """Buffers of one layer's reduced cache (allocated with torch) plus the C state struct."""

    def __init__(self, batch, n_q_heads, n_kv_heads, head_dim, L_cap, k_q_cap, device):
        self.Kc = torch.zeros(batch, n_kv_heads, L_cap, head_dim, dtype=torch.bfloat16, device=device)
        self.Vc = torch.zeros_like(self.Kc)
        self.idx = torch.zeros(batch, n_q_heads, max(1, k_q_cap), dtype=torch.int32, device=device)
        self.step = torch.zeros(1, dtype=torch.int32, device=device)
        self.state = CacheState(0, 0, 0, 0, 0, 0, self.step.data_ptr())

    def indices(self) -> torch.Tensor:
        """Selected positions as [B, H_q, k_q] for the k_q the last select_compact call used."""
        B, Hq = self.idx.shape[0], self.idx.shape[1]
        k_q = self.state.k_q
        return self.idx.flatten()[: B * Hq * k_q].view(B, Hq, k_q)

    def cache(self):
        """(Kc, Vc) cut to the L rows in use."""
        return self.Kc[:, :, : self.state.len], self.Vc[:, :, : self.state.len]


class SageKV:
    """Convenience wrapper: one context, the caller's tensors, the four steps in order."""

    def __init__(self, n_q_heads, n_kv_heads, head_dim=128, batch=1, max_ctx=131072, max_len=8193,
                 softmax_scale=0.0, device="cuda"):
        self.device = torch.device(device)
        self.shape = (n_q_heads, n_kv_heads, head_dim, batch)
        self.G = n_q_heads // n_kv_heads
        with torch.cuda.device(self.device):
            self.ctx = sagekv_create(n_q_heads, n_kv_heads, head_dim, batch, max_ctx, max_len, softmax_scale)

    def set_overlap(self, mode: int):
        sagekv_set_overlap(self.ctx, mode)

    def set_decode_variant(self, variant: int):
        sagekv_set_decode_variant(self.ctx, variant)

    def set_select_overlap(self, mode: int):
        sagekv_set_select_overlap(self.ctx, mode)

    def set_select_hint(self, mode: int, k: int = 0):
        sagekv_set_select_hint(self.ctx, mode, k)

    def status(self) -> int:
        return sagekv_status(self.ctx)

    def close(self):
        if self.ctx is not None:
            sagekv_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def score_stride(self, n_ctx: int, n_init: int, n_recent: int) -> int:
        """Row stride of a score buffer for this context's hint mode (sagekv_scores_row_stride)."""
        return sagekv_scores_row_stride(self.ctx, n_ctx, n_init, n_recent)

    def new_scores(self, n_ctx: int, n_init: int, n_recent: int) -> torch.Tensor:
        Hq, _, _, B = self.shape
        return torch.empty(B * Hq, self.score_stride(n_ctx, n_init, n_recent), dtype=torch.float32,
                           device=self.device)

    def new_layer(self, n_init: int, n_recent: int, k: int, spare_rows: int = 0) -> Layer:
        """Buffers for a reduced cache of L = n_init + k + n_recent + 1 rows (plus `spare_rows` unused ones)."""
        Hq, Hkv, d, B = self.shape
        return Layer(B, Hq, Hkv, d, n_init + k + n_recent + 1 + spare_rows, k // self.G, self.device)

    def score(self, q_last, K, n_init, n_recent, scores=None):
        n_ctx = K.shape[2]
        if scores is None:
            scores = self.new_scores(n_ctx, n_init, n_recent)
        sagekv_score(self.ctx, q_last, K, n_ctx, n_init, n_recent, scores, scores.stride(0))
        return scores

    def select_compact(self, scores, K, V, n_init, n_recent, k, layer: Layer = None):
        if layer is None:
            layer = self.new_layer(n_init, n_recent, k)
        sagekv_select_compact(self.ctx, scores, scores.stride(0) if scores is not None else 0, K, V, K.shape[2],
                              n_init, n_recent, k, layer.idx, layer.Kc, layer.Vc, layer.state)
        return layer

    def decode_attn(self, q, k_new, v_new, layer: Layer, out=None, lse=None):
        if out is None:
            out = torch.empty_like(q)
        sagekv_decode_attn(self.ctx, q, k_new, v_new, layer.Kc, layer.Vc, layer.state, out, lse)
        return out
