"""ctypes binding of libgoodspeed.so: same names as include/goodspeed.h, argument marshalling only.

Every function takes torch tensors that already live on the CUDA device (or, where the header
says "host", on the CPU), checks dtype/contiguity, and passes raw pointers plus the current CUDA
stream.  No arithmetic of the verification path happens in Python.  If the shared library has
not been built, the first call raises; there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libgoodspeed.so")
GS_F32, GS_BF16 = 0, 1
GS_OK = 0
STATUS_NAMES = {0: "GS_OK", 1: "GS_ERR_INVALID_ARG", 2: "GS_ERR_SHAPE", 3: "GS_ERR_UNSUPPORTED",
                4: "GS_ERR_WORKSPACE", 5: "GS_ERR_CUDA", 6: "GS_ERR_TIMEOUT"}

_vp, _i, _f, _d, _sz = C.c_void_p, C.c_int, C.c_float, C.c_double, C.c_size_t

# name -> (restype, argtypes); mirrors include/goodspeed.h
SIGNATURES = {
    "gs_status_str": (C.c_char_p, [_i]),
    "gs_version": (_i, []),
    "gs_verify_attn_workspace": (_sz, [_i, _i, _i, _i, _i, _i, _i, _i]),
    "gs_verify_attn": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _i, _f, _i,
                            _vp, _sz, _vp, _vp]),
    "gs_verify_attn_paged_workspace": (_sz, [_i, _i, _i, _i, _i, _i, _i]),
    "gs_verify_attn_paged": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _i, _i, _f, _i,
                                  _vp, _sz, _vp, _vp]),
    "gs_lm_head_workspace": (_sz, [_i, _i, _i, _i]),
    "gs_lm_head_configure": (_i, [_i, _i, _i]),
    "gs_lm_head_select": (_i, [_i]),
    "gs_spec_accept_select": (_i, [_i]),
    "gs_verify_attn_configure": (_i, [_i]),
    "gs_verify_attn_select": (_i, [_i]),
    "gs_schedule_select": (_i, [_i]),
    "gs_set_dependent_launch": (_i, [_i]),
    "gs_lm_head_logits": (_i, [_vp, _vp, _vp, _i, _i, _i, _i, _vp, _sz, _vp, _vp]),
    "gs_lm_head_logits_w4": (_i, [_vp, _vp, _vp, _vp, _i, _vp, _i, _i, _i, _vp, _vp]),
    "gs_spec_accept_workspace": (_sz, [_i, _i, _i]),
    "gs_spec_accept": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _f, _i, _i, _i,
                            _vp, _vp, _vp, _vp, _vp, _vp,
                            _vp, _vp, _d, _d, _d, _d, _vp, _sz, _vp, _vp]),
    "gs_spec_accept_prestats": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _f, _i, _i, _i,
                                     _vp, _vp, _vp, _vp, _vp, _vp,
                                     _vp, _vp, _d, _d, _d, _d, _vp, _i, _vp, _sz, _vp, _vp]),
    "gs_lm_head_stats_bytes": (_sz, [_i]),
    "gs_lm_head_stats_pays": (_i, [_i]),
    "gs_lm_head_logits_stats": (_i, [_vp, _vp, _vp, _i, _i, _i, _i, _f, _vp, _sz, C.POINTER(C.c_int),
                                     _vp, _sz, _vp, _vp]),
    "gs_spec_accept_static_capacity": (_sz, []),
    "gs_spec_accept_static": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _f, _i, _i, _i,
                                   _vp, _vp, _vp, _vp, _vp, _vp,
                                   _vp, _vp, _d, _d, _d, _d, _vp, _vp]),
    "gs_schedule": (_i, [_vp, _vp, _i, _i, _vp, _vp, _vp, _vp, _vp]),
    "gs_schedule_host": (_i, [_vp, _vp, _i, _i, _vp, _vp, _vp]),
    "gs_selftest_wait_timeout": (_i, [C.c_uint, _vp, _vp, _vp]),
    "gs_verify_round_workspace": (_sz, [_vp]),
    "gs_verify_round_configure": (_i, [_i]),
    "gs_verify_round_reads_in_place": (_i, [_vp]),
    "gs_verify_round_near_rows": (_i, [_vp]),
    "gs_verify_round_host": (_i, [_vp] + [_vp] * 8 + [_vp] * 7 + [_vp, _sz] + [_vp] * 5 + [_vp]),
    "gs_launch_count": (C.c_ulonglong, []),
}


class RoundDesc(C.Structure):
    """Mirror of gs_round_desc."""
    _fields_ = [("N", _i), ("Tq", _i), ("total_kv", _i), ("max_kv_len", _i), ("Hq", _i), ("Hkv", _i),
                ("hd", _i), ("d", _i), ("V", _i), ("C", _i), ("dt", _i), ("scale", _f), ("temperature", _f),
                ("eta", _d), ("beta", _d), ("alpha_min", _d), ("alpha_max", _d)]

_lib = None


class GoodSpeedError(RuntimeError):
    def __init__(self, fn: str, code: int):
        self.code = code
        super().__init__(f"{fn} returned {STATUS_NAMES.get(code, code)}")


def lib() -> C.CDLL:
    """Loads the library (once).  Raises if it was not built: there is no other code path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                               "`python -m paper_2512_09963_b200.build` (needs nvcc)")
        L = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _ptr(t: Optional[torch.Tensor], dtype=None, cuda=True):
    if t is None:
        return None
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"expected {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    if cuda and not t.is_cuda:
        raise ValueError("tensor must be on the CUDA device")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(fn: str, code: int):
    if code != GS_OK:
        raise GoodSpeedError(fn, code)


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return GS_F32
    if t.dtype == torch.bfloat16:
        return GS_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def gs_version() -> int:
    return lib().gs_version()


def gs_status_str(code: int) -> str:
    return lib().gs_status_str(code).decode()


def gs_verify_attn_workspace(N, Tq, total_kv, max_kv_len, Hq, Hkv, hd, dt) -> int:
    return lib().gs_verify_attn_workspace(N, Tq, total_kv, max_kv_len, Hq, Hkv, hd, dt)


def gs_verify_attn_configure(tiles_per_split: int = 0):
    _check("gs_verify_attn_configure", lib().gs_verify_attn_configure(int(tiles_per_split)))


def gs_verify_attn_select(variant: int = 0):
    _check("gs_verify_attn_select", lib().gs_verify_attn_select(int(variant)))


def gs_verify_attn(Q, K, V, O, cu_q, cu_kv, max_kv_len, scale, ws, d_status=None):
    Tq, Hq, hd = Q.shape
    total_kv, Hkv, _ = K.shape
    N = cu_q.numel() - 1
    code = lib().gs_verify_attn(_ptr(Q), _ptr(K, Q.dtype), _ptr(V, Q.dtype), _ptr(O, Q.dtype),
                                _ptr(cu_q, torch.int32), _ptr(cu_kv, torch.int32),
                                N, Tq, total_kv, int(max_kv_len), Hq, Hkv, hd, float(scale), _dt(Q),
                                _ptr(ws), ws.numel() * ws.element_size(), _ptr(d_status, torch.int32),
                                _stream())
    _check("gs_verify_attn", code)


def gs_verify_attn_paged_workspace(N, Tq, max_kv_len, Hq, Hkv, hd, dt) -> int:
    return lib().gs_verify_attn_paged_workspace(N, Tq, max_kv_len, Hq, Hkv, hd, dt)


def gs_verify_attn_paged(Q, K_pool, V_pool, O, cu_q, cu_kv, block_table, max_kv_len, scale, ws, d_status=None):
    """K_pool, V_pool: [n_pages * 128, Hkv, hd]; block_table: [N, max_pages] int32; cu_kv: running sum
    of the cache lengths."""
    Tq, Hq, hd = Q.shape
    rows, Hkv, _ = K_pool.shape
    N, max_pages = block_table.shape
    code = lib().gs_verify_attn_paged(_ptr(Q), _ptr(K_pool, Q.dtype), _ptr(V_pool, Q.dtype), _ptr(O, Q.dtype),
                                      _ptr(cu_q, torch.int32), _ptr(cu_kv, torch.int32),
                                      _ptr(block_table, torch.int32), N, Tq, rows // 128, max_pages,
                                      int(max_kv_len), Hq, Hkv, hd, float(scale), _dt(Q),
                                      _ptr(ws), ws.numel() * ws.element_size(), _ptr(d_status, torch.int32),
                                      _stream())
    _check("gs_verify_attn_paged", code)


def gs_lm_head_workspace(T, d, V, dt) -> int:
    return lib().gs_lm_head_workspace(T, d, V, dt)


def gs_lm_head_configure(m_tiles: int = 0, stages: int = 0, k_rows: int = 0):
    _check("gs_lm_head_configure", lib().gs_lm_head_configure(int(m_tiles), int(stages), int(k_rows)))


def gs_lm_head_select(variant: int = 0):
    _check("gs_lm_head_select", lib().gs_lm_head_select(int(variant)))


def gs_spec_accept_select(variant: int = 0):
    _check("gs_spec_accept_select", lib().gs_spec_accept_select(int(variant)))


def gs_schedule_select(variant: int = 0):
    _check("gs_schedule_select", lib().gs_schedule_select(int(variant)))


def gs_set_dependent_launch(on: bool = True):
    _check("gs_set_dependent_launch", lib().gs_set_dependent_launch(1 if on else 0))


def gs_lm_head_logits(H, W, logits, ws, d_status=None):
    T, d = H.shape
    V = W.shape[1]
    if W.shape[0] != d or tuple(logits.shape) != (T, V):
        raise ValueError("shape mismatch")
    code = lib().gs_lm_head_logits(_ptr(H), _ptr(W, H.dtype), _ptr(logits, torch.float32), T, d, V, _dt(H),
                                   _ptr(ws), ws.numel() * ws.element_size(),
                                   _ptr(d_status, torch.int32), _stream())
    _check("gs_lm_head_logits", code)


GS_ERR_UNSUPPORTED = 3


def gs_lm_head_logits_w4(H, qweight, scales, zeros, group, logits, d_status=None):
    """LM head on a 4-bit weight: qweight [d/8, V] int32 (eight codes per word along d), scales
    [d/group, V] bf16, zeros [d/group, V] uint8 (see the header for the nibble order)."""
    T, d = H.shape
    V = qweight.shape[1]
    if qweight.shape[0] * 8 != d or tuple(logits.shape) != (T, V) or tuple(scales.shape) != (d // group, V) \
            or tuple(zeros.shape) != (d // group, V):
        raise ValueError("shape mismatch")
    code = lib().gs_lm_head_logits_w4(_ptr(H, torch.bfloat16), _ptr(qweight, torch.int32), _ptr(scales, torch.bfloat16),
                                      _ptr(zeros, torch.uint8), int(group), _ptr(logits, torch.float32), T, d, V,
                                      _ptr(d_status, torch.int32), _stream())
    _check("gs_lm_head_logits_w4", code)


def gs_lm_head_stats_bytes(T) -> int:
    return lib().gs_lm_head_stats_bytes(int(T))


def gs_lm_head_stats_pays(T) -> bool:
    """Whether the statistics epilogue is expected to beat the separate statistics pass at T rows."""
    return bool(lib().gs_lm_head_stats_pays(int(T)))


def gs_lm_head_logits_stats(H, W, logits, temperature, stats, ws, d_status=None):
    """LM head that also writes the rows' softmax statistics.  Returns the number of statistics
    entries per row, or None if this shape has no such kernel (nothing was launched then)."""
    T, d = H.shape
    V = W.shape[1]
    if W.shape[0] != d or tuple(logits.shape) != (T, V):
        raise ValueError("shape mismatch")
    n_chunk = C.c_int(0)
    code = lib().gs_lm_head_logits_stats(_ptr(H), _ptr(W, H.dtype), _ptr(logits, torch.float32), T, d, V, _dt(H),
                                         float(temperature), _ptr(stats), stats.numel() * stats.element_size(),
                                         C.byref(n_chunk), _ptr(ws), ws.numel() * ws.element_size(),
                                         _ptr(d_status, torch.int32), _stream())
    if code == GS_ERR_UNSUPPORTED:
        return None
    _check("gs_lm_head_logits_stats", code)
    return int(n_chunk.value)


def gs_spec_accept_prestats(logits, q_probs, draft_tok, cu_q, u_accept, u_sample, temperature,
                            accepted, out_tok, n_out, ratio, p_tok, stats, n_chunk, margin=None,
                            alpha_hat=None, X=None, eta=0.0, beta=0.0, alpha_min=1e-3, alpha_max=0.999,
                            ws=None, d_status=None) -> bool:
    """Acceptance step on statistics from gs_lm_head_logits_stats.  False (nothing launched) if the
    shape needs the plain gs_spec_accept."""
    Tq, V = logits.shape
    N = cu_q.numel() - 1
    f32, i32, f64 = torch.float32, torch.int32, torch.float64
    code = lib().gs_spec_accept_prestats(
        _ptr(logits, f32), _ptr(q_probs, f32), _ptr(draft_tok, i32), _ptr(cu_q, i32),
        _ptr(u_accept, f32), _ptr(u_sample, f32), float(temperature), N, Tq, V,
        _ptr(accepted, i32), _ptr(out_tok, i32), _ptr(n_out, i32), _ptr(ratio, f32), _ptr(p_tok, f32),
        _ptr(margin, f32), _ptr(alpha_hat, f64), _ptr(X, f64), float(eta), float(beta),
        float(alpha_min), float(alpha_max), _ptr(stats), int(n_chunk),
        _ptr(ws), 0 if ws is None else ws.numel() * ws.element_size(), _ptr(d_status, i32), _stream())
    if code == GS_ERR_UNSUPPORTED:
        return False
    _check("gs_spec_accept_prestats", code)
    return True


def gs_spec_accept_workspace(N, Tq, V) -> int:
    return lib().gs_spec_accept_workspace(N, Tq, V)


def gs_spec_accept(logits, q_probs, draft_tok, cu_q, u_accept, u_sample, temperature,
                   accepted, out_tok, n_out, ratio, p_tok, margin=None,
                   alpha_hat=None, X=None, eta=0.0, beta=0.0, alpha_min=1e-3, alpha_max=0.999,
                   ws=None, d_status=None):
    Tq, V = logits.shape
    N = cu_q.numel() - 1
    f32, i32, f64 = torch.float32, torch.int32, torch.float64
    code = lib().gs_spec_accept(_ptr(logits, f32), _ptr(q_probs, f32), _ptr(draft_tok, i32), _ptr(cu_q, i32),
                                _ptr(u_accept, f32), _ptr(u_sample, f32), float(temperature), N, Tq, V,
                                _ptr(accepted, i32), _ptr(out_tok, i32), _ptr(n_out, i32),
                                _ptr(ratio, f32), _ptr(p_tok, f32), _ptr(margin, f32),
                                _ptr(alpha_hat, f64), _ptr(X, f64), float(eta), float(beta),
                                float(alpha_min), float(alpha_max),
                                _ptr(ws), 0 if ws is None else ws.numel() * ws.element_size(),
                                _ptr(d_status, i32), _stream())
    _check("gs_spec_accept", code)


def gs_schedule(X, alpha_hat, C_budget, S_out, s_min=None, s_max=None, d_status=None):
    N = X.numel()
    i32, f64 = torch.int32, torch.float64
    code = lib().gs_schedule(_ptr(X, f64), _ptr(alpha_hat, f64), N, int(C_budget), _ptr(s_min, i32),
                             _ptr(s_max, i32), _ptr(S_out, i32), _ptr(d_status, i32), _stream())
    _check("gs_schedule", code)


def gs_schedule_host(X, alpha_hat, C_budget, S_out, s_min=None, s_max=None):
    """gs_schedule on host arrays (CPU tensors); no CUDA call.  GS_ERR_SHAPE (floors above the
    budget) raises like every other error, after S_out has received the floors."""
    N = X.numel()
    i32, f64 = torch.int32, torch.float64
    hp = lambda t, dt: _ptr(t, dt, cuda=False)
    for t in (X, alpha_hat, S_out, s_min, s_max):
        if t is not None and t.is_cuda:
            raise ValueError("gs_schedule_host takes host tensors")
    code = lib().gs_schedule_host(hp(X, f64), hp(alpha_hat, f64), N, int(C_budget), hp(s_min, i32), hp(s_max, i32),
                                  hp(S_out, i32))
    _check("gs_schedule_host", code)


def gs_selftest_wait_timeout(limit_us, d_status, d_waited_ns=None):
    """One warp waits limit_us microseconds for a barrier nothing completes, then reports
    GS_ERR_TIMEOUT in d_status (see the header)."""
    _check("gs_selftest_wait_timeout",
           lib().gs_selftest_wait_timeout(int(limit_us), _ptr(d_status, torch.int32), _ptr(d_waited_ns, torch.int64),
                                          _stream()))


def gs_launch_count() -> int:
    return int(lib().gs_launch_count())


def gs_verify_round_workspace(desc: RoundDesc) -> int:
    return lib().gs_verify_round_workspace(C.byref(desc))


def gs_verify_round_configure(read_in_place=True):
    """True / 1: in place with the first rows copied meanwhile (default); 2: in place only; False / 0: copy."""
    _check("gs_verify_round_configure", lib().gs_verify_round_configure(int(read_in_place)))


def gs_verify_round_reads_in_place(h_q_probs) -> bool:
    """Whether gs_verify_round_host would read this CPU tensor of draft distributions where it lies."""
    return bool(lib().gs_verify_round_reads_in_place(_ptr(h_q_probs, torch.float32, cuda=False)))


def gs_verify_round_near_rows(desc: RoundDesc) -> int:
    return int(lib().gs_verify_round_near_rows(C.byref(desc)))


def gs_verify_round_host(desc: RoundDesc, h_Q, h_H, h_q_probs, h_draft_tok, h_u_accept, h_u_sample,
                         h_cu_q, h_cu_kv, d_K, d_V, d_W, d_alpha_hat, d_X, d_s_min, d_s_max, d_ws,
                         h_accepted, h_out_tok, h_n_out, h_S_next, h_status):
    """Host tensors (h_*) must be CPU tensors, ideally pinned; d_* are CUDA tensors."""
    i32, f32, f64 = torch.int32, torch.float32, torch.float64
    hp = lambda t, dt=None: _ptr(t, dt, cuda=False)
    for t in (h_Q, h_H, h_q_probs, h_draft_tok, h_u_accept, h_u_sample, h_cu_q, h_cu_kv,
              h_accepted, h_out_tok, h_n_out, h_S_next, h_status):
        if t is not None and t.is_cuda:
            raise ValueError("h_* tensors must live in host memory")
    code = lib().gs_verify_round_host(
        C.byref(desc), hp(h_Q), hp(h_H), hp(h_q_probs, f32), hp(h_draft_tok, i32), hp(h_u_accept, f32),
        hp(h_u_sample, f32), hp(h_cu_q, i32), hp(h_cu_kv, i32),
        _ptr(d_K), _ptr(d_V), _ptr(d_W), _ptr(d_alpha_hat, f64), _ptr(d_X, f64), _ptr(d_s_min, i32),
        _ptr(d_s_max, i32), _ptr(d_ws), d_ws.numel() * d_ws.element_size(),
        hp(h_accepted, i32), hp(h_out_tok, i32), hp(h_n_out, i32), hp(h_S_next, i32), hp(h_status, i32),
        _stream())
    _check("gs_verify_round_host", code)


def gs_spec_accept_static_capacity() -> int:
    return int(lib().gs_spec_accept_static_capacity())


def gs_spec_accept_static(logits, q_probs, draft_tok, cu_q, u_accept, u_sample, temperature,
                          accepted, out_tok, n_out, ratio, p_tok, margin=None,
                          alpha_hat=None, X=None, eta=0.0, beta=0.0, alpha_min=1e-3, alpha_max=0.999,
                          d_status=None):
    """gs_spec_accept without a workspace argument: the scratch is a fixed array inside the library,
    so the call allocates nothing (see the header for the size limit and the sharing rules)."""
    Tq, V = logits.shape
    N = cu_q.numel() - 1
    f32, i32, f64 = torch.float32, torch.int32, torch.float64
    code = lib().gs_spec_accept_static(_ptr(logits, f32), _ptr(q_probs, f32), _ptr(draft_tok, i32),
                                       _ptr(cu_q, i32), _ptr(u_accept, f32), _ptr(u_sample, f32),
                                       float(temperature), N, Tq, V,
                                       _ptr(accepted, i32), _ptr(out_tok, i32), _ptr(n_out, i32),
                                       _ptr(ratio, f32), _ptr(p_tok, f32), _ptr(margin, f32),
                                       _ptr(alpha_hat, f64), _ptr(X, f64), float(eta), float(beta),
                                       float(alpha_min), float(alpha_max), _ptr(d_status, i32), _stream())
    _check("gs_spec_accept_static", code)
