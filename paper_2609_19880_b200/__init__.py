"""Thin Python binding of the D-Quant B200 library (``libdquant.so``, C ABI in include/dq.h).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.
PyTorch supplies device memory and the current stream.  There is no CPU fallback: if the
shared library is missing or fails to load, every call raises.
"""
from __future__ import annotations

import ctypes as C
import os

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libdquant.so")

MAX_LEVELS = 16
MAX_PAIRS = 81
HEAD_DIM = 128
PAGE_TOKENS = 16
WINDOW_TOKENS = 128
MEAN_COMPUTE = 0
MEAN_REUSE = 1

ERRORS = {0: "DQ_OK", -1: "DQ_ERR_ARG", -2: "DQ_ERR_INFEASIBLE", -3: "DQ_ERR_UNSUPPORTED",
          -4: "DQ_ERR_WORKSPACE", -5: "DQ_ERR_CUDA"}

EXPORTS = ["dq_build_tables", "dq_free_tables", "dq_tables_info", "dq_encode_tokens", "dq_encode_tokens_rope",
           "dq_decode_workspace_bytes", "dq_decode_attention", "dq_decode_attention_residual",
           "dq_decode_attention_multi", "dq_window_append", "dq_decode_step",
           "dq_decode_attention_static", "dq_decode_tokens",
           "dq_bf16_decode_attention", "dq_microbench_decode_loop", "dq_set_option", "dq_get_option", "dq_profile_enable", "dq_profile_read",
           "dq_strerror", "dq_last_cuda_error"]


class DqError(RuntimeError):
    def __init__(self, code, what):
        self.code = code
        super().__init__(f"{what}: {ERRORS.get(code, code)}")


class TableOpts(C.Structure):
    _fields_ = [("head_dim", C.c_int), ("alpha", C.c_double), ("has_mean", C.c_int), ("rotate", C.c_int),
                ("heads_per_stream", C.c_int), ("drift_early_exit", C.c_int), ("sigma_bits", C.c_int),
                ("pair_symbols", C.c_int)]


class TableInfo(C.Structure):
    _fields_ = [("levels", C.c_int), ("head_dim", C.c_int), ("rec_bytes", C.c_int),
                ("container_bytes", C.c_int), ("budget_bits", C.c_int), ("mstar", C.c_int),
                ("has_mean", C.c_int), ("rotate", C.c_int), ("alpha", C.c_double),
                ("f", C.c_int32 * MAX_LEVELS), ("c", C.c_int32 * (MAX_LEVELS + 1)),
                ("r", C.c_float * MAX_LEVELS), ("R", C.c_uint32 * MAX_LEVELS), ("lut", C.c_uint32 * 256),
                ("heads_per_stream", C.c_int), ("rec_words", C.c_int), ("sigma_bits", C.c_int),
                ("drift_early_exit", C.c_int), ("pair_symbols", C.c_int), ("ustar", C.c_int),
                ("pair_f", C.c_int32 * MAX_PAIRS), ("pair_R", C.c_uint32 * MAX_PAIRS)]


_lib = None


def lib():
    """Load libdquant.so (built by ``_build.build()``); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2609_19880_b200._build` "
                              "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        vp, i32, f32, f64, sz = C.c_void_p, C.c_int, C.c_float, C.c_double, C.c_size_t
        L.dq_build_tables.restype = i32
        L.dq_build_tables.argtypes = [i32, f64, C.POINTER(TableOpts), C.POINTER(vp)]
        L.dq_free_tables.restype = None
        L.dq_free_tables.argtypes = [vp]
        L.dq_tables_info.restype = i32
        L.dq_tables_info.argtypes = [vp, C.POINTER(TableInfo)]
        L.dq_encode_tokens.restype = i32
        L.dq_encode_tokens.argtypes = [vp, vp, vp, vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, i32, i32, vp, vp]
        L.dq_encode_tokens_rope.restype = i32
        L.dq_encode_tokens_rope.argtypes = [vp, vp, vp, vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, i32, i32, vp, vp, i32,
                                            vp, vp]
        L.dq_decode_workspace_bytes.restype = sz
        L.dq_decode_workspace_bytes.argtypes = [i32, i32, i32]
        L.dq_decode_attention.restype = i32
        L.dq_decode_attention.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, vp, i32, vp, i32, i32, i32, f32,
                                          vp, vp, vp, sz, vp]
        L.dq_decode_attention_residual.restype = i32
        L.dq_decode_attention_residual.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, vp, i32, vp, vp, vp, vp, i32,
                                                   i32, i32, i32, f32, vp, vp, vp, sz, vp]
        L.dq_decode_attention_multi.restype = i32
        L.dq_decode_attention_multi.argtypes = [vp, vp, vp, i32, vp, vp, vp, vp, i32, vp, i32, vp, vp, vp, vp, i32,
                                                i32, i32, i32, f32, vp, vp, vp, sz, vp]
        L.dq_decode_step.restype = i32
        L.dq_decode_step.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, i32, vp, i32, i32, i32, f32, vp, vp,
                                     vp, sz, vp, vp]
        L.dq_window_append.restype = i32
        L.dq_window_append.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, vp]
        L.dq_decode_attention_static.restype = i32
        L.dq_decode_attention_static.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, vp, i32, vp, i32, i32, i32, f32,
                                                 vp, vp, vp]
        L.dq_decode_tokens.restype = i32
        L.dq_decode_tokens.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp, i32, i32, vp, vp, vp]
        L.dq_bf16_decode_attention.restype = i32
        L.dq_bf16_decode_attention.argtypes = [vp, vp, vp, vp, i32, vp, i32, i32, i32, f32, vp, vp, sz, vp]
        L.dq_microbench_decode_loop.restype = i32
        L.dq_microbench_decode_loop.argtypes = [vp, vp, sz, i32, i32, i32, i32, vp, vp]
        L.dq_set_option.restype = i32
        L.dq_set_option.argtypes = [i32, C.c_longlong]
        L.dq_get_option.restype = C.c_longlong
        L.dq_get_option.argtypes = [i32]
        L.dq_profile_enable.restype = None
        L.dq_profile_enable.argtypes = [i32]
        L.dq_profile_read.restype = i32
        L.dq_profile_read.argtypes = [C.POINTER(C.c_float), i32]
        L.dq_strerror.restype = C.c_char_p
        L.dq_strerror.argtypes = [i32]
        L.dq_last_cuda_error.restype = C.c_char_p
        L.dq_last_cuda_error.argtypes = []
        _lib = L
    return _lib


def _check(rc, what):
    if rc != 0:
        msg = what
        if rc == -5:
            msg += " [" + lib().dq_last_cuda_error().decode() + "]"
        raise DqError(rc, msg)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


class Tables:
    """Owner of one ``dq_tables*`` (host memory inside the library)."""

    def __init__(self, handle):
        self._h = C.c_void_p(handle)

    @property
    def handle(self):
        return self._h

    def info(self) -> TableInfo:
        out = TableInfo()
        _check(lib().dq_tables_info(self._h, C.byref(out)), "dq_tables_info")
        return out

    def __del__(self):
        try:
            if self._h and _lib is not None:
                _lib.dq_free_tables(self._h)
                self._h = None
        except Exception:
            pass


def dq_build_tables(levels: int, bits_per_elem: float, *, alpha: float = 1.4, has_mean: bool = False,
                    rotate: bool = True, head_dim: int = HEAD_DIM, heads_per_stream: int = 1,
                    drift_early_exit: bool = False, sigma_bits: int = 32, pair_symbols: bool = False) -> Tables:
    """``heads_per_stream`` = hs > 1 builds tables for streams that span hs KV heads of a token
    (hs = Hkv: the paper's token-wide default); bits_per_elem then refers to hs * 128 values.
    ``drift_early_exit`` / ``sigma_bits`` / ``pair_symbols`` select the opt-in codec variants."""
    opts = TableOpts(head_dim, float(alpha), int(has_mean), int(rotate), int(heads_per_stream),
                     int(drift_early_exit), int(sigma_bits), int(pair_symbols))
    h = C.c_void_p()
    _check(lib().dq_build_tables(int(levels), float(bits_per_elem), C.byref(opts), C.byref(h)), "dq_build_tables")
    return Tables(h.value)


def dq_tables_info(t: Tables) -> TableInfo:
    return t.info()


ROPE_HALF, ROPE_PAIRS = 1, 2


def dq_encode_tokens(tk, tv, k_bf16, v_bf16, seq_id, pos, slot, k_cont, v_cont, k_mean_q=None,
                     k_mean_scale=None, mean_mode: int = MEAN_COMPUTE, status=None, stream=None, rope=None):
    """K/V bf16 [T, Hkv, 128] -> containers (+ window means).  All tensors on the device.
    rope = (cos f32 [positions, 64], sin, style): keys are given before their rotary embedding."""
    ref = k_bf16 if k_bf16 is not None else v_bf16
    T, Hkv = int(ref.shape[0]), int(ref.shape[1])
    max_windows = int(k_mean_q.shape[1]) if k_mean_q is not None else 0
    common = (tk.handle if tk else None, tv.handle if tv else None, _ptr(k_bf16), _ptr(v_bf16),
              T, Hkv, _ptr(seq_id), _ptr(pos), _ptr(slot), _ptr(k_cont), _ptr(v_cont),
              _ptr(k_mean_q), _ptr(k_mean_scale), max_windows, int(mean_mode))
    if rope is None:
        rc = lib().dq_encode_tokens(*common, _ptr(status), _stream(stream))
    else:
        cs, sn, style = rope
        rc = lib().dq_encode_tokens_rope(*common, _ptr(cs), _ptr(sn), int(style), _ptr(status), _stream(stream))
    _check(rc, "dq_encode_tokens")


def dq_decode_workspace_bytes(B: int, Hq: int, max_pages: int) -> int:
    return int(lib().dq_decode_workspace_bytes(int(B), int(Hq), int(max_pages)))


def dq_decode_attention(tk, tv, q_bf16, k_cont, v_cont, k_mean_q, k_mean_scale, page_table, seq_lens,
                        Hkv: int, sm_scale: float, out_bf16, workspace, out_f32=None, stream=None):
    """q bf16 [B, Hq, 128], containers, seq_lens -> out bf16 [B, Hq, 128]."""
    B, Hq = int(q_bf16.shape[0]), int(q_bf16.shape[1])
    max_windows = int(k_mean_q.shape[1]) if k_mean_q is not None else 0
    rc = lib().dq_decode_attention(tk.handle, tv.handle, _ptr(q_bf16), _ptr(k_cont), _ptr(v_cont), _ptr(k_mean_q),
                                   _ptr(k_mean_scale), max_windows, _ptr(page_table), int(page_table.shape[1]),
                                   _ptr(seq_lens), B, Hq, int(Hkv), float(sm_scale), _ptr(out_bf16),
                                   _ptr(out_f32), _ptr(workspace), int(workspace.numel() * workspace.element_size()),
                                   _stream(stream))
    _check(rc, "dq_decode_attention")


def dq_decode_attention_residual(tk, tv, q_bf16, k_cont, v_cont, k_mean_q, k_mean_scale, page_table, seq_lens,
                                 resid_k, resid_v, resid_lens, Hkv: int, sm_scale: float, out_bf16, workspace,
                                 out_f32=None, stream=None):
    """Decode attention over the compressed cache plus a BF16 residual window:
    resid_k / resid_v bf16 [B, cap, Hkv, 128], resid_lens int32 [B]."""
    B, Hq = int(q_bf16.shape[0]), int(q_bf16.shape[1])
    max_windows = int(k_mean_q.shape[1]) if k_mean_q is not None else 0
    rc = lib().dq_decode_attention_residual(
        tk.handle, tv.handle, _ptr(q_bf16), _ptr(k_cont), _ptr(v_cont), _ptr(k_mean_q), _ptr(k_mean_scale),
        max_windows, _ptr(page_table), int(page_table.shape[1]), _ptr(seq_lens), _ptr(resid_k), _ptr(resid_v),
        _ptr(resid_lens), int(resid_k.shape[1]), B, Hq, int(Hkv), float(sm_scale), _ptr(out_bf16), _ptr(out_f32),
        _ptr(workspace), int(workspace.numel() * workspace.element_size()), _stream(stream))
    _check(rc, "dq_decode_attention_residual")


def dq_decode_attention_multi(tk, tv, q_bf16, k_cont, v_cont, k_mean_q, k_mean_scale, page_table, seq_lens,
                              Hkv: int, sm_scale: float, out_bf16, workspace, out_f32=None, resid_k=None,
                              resid_v=None, resid_lens=None, stream=None):
    """q bf16 [B, q_len, Hq, 128] -> out bf16 [B, q_len, Hq, 128]: q_len query tokens per sequence share
    one pass over the cache; seq_lens (+ resid_lens) include the q_len newest tokens."""
    B, q_len, Hq = int(q_bf16.shape[0]), int(q_bf16.shape[1]), int(q_bf16.shape[2])
    max_windows = int(k_mean_q.shape[1]) if k_mean_q is not None else 0
    rc = lib().dq_decode_attention_multi(
        tk.handle, tv.handle, _ptr(q_bf16), q_len, _ptr(k_cont), _ptr(v_cont), _ptr(k_mean_q), _ptr(k_mean_scale),
        max_windows, _ptr(page_table), int(page_table.shape[1]), _ptr(seq_lens), _ptr(resid_k), _ptr(resid_v),
        _ptr(resid_lens), int(resid_k.shape[1]) if resid_k is not None else 0, B, Hq, int(Hkv), float(sm_scale),
        _ptr(out_bf16), _ptr(out_f32), _ptr(workspace), int(workspace.numel() * workspace.element_size()),
        _stream(stream))
    _check(rc, "dq_decode_attention_multi")


def dq_decode_step(tk, tv, k_new, v_new, slot_new, q_bf16, k_cont, v_cont, k_mean_q, k_mean_scale, page_table,
                   seq_lens, Hkv: int, sm_scale: float, out_bf16, workspace, out_f32=None, status=None, stream=None):
    """Encode the newest token of every sequence (k_new / v_new bf16 [B, Hkv, 128] at slot_new, position
    seq_lens - 1) and attend over the whole cache, as one overlapped launch sequence."""
    B, Hq = int(q_bf16.shape[0]), int(q_bf16.shape[1])
    max_windows = int(k_mean_q.shape[1]) if k_mean_q is not None else 0
    rc = lib().dq_decode_step(tk.handle, tv.handle, _ptr(k_new), _ptr(v_new), _ptr(slot_new), _ptr(q_bf16),
                              _ptr(k_cont), _ptr(v_cont), _ptr(k_mean_q), _ptr(k_mean_scale), max_windows,
                              _ptr(page_table), int(page_table.shape[1]), _ptr(seq_lens), B, Hq, int(Hkv),
                              float(sm_scale), _ptr(out_bf16), _ptr(out_f32), _ptr(workspace),
                              int(workspace.numel() * workspace.element_size()), _ptr(status), _stream(stream))
    _check(rc, "dq_decode_step")


def dq_window_append(k_bf16, v_bf16, resid_k, resid_v, resid_lens, stream=None):
    """New tokens bf16 [B, Hkv, 128] -> BF16 window [B, cap, Hkv, 128] at position resid_lens[b]; resid_lens += 1."""
    B, Hkv = int(k_bf16.shape[0]), int(k_bf16.shape[1])
    _check(lib().dq_window_append(_ptr(k_bf16), _ptr(v_bf16), _ptr(resid_k), _ptr(resid_v), _ptr(resid_lens),
                                  int(resid_k.shape[1]), B, Hkv, _stream(stream)), "dq_window_append")


STATIC_SCRATCH_BYTES = 4 << 20


def dq_decode_attention_static(tk, tv, q_bf16, k_cont, v_cont, k_mean_q, k_mean_scale, page_table, seq_lens,
                               Hkv: int, sm_scale: float, out_bf16, out_f32=None, stream=None):
    """dq_decode_attention for callers that cannot allocate a workspace: the library's built-in
    scratch array (STATIC_SCRATCH_BYTES, shared by all calls) is used instead.  Raises
    DqError(DQ_ERR_WORKSPACE) when the call would need more than that.  Calls must not overlap
    on the GPU; make the first call on a device outside any stream capture."""
    B, Hq = int(q_bf16.shape[0]), int(q_bf16.shape[1])
    max_windows = int(k_mean_q.shape[1]) if k_mean_q is not None else 0
    rc = lib().dq_decode_attention_static(tk.handle, tv.handle, _ptr(q_bf16), _ptr(k_cont), _ptr(v_cont),
                                          _ptr(k_mean_q), _ptr(k_mean_scale), max_windows, _ptr(page_table),
                                          int(page_table.shape[1]), _ptr(seq_lens), B, Hq, int(Hkv),
                                          float(sm_scale), _ptr(out_bf16), _ptr(out_f32), _stream(stream))
    if rc == -4:
        raise DqError(rc, "dq_decode_attention_static [" + lib().dq_last_cuda_error().decode() + "]")
    _check(rc, "dq_decode_attention_static")


def dq_decode_tokens(t, cont, slot, Hkv: int, symbols=None, dequant=None, mean_q=None, mean_scale=None,
                     seq_id=None, pos=None, stream=None):
    max_windows = int(mean_q.shape[1]) if mean_q is not None else 0
    rc = lib().dq_decode_tokens(t.handle, _ptr(cont), _ptr(mean_q), _ptr(mean_scale), max_windows, _ptr(seq_id),
                                _ptr(pos), _ptr(slot), int(slot.shape[0]), int(Hkv), _ptr(symbols), _ptr(dequant),
                                _stream(stream))
    _check(rc, "dq_decode_tokens")


def dq_bf16_decode_attention(q_bf16, k_pages, v_pages, page_table, seq_lens, Hkv: int, sm_scale: float,
                             out_bf16, workspace, stream=None):
    B, Hq = int(q_bf16.shape[0]), int(q_bf16.shape[1])
    rc = lib().dq_bf16_decode_attention(_ptr(q_bf16), _ptr(k_pages), _ptr(v_pages), _ptr(page_table),
                                        int(page_table.shape[1]), _ptr(seq_lens), B, Hq, int(Hkv), float(sm_scale),
                                        _ptr(out_bf16), _ptr(workspace),
                                        int(workspace.numel() * workspace.element_size()), _stream(stream))
    _check(rc, "dq_bf16_decode_attention")


def dq_microbench_decode_loop(table, bytes_u8, ctas: int, threads: int, chains: int, reps: int, out_u32, stream=None):
    """Bare rANS decode loop (measurement aid); time it with CUDA events on the stream."""
    rc = lib().dq_microbench_decode_loop(table.handle, _ptr(bytes_u8), int(bytes_u8.numel()), int(ctas), int(threads),
                                         int(chains), int(reps), _ptr(out_u32), _stream(stream))
    _check(rc, "dq_microbench_decode_loop")


OPT_STEP_POLL_LIMIT = 1
OPT_ENCODE_BATCH_MIN = 2


def dq_set_option(key: int, value: int):
    """Process-wide tuning option (OPT_*); a negative value restores the library default."""
    _check(lib().dq_set_option(int(key), int(value)), "dq_set_option")


def dq_get_option(key: int) -> int:
    return int(lib().dq_get_option(int(key)))


def dq_profile_enable(on):
    """0 / False: off; k > 0: time the fused kernel of every k-th dq_decode_attention call."""
    lib().dq_profile_enable(int(on))


def dq_profile_read(max_records: int = 4096):
    """Durations (ms) of the fused attention kernel for the calls made since enabling."""
    buf = (C.c_float * max_records)()
    n = lib().dq_profile_read(buf, max_records)
    return [float(buf[i]) for i in range(n)]
