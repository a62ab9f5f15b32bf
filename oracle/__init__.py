"""ctypes driver of the D-Quant CPU oracle (TEST INFRASTRUCTURE, not product code).

Compiles ``dq_oracle.c`` with gcc on first use and exposes its functions on numpy
arrays.  Only the tests, the smoke check and the benchmark's CPU-baseline leg may
import this package; the CUDA library and its Python binding never do.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dq_oracle.c")
_LIB = os.path.join(_HERE, "libdq_oracle.so")
_lock = threading.Lock()
_lib = None

MAX_LEVELS = 16
WINDOW = 128
PAGE = 16


def build(force: bool = False) -> str:
    """Compile the oracle (no fast-math, no FMA contraction) and return the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        cmd = ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


class Table(C.Structure):
    _fields_ = [
        ("M", C.c_int), ("n", C.c_int), ("rec", C.c_int), ("C", C.c_int), ("B", C.c_int),
        ("mstar", C.c_int), ("feasible", C.c_int), ("has_mean", C.c_int), ("rotate", C.c_int),
        ("alpha", C.c_double), ("E", C.c_double),
        ("p", C.c_double * MAX_LEVELS), ("q", C.c_double * MAX_LEVELS),
        ("f", C.c_int32 * MAX_LEVELS), ("c", C.c_int32 * (MAX_LEVELS + 1)),
        ("r", C.c_float * MAX_LEVELS), ("R", C.c_uint32 * MAX_LEVELS),
        ("lut_m", C.c_uint8 * 256), ("lut_f", C.c_uint8 * 256), ("lut_d", C.c_uint8 * 256),
        ("sigma", C.c_int), ("early_exit", C.c_int),
        ("pair", C.c_int), ("ustar", C.c_int),
        ("pf", C.c_int32 * 256), ("pc", C.c_int32 * 257), ("pr", C.c_float * 256), ("pR", C.c_uint32 * 256),
        ("plut_u", C.c_uint8 * 256), ("plut_f", C.c_uint8 * 256), ("plut_d", C.c_uint8 * 256),
    ]

    @property
    def L(self):
        """Lower bound of the state interval: 2^23 (sigma = 32) or 2^15 (sigma = 24)."""
        return 1 << (self.sigma - 9)

    @property
    def state_bytes(self):
        return self.sigma // 8

    def freqs(self):
        return [int(self.f[m]) for m in range(self.M)]

    def pair_freqs(self):
        """Frequencies of the pair alphabet, index u = a * M + b (paired-symbol variant)."""
        return [int(self.pf[u]) for u in range(self.M * self.M)]

    def code_length(self, sym) -> int:
        """Fixed-point code length (1/65536 bit) of a symbol sequence under this table's alphabet."""
        if self.pair:
            return sum(int(self.pR[int(sym[j]) * self.M + int(sym[j + 1])]) for j in range(0, len(sym), 2))
        return sum(int(self.R[int(m)]) for m in sym)

    def cum(self):
        return [int(self.c[m]) for m in range(self.M + 1)]

    def entropy(self):
        f = np.array(self.freqs(), dtype=np.float64) / 256.0
        return float(-(f * np.log2(f)).sum())

    def model_entropy(self):
        p = np.array([self.p[m] for m in range(self.M)])
        return float(-(p * np.log2(p)).sum())


def lib():
    global _lib
    with _lock:
        if _lib is None:
            L = C.CDLL(build())
            assert L.dqo_table_size() == C.sizeof(Table), "oracle struct layout mismatch"
            L.dqo_expected_max.restype = C.c_double
            L.dqo_expected_max.argtypes = [C.c_int]
            L.dqo_f64_to_f16.restype = C.c_uint16
            L.dqo_f64_to_f16.argtypes = [C.c_double]
            L.dqo_f16_to_f32.restype = C.c_float
            L.dqo_f16_to_f32.argtypes = [C.c_uint16]
            L.dqo_drift.restype = C.c_int64
            L.dqo_rans_encode.restype = C.c_int
            L.dqo_build_table.restype = C.c_int
            L.dqo_build_table.argtypes = [C.c_int, C.c_int, C.c_int, C.c_double, C.c_int, C.c_int,
                                          C.POINTER(Table)]
            L.dqo_build_table_ex.restype = C.c_int
            L.dqo_build_table_ex.argtypes = [C.c_int, C.c_int, C.c_int, C.c_double, C.c_int, C.c_int,
                                             C.c_int, C.c_int, C.c_int, C.POINTER(Table)]
            _lib = L
    return _lib


def _p(a, ct=None):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(C.c_void_p)


def num_threads() -> int:
    return int(lib().dqo_num_threads())


def expected_max(n: int) -> float:
    return float(lib().dqo_expected_max(n))


def f64_to_f16_bits(v: float) -> int:
    return int(lib().dqo_f64_to_f16(float(v)))


def f16_bits_to_f32(h: int) -> float:
    return float(lib().dqo_f16_to_f32(int(h)))


def rec_bytes(bits_per_elem: float, n: int) -> int:
    """Record size in bytes for a storage budget given in bits per element."""
    return int(np.floor(bits_per_elem * n / 8.0 + 1e-9))


def build_table(levels: int, n: int, rec: int, alpha: float = 1.4, has_mean: bool = False,
                rotate: bool = True, allow_infeasible: bool = False, sigma: int = 32,
                early_exit: bool = False, pair: bool = False) -> Table:
    """sigma / early_exit / pair select the opt-in codec variants (defaults: the paper's codec)."""
    T = Table()
    if sigma == 32 and not early_exit and not pair:
        rc = lib().dqo_build_table(levels, n, rec, float(alpha), int(has_mean), int(rotate), C.byref(T))
    else:
        rc = lib().dqo_build_table_ex(levels, n, rec, float(alpha), int(has_mean), int(rotate), int(sigma),
                                      int(early_exit), int(pair), C.byref(T))
    if rc == -1 or (rc != 0 and not allow_infeasible):
        raise ValueError(f"oracle table build failed rc={rc} (M={levels}, n={n}, rec={rec})")
    return T


def fwht_f32(x: np.ndarray) -> np.ndarray:
    y = np.ascontiguousarray(x, dtype=np.float32).copy()
    for row in y.reshape(-1, y.shape[-1]):
        lib().dqo_fwht_f32(_p(row), C.c_int(row.shape[0]))
    return y


def fwht_f64(x: np.ndarray) -> np.ndarray:
    y = np.ascontiguousarray(x, dtype=np.float64).copy()
    for row in y.reshape(-1, y.shape[-1]):
        lib().dqo_fwht_f64(_p(row), C.c_int(row.shape[0]))
    return y


def drift(z: np.ndarray, s: float, o: float, T: Table):
    """Function Drift of Algorithm 1.  Returns (symbols uint8[n], length in 1/65536 bit)."""
    z = np.ascontiguousarray(z, dtype=np.float32)
    m = np.zeros(z.shape[0], dtype=np.uint8)
    ln = lib().dqo_drift(_p(z), C.c_int(z.shape[0]), C.c_float(s), C.c_float(o), C.byref(T), _p(m))
    return m, int(ln)


def rans_encode(sym: np.ndarray, T: Table, cap: int):
    """Returns (payload uint8[cap], k) or (None, -1) when 4 + k exceeds cap."""
    sym = np.ascontiguousarray(sym, dtype=np.uint8)
    out = np.zeros(cap, dtype=np.uint8)
    k = lib().dqo_rans_encode(_p(sym), C.c_int(sym.shape[0]), C.byref(T), _p(out), C.c_int(cap))
    return (out, k) if k >= 0 else (None, -1)


def rans_decode(payload: np.ndarray, n: int, T: Table):
    """Returns (symbols uint8[n], final state, final ptr)."""
    payload = np.ascontiguousarray(payload, dtype=np.uint8)
    sym = np.zeros(n, dtype=np.uint8)
    end = np.zeros(2, dtype=np.uint32)
    lib().dqo_rans_decode(_p(payload), C.c_int(payload.shape[0]), C.c_int(n), C.byref(T), _p(sym),
                          _p(end))
    return sym, int(end[0]), int(end[1])


def encode_stream(z: np.ndarray, T: Table):
    """Algorithm 1 on one prepared stream.  Returns (record uint8[rec], symbols, stats[4])."""
    z = np.ascontiguousarray(z, dtype=np.float32)
    assert z.shape[0] == T.n and T.n % 32 == 0
    rec = np.zeros(T.rec, dtype=np.uint8)
    sym = np.zeros(T.n, dtype=np.uint8)
    st = np.zeros(4, dtype=np.uint32)
    lib().dqo_encode_stream(_p(z), C.byref(T), _p(rec), _p(st), _p(sym))
    return rec, sym, st


ROPE_NONE, ROPE_HALF, ROPE_PAIRS = 0, 1, 2


def rope_f32(x: np.ndarray, cs: np.ndarray, sn: np.ndarray, style: int) -> np.ndarray:
    """Rotary embedding of one head vector (binary32); cs / sn: d/2 entries of this position."""
    y = np.ascontiguousarray(x, dtype=np.float32).copy()
    cs = np.ascontiguousarray(cs, dtype=np.float32)
    sn = np.ascontiguousarray(sn, dtype=np.float32)
    lib().dqo_rope_f32(_p(y), C.c_int(y.shape[0]), _p(cs), _p(sn), C.c_int(style))
    return y


def _rope_args(rope, d):
    if rope is None:
        return None, None, 0
    cs, sn, style = rope
    cs = np.ascontiguousarray(cs, dtype=np.float32)
    sn = np.ascontiguousarray(sn, dtype=np.float32)
    assert cs.shape == sn.shape and cs.shape[1] == d // 2 and style in (ROPE_HALF, ROPE_PAIRS)
    return cs, sn, style


def window_means(k_bf16: np.ndarray, seq_id, pos, mean_q: np.ndarray, mean_scale: np.ndarray,
                 mode: int, rotate: bool = True, rope=None):
    """k_bf16: uint16 [T, Hkv, n] (bf16 bits).  mean_q int8 [S, Wmax, Hkv, n] and
    mean_scale f32 [S, Wmax, Hkv] are updated in place."""
    T_tok, Hkv, n = k_bf16.shape
    Wmax = mean_q.shape[1]
    seq_id = np.ascontiguousarray(seq_id, dtype=np.int32)
    pos = np.ascontiguousarray(pos, dtype=np.int32)
    cs, sn, style = _rope_args(rope, n)
    assert style == 0 or int(pos.max(initial=0)) < cs.shape[0]
    lib().dqo_window_means(_p(k_bf16), C.c_int(T_tok), C.c_int(Hkv), C.c_int(n), _p(seq_id), _p(pos),
                           _p(mean_q), _p(mean_scale), C.c_int(Wmax), C.c_int(mode),
                           C.c_int(int(rotate)), _p(cs), _p(sn), C.c_int(style))


def encode_tokens(T: Table, x_bf16: np.ndarray, seq_id, pos, slot, cont: np.ndarray,
                  mean_q=None, mean_scale=None, rope=None):
    """x_bf16: uint16 [T, Hkv, d]; cont: uint8 [pages, Hkv / hs, 16, rec] updated in place, where
    hs = T.n / d heads share one stream (hs = 1: per token-head; hs = Hkv: per token).
    rope = (cos f32 [positions, d/2], sin, style): x holds keys before their rotary embedding.
    Returns stats uint32[4]."""
    T_tok, Hkv, n = x_bf16.shape
    hs = max(1, T.n // n)
    assert T.n == hs * n and Hkv % hs == 0 and (hs == 1 or n == 128)
    assert cont.dtype == np.uint8 and cont.shape[-1] == T.rec and cont.shape[1] == Hkv // hs
    seq_id = np.ascontiguousarray(seq_id, dtype=np.int32)
    pos = np.ascontiguousarray(pos, dtype=np.int32)
    slot = np.ascontiguousarray(slot, dtype=np.int32)
    Wmax = mean_q.shape[1] if mean_q is not None else 0
    st = np.zeros(4, dtype=np.uint32)
    cs, sn, style = _rope_args(rope, n)
    assert style == 0 or int(pos.max(initial=0)) < cs.shape[0]
    lib().dqo_encode_tokens(C.byref(T), _p(x_bf16), C.c_int(T_tok), C.c_int(Hkv), _p(seq_id), _p(pos),
                            _p(slot), _p(cont), _p(mean_q), _p(mean_scale), C.c_int(Wmax), _p(st),
                            _p(cs), _p(sn), C.c_int(style))
    return st


def decode_tokens(T: Table, cont: np.ndarray, seq_id, pos, slot, Hkv: int, mean_q=None,
                  mean_scale=None, want_dequant: bool = True):
    """Returns (symbols uint8 [T, Hkv, d], dequant f32 [T, Hkv, d] in the rotated domain);
    d = min(T.n, 128)."""
    seq_id = np.ascontiguousarray(seq_id, dtype=np.int32)
    pos = np.ascontiguousarray(pos, dtype=np.int32)
    slot = np.ascontiguousarray(slot, dtype=np.int32)
    T_tok = slot.shape[0]
    d = min(T.n, 128)
    assert cont.shape[1] == Hkv // max(1, T.n // d)
    sym = np.zeros((T_tok, Hkv, d), dtype=np.uint8)
    deq = np.zeros((T_tok, Hkv, d), dtype=np.float32) if want_dequant else None
    Wmax = mean_q.shape[1] if mean_q is not None else 0
    lib().dqo_decode_tokens(C.byref(T), _p(cont), _p(mean_q), _p(mean_scale), C.c_int(Wmax),
                            _p(seq_id), _p(pos), _p(slot), C.c_int(T_tok), C.c_int(Hkv), _p(sym),
                            _p(deq))
    return sym, deq


def attention(TK: Table, TV: Table, q_bf16: np.ndarray, k_cont, v_cont, mean_q, mean_scale,
              page_table: np.ndarray, seq_lens, Hkv: int, sm_scale: float, only=None,
              resid_k=None, resid_v=None, resid_lens=None):
    """fp64 decode-step attention over the containers.  q_bf16: uint16 [B, Hq, n].
    only=(b, hq) computes a single output row (others stay NaN).  Returns f64 [B, Hq, n].
    resid_k / resid_v: uint16 [B, cap, Hkv, n] bf16 bits of the uncompressed residual window,
    resid_lens[b] of whose tokens follow the compressed ones of sequence b."""
    B, Hq, n = q_bf16.shape
    page_table = np.ascontiguousarray(page_table, dtype=np.int32)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    out = np.full((B, Hq, n), np.nan, dtype=np.float64)
    Wmax = mean_q.shape[1] if mean_q is not None else 0
    ob, oh = (-1, -1) if only is None else only
    cap = 0
    if resid_k is not None:
        resid_lens = np.ascontiguousarray(resid_lens, dtype=np.int32)
        cap = int(resid_k.shape[1])
    lib().dqo_attention(C.byref(TK), C.byref(TV), _p(q_bf16), _p(k_cont), _p(v_cont), _p(mean_q),
                        _p(mean_scale), C.c_int(Wmax), _p(page_table), C.c_int(page_table.shape[1]),
                        _p(seq_lens), C.c_int(B), C.c_int(Hq), C.c_int(Hkv), C.c_double(sm_scale),
                        _p(out), C.c_int(ob), C.c_int(oh), _p(resid_k), _p(resid_v), _p(resid_lens),
                        C.c_int(cap))
    return out
