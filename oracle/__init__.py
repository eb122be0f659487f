"""Python face of the float64 CPU oracle (``sgbv_oracle.c``).

TEST INFRASTRUCTURE ONLY: the test-suite, the smoke check and the CPU-baseline leg of the
benchmark are the only callers.  The product path never imports this package, and this package
imports nothing from the product.

All arrays are numpy arrays on the host.  Logits are float32 (bf16 inputs are widened exactly by
the caller before they get here); every computation inside is float64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sgbv_oracle.c")
_LIB = os.path.join(_HERE, "libsgbv_oracle.so")

STATUS_TOKEN_RANGE = 1
STATUS_NONFINITE = 2
STATUS_DEGENERATE_RESIDUAL = 4


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over batch rows). Returns the library path."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        cmd = ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c99", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        fp = ctypes.POINTER(ctypes.c_float)
        ip = ctypes.POINTER(ctypes.c_int32)
        lib.sgbv_oracle_softmax.restype = ctypes.c_double
        lib.sgbv_oracle_softmax.argtypes = [fp, ctypes.c_int, ctypes.c_double, dp]
        lib.sgbv_oracle_g.restype = ctypes.c_double
        lib.sgbv_oracle_g.argtypes = [ctypes.c_double, ctypes.c_int]
        lib.sgbv_oracle_resmass.restype = ctypes.c_double
        lib.sgbv_oracle_resmass.argtypes = [dp, dp, ctypes.c_int, ctypes.c_double, ctypes.c_double,
                                            ctypes.c_int, dp]
        lib.sgbv_oracle_h_sub.restype = ctypes.c_double
        lib.sgbv_oracle_h_sub.argtypes = [ctypes.c_double, ctypes.c_double, ctypes.c_double,
                                          ctypes.c_int]
        lib.sgbv_oracle_h_full.restype = ctypes.c_double
        lib.sgbv_oracle_h_full.argtypes = [ctypes.c_double, ctypes.c_double, ctypes.c_int]
        lib.sgbv_oracle_scan.restype = None
        lib.sgbv_oracle_scan.argtypes = [dp, ip, fp, ctypes.c_int, ctypes.c_int, ip, ip]
        lib.sgbv_oracle_sample.restype = ctypes.c_int32
        lib.sgbv_oracle_sample.argtypes = [dp, ctypes.c_int, ctypes.c_double, dp]
        lib.sgbv_oracle_verify.restype = ctypes.c_int
        lib.sgbv_oracle_verify.argtypes = [fp, fp, ip, fp, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                           ctypes.c_int, ctypes.c_double, ip, ip, ip, dp, dp, dp,
                                           dp, ip, dp, dp, ctypes.c_int]
        lib.sgbv_oracle_modify.restype = ctypes.c_int
        lib.sgbv_oracle_modify.argtypes = [fp, fp, dp, dp, fp, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                           ctypes.c_double, ip, dp, dp, dp, dp, ip, dp]
        lib.sgbv_oracle_draw_tokens.restype = ctypes.c_int
        lib.sgbv_oracle_draw_tokens.argtypes = [fp, fp, ctypes.c_int, ctypes.c_int, ctypes.c_double, ip, dp, dp]
        lib.sgbv_oracle_kseq_rho.restype = ctypes.c_double
        lib.sgbv_oracle_kseq_rho.argtypes = [dp, dp, ctypes.c_int, ctypes.c_int]
        lib.sgbv_oracle_kseq_verify.restype = ctypes.c_int
        lib.sgbv_oracle_kseq_verify.argtypes = [fp, fp, ip, fp, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                                ctypes.c_int, ctypes.c_double, ip, ip, dp, dp, ip, dp, dp]
        _lib = lib
    return _lib


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def softmax(z, T: float = 1.0):
    """softmax(z/T) of one row in float64; returns (prob[V], log-normaliser)."""
    z = _f32(z)
    prob = np.empty(z.shape[0], dtype=np.float64)
    lse = _load().sgbv_oracle_softmax(_p(z, ctypes.c_float), z.shape[0], float(T),
                                      _p(prob, ctypes.c_double))
    return prob, lse


def g(u: float, K: int) -> float:
    """1 - (1-u)^K."""
    return _load().sgbv_oracle_g(float(u), int(K))


def resmass(q, p, a: float, b: float, K: int):
    """Residual mass S and its V summands for joint prefix probabilities (a, b)."""
    q, p = _f64(q), _f64(p)
    w = np.empty(q.shape[0], dtype=np.float64)
    S = _load().sgbv_oracle_resmass(_p(q, ctypes.c_double), _p(p, ctypes.c_double), q.shape[0],
                                    float(a), float(b), int(K), _p(w, ctypes.c_double))
    return S, w


def h_sub(a: float, b: float, S: float, K: int) -> float:
    """Eq. 2 acceptance weight of a proper sub-block."""
    return _load().sgbv_oracle_h_sub(float(a), float(b), float(S), int(K))


def h_full(a: float, b: float, K: int) -> float:
    """Eq. 3 acceptance weight of the whole block."""
    return _load().sgbv_oracle_h_full(float(a), float(b), int(K))


def scan(h, tok, eta):
    """Algorithm 1's scan for one batch row. h, eta: [K, gamma]; tok: [K, gamma]. -> (tau, f)."""
    h, tok, eta = _f64(h), _i32(tok), _f32(eta)
    K, gamma = h.shape
    tau = ctypes.c_int32(0)
    f = ctypes.c_int32(0)
    _load().sgbv_oracle_scan(_p(h, ctypes.c_double), _p(tok, ctypes.c_int32),
                             _p(eta, ctypes.c_float), K, gamma, ctypes.byref(tau),
                             ctypes.byref(f))
    return tau.value, f.value


def sample(w, u: float):
    """Inverse-CDF draw from un-normalised masses w. -> (index or -1, margin)."""
    w = _f64(w)
    margin = ctypes.c_double(0.0)
    y = _load().sgbv_oracle_sample(_p(w, ctypes.c_double), w.shape[0], float(u),
                                   ctypes.byref(margin))
    return int(y), margin.value


@dataclass
class VerifyResult:
    tau: np.ndarray            # [B] int32 accepted length
    f: np.ndarray              # [B] int32 accepted draft, -1 when tau == 0
    tokens: np.ndarray         # [B, gamma+1] int32
    h: np.ndarray              # [B, K, gamma] float64 acceptance weights (index i-1)
    S: np.ndarray              # [B, K, gamma] float64 residual masses S_i, i = 0..gamma-1
    loga: np.ndarray           # [B, K, gamma+1] float64 log q(x_k^i)
    logb: np.ndarray           # [B, K, gamma+1] float64 log p(x_k^i)
    status: np.ndarray         # [B] int32 flags
    margin_accept: np.ndarray  # [B] min |eta - h| over the K*gamma trials of the row
    margin_sample: np.ndarray  # [B] distance of u_s to the nearer CDF edge of the drawn cell
    threads: int


def verify(zq, zp, tok, uniforms, temperature: float = 1.0, nthreads: int = 0) -> VerifyResult:
    """One verify step over the batch. zq [B,K,gamma+1,V], zp [B,K,gamma,V], tok [B,K,gamma],
    uniforms [B,K*gamma+1]."""
    zq, zp, tok, uniforms = _f32(zq), _f32(zp), _i32(tok), _f32(uniforms)
    B, K, g1, V = zq.shape
    gamma = g1 - 1
    assert zp.shape == (B, K, gamma, V), zp.shape
    assert tok.shape == (B, K, gamma), tok.shape
    assert uniforms.shape == (B, K * gamma + 1), uniforms.shape
    tau = np.empty(B, np.int32)
    f = np.empty(B, np.int32)
    tokens = np.empty((B, gamma + 1), np.int32)
    h = np.empty((B, K, gamma), np.float64)
    S = np.empty((B, K, gamma), np.float64)
    la = np.empty((B, K, gamma + 1), np.float64)
    lb = np.empty((B, K, gamma + 1), np.float64)
    status = np.empty(B, np.int32)
    ma = np.empty(B, np.float64)
    ms = np.empty(B, np.float64)
    used = _load().sgbv_oracle_verify(
        _p(zq, ctypes.c_float), _p(zp, ctypes.c_float), _p(tok, ctypes.c_int32),
        _p(uniforms, ctypes.c_float), B, K, gamma, V, float(temperature),
        _p(tau, ctypes.c_int32), _p(f, ctypes.c_int32), _p(tokens, ctypes.c_int32),
        _p(h, ctypes.c_double), _p(S, ctypes.c_double), _p(la, ctypes.c_double),
        _p(lb, ctypes.c_double), _p(status, ctypes.c_int32), _p(ma, ctypes.c_double),
        _p(ms, ctypes.c_double), int(nthreads))
    if used < 0:
        raise ValueError("oracle: bad argument")
    return VerifyResult(tau, f, tokens, h, S, la, lb, status, ma, ms, used)


@dataclass
class ModifyResult:
    token: np.ndarray     # [B] int32 token drawn from q_new
    loga: np.ndarray      # [B] carried log q(s, token)
    logb: np.ndarray      # [B] carried log p(s, token)
    R: np.ndarray         # [B] normaliser over a: sum_x q(x|s)(1 - min{(b/a) p(x|s)/q(x|s), 1})^K
    qnew: np.ndarray      # [B, V] the modified distribution (None unless asked for)
    status: np.ndarray    # [B] int32 flags
    margin: np.ndarray    # [B] distance of u to the nearer CDF edge of the drawn cell


def modify(zq, zp, loga, logb, u, K: int, temperature: float = 1.0, want_qnew: bool = False) -> ModifyResult:
    """One position of Algorithm 2 for every batch row. zq, zp [B,V]; loga, logb, u [B]."""
    zq, zp, u = _f32(zq), _f32(zp), _f32(u)
    loga, logb = _f64(loga), _f64(logb)
    B, V = zq.shape
    assert zp.shape == (B, V) and loga.shape == (B,) and logb.shape == (B,) and u.shape == (B,)
    tok = np.empty(B, np.int32)
    la, lb, R, mg = (np.empty(B, np.float64) for _ in range(4))
    st = np.empty(B, np.int32)
    qn = np.empty((B, V), np.float64) if want_qnew else None
    rc = _load().sgbv_oracle_modify(_p(zq, ctypes.c_float), _p(zp, ctypes.c_float), _p(loga, ctypes.c_double),
                                    _p(logb, ctypes.c_double), _p(u, ctypes.c_float), B, V, int(K),
                                    float(temperature), _p(tok, ctypes.c_int32), _p(la, ctypes.c_double),
                                    _p(lb, ctypes.c_double), _p(R, ctypes.c_double),
                                    _p(qn, ctypes.c_double) if want_qnew else None, _p(st, ctypes.c_int32),
                                    _p(mg, ctypes.c_double))
    if rc < 0:
        raise ValueError("oracle: bad argument")
    return ModifyResult(tok, la, lb, R, qn, st, mg)


def kseq_rho(q, p, n: int) -> float:
    """K-SEQ's rho for n candidate drafts: the root of 1 - (1 - beta(rho))^n = rho beta(rho) in [1, n]."""
    q, p = _f64(q), _f64(p)
    return _load().sgbv_oracle_kseq_rho(_p(q, ctypes.c_double), _p(p, ctypes.c_double), q.shape[0], int(n))


@dataclass
class KseqResult:
    tau: np.ndarray            # [B] accepted length
    tokens: np.ndarray         # [B, gamma+1]
    rho: np.ndarray            # [B, gamma] rho of every position reached (NaN elsewhere)
    acc: np.ndarray            # [B, K, gamma] acceptance probability of every token tried (NaN elsewhere)
    status: np.ndarray         # [B]
    margin_accept: np.ndarray  # [B]
    margin_sample: np.ndarray  # [B]


def kseq_verify(zq, zp, tok, uniforms, temperature: float = 1.0) -> KseqResult:
    """Position-wise K-SEQ verification (token-level speculative sampling at K = 1)."""
    zq, zp, tok, uniforms = _f32(zq), _f32(zp), _i32(tok), _f32(uniforms)
    B, K, g1, V = zq.shape
    gamma = g1 - 1
    assert zp.shape == (B, K, gamma, V) and tok.shape == (B, K, gamma) and uniforms.shape == (B, K * gamma + 1)
    tau = np.empty(B, np.int32)
    tokens = np.empty((B, gamma + 1), np.int32)
    rho = np.empty((B, gamma), np.float64)
    acc = np.empty((B, K, gamma), np.float64)
    st = np.empty(B, np.int32)
    ma, ms = np.empty(B, np.float64), np.empty(B, np.float64)
    rc = _load().sgbv_oracle_kseq_verify(_p(zq, ctypes.c_float), _p(zp, ctypes.c_float), _p(tok, ctypes.c_int32),
                                         _p(uniforms, ctypes.c_float), B, K, gamma, V, float(temperature),
                                         _p(tau, ctypes.c_int32), _p(tokens, ctypes.c_int32),
                                         _p(rho, ctypes.c_double), _p(acc, ctypes.c_double),
                                         _p(st, ctypes.c_int32), _p(ma, ctypes.c_double), _p(ms, ctypes.c_double))
    if rc < 0:
        raise ValueError("oracle: bad argument")
    return KseqResult(tau, tokens, rho, acc, st, ma, ms)


def draw_tokens(z, u, temperature: float = 1.0):
    """Algorithm 3's draft draw for one position: token r ~ softmax(z[r]/T) by inverse CDF.
    z [N,V], u [N] -> (tokens int32 [N], log-probabilities [N], margins [N])"""
    z, u = _f32(z), _f32(u)
    N, V = z.shape
    tok = np.empty(N, np.int32)
    lp, mg = np.empty(N, np.float64), np.empty(N, np.float64)
    rc = _load().sgbv_oracle_draw_tokens(_p(z, ctypes.c_float), _p(u, ctypes.c_float), N, V, float(temperature),
                                         _p(tok, ctypes.c_int32), _p(lp, ctypes.c_double), _p(mg, ctypes.c_double))
    if rc < 0:
        raise ValueError("oracle: bad argument")
    return tok, lp, mg
