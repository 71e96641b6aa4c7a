"""ctypes front end of the plain-C FP64 oracle (test infrastructure only).

Inputs are BF16 bit patterns (numpy ``uint16``) shaped ``[B, H, N, d]``; outputs
are FP64 and never cast.  See ``gproj_oracle.c`` for the formulas
(Eq. "row-attention", Eq. "row-gradients").
"""
import ctypes

import numpy as np

from . import build as _build

_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        u16p = ctypes.POINTER(ctypes.c_uint16)
        f64p = ctypes.POINTER(ctypes.c_double)
        i32p = ctypes.POINTER(ctypes.c_int)
        lib.gproj_oracle_head_rows.restype = ctypes.c_int
        lib.gproj_oracle_head_rows.argtypes = [u16p, u16p, u16p, u16p, ctypes.c_int, ctypes.c_int,
                                               ctypes.c_double, ctypes.c_int, i32p, ctypes.c_int,
                                               f64p, f64p, f64p, f64p]
        lib.gproj_oracle_head_keys.restype = ctypes.c_int
        lib.gproj_oracle_head_keys.argtypes = [u16p, u16p, u16p, u16p, ctypes.c_int, ctypes.c_int,
                                               ctypes.c_double, ctypes.c_int, f64p, f64p, i32p, ctypes.c_int,
                                               f64p, f64p]
        lib.gproj_oracle_rect_rows.restype = ctypes.c_int
        lib.gproj_oracle_rect_rows.argtypes = [u16p, u16p, u16p, u16p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                               ctypes.c_double, ctypes.c_int, i32p, ctypes.c_int,
                                               f64p, f64p, f64p, f64p]
        lib.gproj_oracle_rect_keys.restype = ctypes.c_int
        lib.gproj_oracle_rect_keys.argtypes = [u16p, u16p, u16p, u16p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                               ctypes.c_double, ctypes.c_int, f64p, f64p, i32p, ctypes.c_int,
                                               f64p, f64p]
        lib.gproj_oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def num_threads() -> int:
    """Threads the oracle's OpenMP loops will use on this host."""
    return int(_load().gproj_oracle_num_threads())


def _u16(x):
    x = np.ascontiguousarray(x)
    if x.dtype != np.uint16:
        raise TypeError("oracle inputs are BF16 bit patterns (numpy uint16)")
    return x


def _p(x, ct):
    return x.ctypes.data_as(ctypes.POINTER(ct))


def head_rows_f64(q, k, v, u, alpha, causal, rows):
    """O, LSE, mu_a and dQ of the listed query rows of ONE head ([N, d] inputs)."""
    q, k, v, u = map(_u16, (q, k, v, u))
    N, d = q.shape
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    n = rows.shape[0]
    O = np.empty((n, d)); LSE = np.empty(n); MUA = np.empty(n); dQ = np.empty((n, d))
    rc = _load().gproj_oracle_head_rows(_p(q, ctypes.c_uint16), _p(k, ctypes.c_uint16), _p(v, ctypes.c_uint16),
                                        _p(u, ctypes.c_uint16), N, d, float(alpha), int(bool(causal)),
                                        _p(rows, ctypes.c_int), n,
                                        _p(O, ctypes.c_double), _p(LSE, ctypes.c_double),
                                        _p(MUA, ctypes.c_double), _p(dQ, ctypes.c_double))
    if rc != 0:
        raise RuntimeError("gproj_oracle_head_rows failed")
    return O, LSE, MUA, dQ


def head_keys_f64(q, k, v, u, alpha, causal, LSE, MUA, keys):
    """dK and dV of the listed key rows of ONE head, given LSE and mu_a of every query row."""
    q, k, v, u = map(_u16, (q, k, v, u))
    N, d = q.shape
    LSE = np.ascontiguousarray(LSE, dtype=np.float64); MUA = np.ascontiguousarray(MUA, dtype=np.float64)
    assert LSE.shape == (N,) and MUA.shape == (N,)
    keys = np.ascontiguousarray(keys, dtype=np.int32)
    n = keys.shape[0]
    dK = np.empty((n, d)); dV = np.empty((n, d))
    rc = _load().gproj_oracle_head_keys(_p(q, ctypes.c_uint16), _p(k, ctypes.c_uint16), _p(v, ctypes.c_uint16),
                                        _p(u, ctypes.c_uint16), N, d, float(alpha), int(bool(causal)),
                                        _p(LSE, ctypes.c_double), _p(MUA, ctypes.c_double),
                                        _p(keys, ctypes.c_int), n,
                                        _p(dK, ctypes.c_double), _p(dV, ctypes.c_double))
    if rc != 0:
        raise RuntimeError("gproj_oracle_head_keys failed")
    return dK, dV


def attn_fwd_bwd_f64(Q, K, V, dO, alpha, causal, heads=None):
    """Exact forward and VJP for BF16-bit inputs Q, dO ``[B, H, N, d]`` and K, V ``[B, Hkv, N, d]`` (H % Hkv == 0).

    Query head h reads key / value head h // (H // Hkv); dK and dV sum over the query heads that share a KV head
    (Section 3.1, text after Eq. "row-gradients").  ``heads`` optionally restricts the work to a list of flat
    (b*H + h) query-head indices (only for Hkv == H); the returned arrays then have that many leading entries.
    Returns a dict with O, LSE, MUA, dQ ([.., H, ..]) and dK, dV ([.., Hkv, ..]) in FP64, uncast.
    """
    Q, K, V, dO = map(_u16, (Q, K, V, dO))
    B, H, N, d = Q.shape
    Hkv = K.shape[1]
    if K.shape != (B, Hkv, N, d) or V.shape != K.shape or dO.shape != Q.shape or H % Hkv != 0:
        raise ValueError("shape mismatch")
    G = H // Hkv
    Qf, Uf = Q.reshape(B * H, N, d), dO.reshape(B * H, N, d)
    Kf, Vf = K.reshape(B * Hkv, N, d), V.reshape(B * Hkv, N, d)
    kv_of = lambda bh: (bh // H) * Hkv + (bh % H) // G
    if heads is not None and G != 1:
        raise ValueError("a head subset is only supported without grouped queries")
    idx = list(range(B * H)) if heads is None else list(heads)
    n = len(idx)
    out = {"O": np.empty((n, N, d)), "LSE": np.empty((n, N)), "MUA": np.empty((n, N)), "dQ": np.empty((n, N, d))}
    nkv = B * Hkv if heads is None else n
    out["dK"] = np.zeros((nkv, N, d)); out["dV"] = np.zeros((nkv, N, d))
    allrows = np.arange(N, dtype=np.int32)
    for t, bh in enumerate(idx):
        kv = kv_of(bh)
        O, LSE, MUA, dQ = head_rows_f64(Qf[bh], Kf[kv], Vf[kv], Uf[bh], alpha, causal, allrows)
        dK, dV = head_keys_f64(Qf[bh], Kf[kv], Vf[kv], Uf[bh], alpha, causal, LSE, MUA, allrows)
        out["O"][t], out["LSE"][t], out["MUA"][t], out["dQ"][t] = O, LSE, MUA, dQ
        slot = kv if heads is None else t
        out["dK"][slot] += dK
        out["dV"][slot] += dV
    if heads is None:
        for key in ("O", "LSE", "MUA", "dQ"):
            out[key] = out[key].reshape((B, H) + out[key].shape[1:])
        for key in ("dK", "dV"):
            out[key] = out[key].reshape((B, Hkv) + out[key].shape[1:])
    return out


def attn_rect_f64(Q, K, V, dO, alpha, causal):
    """Exact forward and VJP with N_q queries and N_k keys: Q, dO ``[B, H, Nq, d]``, K, V ``[B, Hkv, Nk, d]`` (BF16 bits).

    Causal support of query i: keys j <= i + (Nk - Nq) (the diagonal ends at the last query and the last key); a row with
    an empty support has O = dQ = 0 and LSE = +inf (Algorithm 1, line 14, gives such a row no correction either).
    Returns O, LSE, MUA, dQ ([B, H, Nq, ..]) and dK, dV ([B, Hkv, Nk, d]) in FP64.
    """
    Q, K, V, dO = map(_u16, (Q, K, V, dO))
    B, H, Nq, d = Q.shape
    Hkv, Nk = K.shape[1], K.shape[2]
    if K.shape != (B, Hkv, Nk, d) or V.shape != K.shape or dO.shape != Q.shape or H % Hkv != 0:
        raise ValueError("shape mismatch")
    G = H // Hkv
    out = {"O": np.empty((B, H, Nq, d)), "LSE": np.empty((B, H, Nq)), "MUA": np.empty((B, H, Nq)), "dQ": np.empty((B, H, Nq, d)),
           "dK": np.zeros((B, Hkv, Nk, d)), "dV": np.zeros((B, Hkv, Nk, d))}
    rows = np.arange(Nq, dtype=np.int32); keys = np.arange(Nk, dtype=np.int32)
    lib = _load()
    for b in range(B):
        for h in range(H):
            q, u, k, v = Q[b, h], dO[b, h], K[b, h // G], V[b, h // G]
            args = (_p(q, ctypes.c_uint16), _p(k, ctypes.c_uint16), _p(v, ctypes.c_uint16), _p(u, ctypes.c_uint16),
                    Nq, Nk, d, float(alpha), int(bool(causal)))
            O = np.empty((Nq, d)); LSE = np.empty(Nq); MUA = np.empty(Nq); dQ = np.empty((Nq, d))
            if lib.gproj_oracle_rect_rows(*args, _p(rows, ctypes.c_int), Nq, _p(O, ctypes.c_double), _p(LSE, ctypes.c_double),
                                          _p(MUA, ctypes.c_double), _p(dQ, ctypes.c_double)) != 0:
                raise RuntimeError("gproj_oracle_rect_rows failed")
            dK = np.empty((Nk, d)); dV = np.empty((Nk, d))
            if lib.gproj_oracle_rect_keys(*args, _p(LSE, ctypes.c_double), _p(MUA, ctypes.c_double), _p(keys, ctypes.c_int), Nk,
                                          _p(dK, ctypes.c_double), _p(dV, ctypes.c_double)) != 0:
                raise RuntimeError("gproj_oracle_rect_keys failed")
            out["O"][b, h], out["LSE"][b, h], out["MUA"][b, h], out["dQ"][b, h] = O, LSE, MUA, dQ
            out["dK"][b, h // G] += dK
            out["dV"][b, h // G] += dV
    return out


def rel_l2_percent(approx, exact) -> float:
    """100 * ||approx - exact||_2 / ||exact||_2 over the full tensor (Appendix "Reference and metric")."""
    approx = np.asarray(approx, dtype=np.float64); exact = np.asarray(exact, dtype=np.float64)
    den = np.linalg.norm(exact.ravel())
    num = np.linalg.norm((approx - exact).ravel())
    if den == 0.0:
        return 0.0 if num == 0.0 else float("inf")
    return 100.0 * num / den
