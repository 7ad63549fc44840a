"""ctypes face of the Power-SMC CPU oracle -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the CPU-baseline leg of the benchmark may
import this module.  It compiles ``psmc_oracle.c`` with gcc on first use and
marshals arguments; every piece of arithmetic lives in the C file, which
follows Algorithm 1, Eq. 5, Eq. 7, Section 4.3 / Appendix B, Appendix C and
Appendix D of the paper.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "psmc_oracle.c")
_HDR = os.path.join(_HERE, "psmc_oracle.h")
_LIB = os.path.join(_HERE, "libpsmc_oracle.so")

F32, BF16, F64 = 0, 1, 2
STREAM_TOKEN, STREAM_RESAMPLE, STREAM_SELECT = 1, 2, 3


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fused multiply-add contraction, OpenMP across rows)."""
    newest = max(os.path.getmtime(_SRC), os.path.getmtime(_HDR))
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < newest:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-std=c99", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None

_i32p = C.POINTER(C.c_int32)
_f64p = C.POINTER(C.c_double)
_u8p = C.POINTER(C.c_uint8)


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.orc_sm64.restype = C.c_uint64
        L.orc_sm64.argtypes = [C.c_uint64]
        L.orc_hash5.restype = C.c_uint64
        L.orc_hash5.argtypes = [C.c_uint64] * 5
        L.orc_uniform.restype = C.c_double
        L.orc_uniform.argtypes = [C.c_uint64]
        L.orc_alpha_at.restype = C.c_double
        L.orc_alpha_at.argtypes = [C.c_double, C.c_int, C.c_int]
        L.orc_beta_at.restype = C.c_double
        L.orc_beta_at.argtypes = [C.c_double, C.c_double, C.c_int, C.c_int]
        L.orc_row.restype = C.c_int
        L.orc_row.argtypes = [_f64p, C.c_int, C.c_double, C.c_double, C.c_double, C.c_int,
                              C.POINTER(C.c_int), C.POINTER(C.c_int)] + [_f64p] * 6
        L.orc_row_masked.restype = C.c_int
        L.orc_row_masked.argtypes = [_f64p, C.c_int, C.c_double, C.c_double, C.c_double, C.c_int, C.c_double, C.c_int,
                                     C.c_int] + [C.POINTER(C.c_int)] * 4 + [_f64p] * 5
        L.orc_set_proposal_mask.restype = C.c_int
        L.orc_set_proposal_mask.argtypes = [C.c_void_p, C.c_int, C.c_double]
        L.orc_set_force_k.restype = None
        L.orc_set_force_k.argtypes = [C.c_void_p, _i32p]
        L.orc_ess.restype = None
        L.orc_ess.argtypes = [_f64p, C.c_int] + [_f64p] * 4
        L.orc_systematic.restype = None
        L.orc_systematic.argtypes = [_f64p, C.c_int, C.c_double, C.c_double, _i32p, _f64p]
        for name in ("orc_stratified", "orc_multinomial", "orc_residual"):
            f = getattr(L, name)
            f.restype = None
            f.argtypes = [_f64p, C.c_int, C.c_double, _f64p, _i32p, _f64p]
        L.orc_set_resampler.restype = C.c_int
        L.orc_set_resampler.argtypes = [C.c_void_p, C.c_int]
        L.orc_slot_map.restype = None
        L.orc_slot_map.argtypes = [_i32p, C.c_int, _i32p]
        L.orc_create.restype = C.c_void_p
        L.orc_create.argtypes = [C.c_int, C.c_int, C.c_int, C.c_double, C.c_double, C.c_double,
                                 C.c_int, C.c_uint64, C.c_int, C.c_int, _i32p]
        L.orc_destroy.restype = None
        L.orc_destroy.argtypes = [C.c_void_p]
        L.orc_reset.restype = None
        L.orc_reset.argtypes = [C.c_void_p, C.c_uint64]
        L.orc_step.restype = C.c_int
        L.orc_step.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int64, _i32p, _i32p, _i32p]
        L.orc_reindex_tensor.restype = None
        L.orc_reindex_tensor.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int,
                                         C.c_int, C.c_int64, C.c_int64, _i32p, _i32p, _i32p]
        L.orc_select.restype = None
        L.orc_select.argtypes = [C.c_void_p, _i32p, _i32p, _i32p]
        L.orc_t.restype = C.c_int
        L.orc_t.argtypes = [C.c_void_p]
        for name, typ in (("orc_tokens", _i32p), ("orc_last_tokens", _i32p), ("orc_tokens_own", _i32p),
                          ("orc_tok_margin", _f64p), ("orc_log_weights", _f64p), ("orc_log_inc", _f64p),
                          ("orc_logp_tok", _f64p), ("orc_cum_logp", _f64p), ("orc_ancestors", _i32p),
                          ("orc_anc_own", _i32p), ("orc_anc_margin", _f64p),
                          ("orc_slot_map_view", _i32p), ("orc_resampled", _i32p),
                          ("orc_resampled_own", _i32p), ("orc_ess_view", _f64p), ("orc_log_z", _f64p),
                          ("orc_lens", _i32p), ("orc_done", _u8p), ("orc_k_used", _i32p), ("orc_k_own", _i32p),
                          ("orc_k_margin", _f64p)):
            f = getattr(L, name)
            f.restype = typ
            f.argtypes = [C.c_void_p]
        L.orc_log_z_final.restype = None
        L.orc_log_z_final.argtypes = [C.c_void_p, _f64p]
        L.orc_set_state.restype = None
        L.orc_set_state.argtypes = [C.c_void_p, _f64p, _f64p, _u8p, _i32p]
        _lib = L
    return _lib


def _ptr(a, typ):
    return None if a is None else a.ctypes.data_as(typ)


def sm64(x: int) -> int:
    return lib().orc_sm64(C.c_uint64(x & (2**64 - 1)))


def hash5(a: int, b: int, c: int, d: int, e: int) -> int:
    m = 2**64 - 1
    return lib().orc_hash5(a & m, b & m, c & m, d & m, e & m)


def uniform(h: int) -> float:
    return lib().orc_uniform(h)


def alpha_at(alpha: float, ramp: int, t: int) -> float:
    return lib().orc_alpha_at(alpha, ramp, t)


def beta_at(alpha: float, tau: float, ramp: int, t: int) -> float:
    return lib().orc_beta_at(alpha, tau, ramp, t)


def row(logits, beta: float, alpha_t: float, U: float, force: int = -1) -> dict:
    """One row of Algorithm 1's inner loop on double logits."""
    l = np.ascontiguousarray(logits, dtype=np.float64)
    y, y_own = C.c_int(), C.c_int()
    out = [C.c_double() for _ in range(6)]
    rc = lib().orc_row(_ptr(l, _f64p), l.size, beta, alpha_t, U, force, C.byref(y), C.byref(y_own),
                       *[C.byref(o) for o in out])
    if rc:
        raise FloatingPointError("row has a NaN, a +inf or no finite logit")
    names = ("logp_y", "logq_y", "log_omega", "L1", "Lbeta", "margin")
    d = {n: o.value for n, o in zip(names, out)}
    d["y"], d["y_own"] = y.value, y_own.value
    return d


def row_masked(logits, beta: float, alpha_t: float, U: float, top_k: int = 0, top_p: float = 0.0, force_k: int = 0,
               force: int = -1) -> dict:
    """One row with the proposal restricted to the top_k best tokens, or to the nucleus of mass top_p."""
    l = np.ascontiguousarray(logits, dtype=np.float64)
    ints = [C.c_int() for _ in range(4)]
    out = [C.c_double() for _ in range(5)]
    rc = lib().orc_row_masked(_ptr(l, _f64p), l.size, beta, alpha_t, U, top_k, top_p, force_k, force,
                              *[C.byref(o) for o in ints], *[C.byref(o) for o in out])
    if rc == 1:
        raise ValueError("exactly one of top_k and top_p must be set")
    if rc:
        raise FloatingPointError("row has a NaN, a +inf or no finite logit")
    d = {n: o.value for n, o in zip(("k_margin", "logp_y", "logq_y", "log_omega", "margin"), out)}
    d.update({n: o.value for n, o in zip(("y", "y_own", "k", "k_own"), ints)})
    return d


def ess(logW) -> dict:
    lw = np.ascontiguousarray(logW, dtype=np.float64)
    o = [C.c_double() for _ in range(4)]
    lib().orc_ess(_ptr(lw, _f64p), lw.size, *[C.byref(x) for x in o])
    return dict(M=o[0].value, s1=o[1].value, s2=o[2].value, ess=o[3].value)


def systematic(w, u0: float):
    """Ancestors for unnormalised weights w and offset u0; returns (A, margin)."""
    w = np.ascontiguousarray(w, dtype=np.float64)
    s1 = 0.0
    for x in w:  # sequential, as in the C loop
        s1 += float(x)
    A = np.zeros(w.size, dtype=np.int32)
    mg = C.c_double()
    lib().orc_systematic(_ptr(w, _f64p), w.size, s1, u0, _ptr(A, _i32p), C.byref(mg))
    return A, mg.value


SYSTEMATIC, STRATIFIED, MULTINOMIAL, RESIDUAL = 0, 1, 2, 3


def resample(kind: int, w, u):
    """Ancestors under the stratified / multinomial / residual scheme for unnormalised weights w and
    uniforms u (one per particle); returns (A, margin)."""
    w = np.ascontiguousarray(w, dtype=np.float64)
    u = np.ascontiguousarray(u, dtype=np.float64)
    assert u.size == w.size
    s1 = 0.0
    for x in w:  # sequential, as in the C loop
        s1 += float(x)
    A = np.zeros(w.size, dtype=np.int32)
    mg = C.c_double()
    f = {STRATIFIED: lib().orc_stratified, MULTINOMIAL: lib().orc_multinomial, RESIDUAL: lib().orc_residual}[kind]
    f(_ptr(w, _f64p), w.size, s1, _ptr(u, _f64p), _ptr(A, _i32p), C.byref(mg))
    return A, mg.value


def slot_map(A):
    A = np.ascontiguousarray(A, dtype=np.int32)
    m = np.zeros_like(A)
    lib().orc_slot_map(_ptr(A, _i32p), A.size, _ptr(m, _i32p))
    return m


def reindex_tensor(dst, src, idx, copy_len=None, copy_from=None):
    """dst/src: C-contiguous numpy arrays [R, H, max_len, D]; in place when they are the same array.
    Row k receives positions [copy_from[k], copy_len[k]) of row idx[k] (defaults 0 and max_len)."""
    R, H, max_len, D = src.shape
    assert src.flags.c_contiguous and dst.flags.c_contiguous and dst.shape == src.shape
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    cl = None if copy_len is None else np.ascontiguousarray(copy_len, dtype=np.int32)
    cf = None if copy_from is None else np.ascontiguousarray(copy_from, dtype=np.int32)
    lib().orc_reindex_tensor(dst.ctypes.data, src.ctypes.data, R, H, max_len, D, src.itemsize,
                             H * max_len * D, max_len * D, _ptr(idx, _i32p), _ptr(cl, _i32p), _ptr(cf, _i32p))


class Oracle:
    """The particle system of Algorithm 1 for G independent groups of N particles."""

    def __init__(self, N, V, alpha, tau, kappa, ramp, seed, eos, G=1, T_max=4096, prompt_len=None):
        self.G, self.N, self.V, self.R, self.T_max = G, N, V, G * N, T_max
        self.alpha, self.tau, self.kappa, self.ramp, self.eos, self.seed = alpha, tau, kappa, ramp, eos, seed
        pl = None if prompt_len is None else np.ascontiguousarray(prompt_len, dtype=np.int32)
        self._h = lib().orc_create(G, N, V, alpha, tau, kappa, ramp, seed, eos, T_max, _ptr(pl, _i32p))
        if not self._h:
            raise ValueError("invalid oracle arguments")

    def __del__(self):
        if getattr(self, "_h", None):
            lib().orc_destroy(self._h)
            self._h = None

    def reset(self, seed):
        self.seed = seed
        lib().orc_reset(self._h, seed)

    def set_resampler(self, kind: int):
        if lib().orc_set_resampler(self._h, kind):
            raise ValueError("unknown resampling scheme")

    def set_proposal_mask(self, top_k: int = 0, top_p: float = 0.0):
        if lib().orc_set_proposal_mask(self._h, top_k, top_p):
            raise ValueError("at most one of top_k and top_p, top_p in (0, 1]")

    def step(self, logits, dtype=None, ld=None, force_tok=None, force_resample=None, force_anc=None, force_k=None):
        """logits: numpy [R, V] of float64 / float32, or uint16 holding bf16 bit patterns."""
        a = np.ascontiguousarray(logits)
        fk = None if force_k is None else np.ascontiguousarray(force_k, dtype=np.int32)
        lib().orc_set_force_k(self._h, _ptr(fk, _i32p))
        if dtype is None:
            dtype = {np.dtype(np.float64): F64, np.dtype(np.float32): F32, np.dtype(np.uint16): BF16}[a.dtype]
        if ld is None:
            ld = a.shape[-1]
        ft = None if force_tok is None else np.ascontiguousarray(force_tok, dtype=np.int32)
        fr = None if force_resample is None else np.ascontiguousarray(force_resample, dtype=np.int32)
        fa = None if force_anc is None else np.ascontiguousarray(force_anc, dtype=np.int32)
        rc = lib().orc_step(self._h, a.ctypes.data, dtype, ld, _ptr(ft, _i32p), _ptr(fr, _i32p), _ptr(fa, _i32p))
        lib().orc_set_force_k(self._h, None)
        if rc == 5:
            raise FloatingPointError("a row has a NaN, a +inf or no finite logit")
        if rc:
            raise RuntimeError("oracle step failed with code %d" % rc)

    def select(self):
        toks = np.zeros((self.G, self.T_max), dtype=np.int32)
        ln = np.zeros(self.G, dtype=np.int32)
        ix = np.zeros(self.G, dtype=np.int32)
        lib().orc_select(self._h, _ptr(toks, _i32p), _ptr(ln, _i32p), _ptr(ix, _i32p))
        return toks, ln, ix

    def set_state(self, logW=None, S=None, done=None, lens=None):
        a = None if logW is None else np.ascontiguousarray(logW, dtype=np.float64)
        b = None if S is None else np.ascontiguousarray(S, dtype=np.float64)
        c = None if done is None else np.ascontiguousarray(done, dtype=np.uint8)
        d = None if lens is None else np.ascontiguousarray(lens, dtype=np.int32)
        lib().orc_set_state(self._h, _ptr(a, _f64p), _ptr(b, _f64p), _ptr(c, _u8p), _ptr(d, _i32p))

    def _view(self, name, n, dt):
        p = getattr(lib(), name)(self._h)
        return np.ctypeslib.as_array(p, shape=(n,)).astype(dt, copy=True)

    t = property(lambda s: lib().orc_t(s._h))
    tokens = property(lambda s: s._view("orc_tokens", s.R, np.int32))
    last_tokens = property(lambda s: s._view("orc_last_tokens", s.R, np.int32))
    tokens_own = property(lambda s: s._view("orc_tokens_own", s.R, np.int32))
    tok_margin = property(lambda s: s._view("orc_tok_margin", s.R, np.float64))
    log_weights = property(lambda s: s._view("orc_log_weights", s.R, np.float64))
    log_inc = property(lambda s: s._view("orc_log_inc", s.R, np.float64))
    logp_tok = property(lambda s: s._view("orc_logp_tok", s.R, np.float64))
    cum_logp = property(lambda s: s._view("orc_cum_logp", s.R, np.float64))
    ancestors = property(lambda s: s._view("orc_ancestors", s.R, np.int32))
    anc_own = property(lambda s: s._view("orc_anc_own", s.R, np.int32))
    anc_margin = property(lambda s: s._view("orc_anc_margin", s.G, np.float64))
    slot_map = property(lambda s: s._view("orc_slot_map_view", s.R, np.int32))
    resampled = property(lambda s: s._view("orc_resampled", s.G, np.int32))
    resampled_own = property(lambda s: s._view("orc_resampled_own", s.G, np.int32))
    ess = property(lambda s: s._view("orc_ess_view", s.G, np.float64))
    log_z = property(lambda s: s._view("orc_log_z", s.G, np.float64))
    lens = property(lambda s: s._view("orc_lens", s.R, np.int32))
    done = property(lambda s: s._view("orc_done", s.R, np.uint8))
    k_used = property(lambda s: s._view("orc_k_used", s.R, np.int32))
    k_own = property(lambda s: s._view("orc_k_own", s.R, np.int32))
    k_margin = property(lambda s: s._view("orc_k_margin", s.R, np.float64))

    @property
    def log_z_final(self):
        out = np.zeros(self.G, dtype=np.float64)
        lib().orc_log_z_final(self._h, _ptr(out, _f64p))
        return out
