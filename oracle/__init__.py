"""CPU oracle (test infrastructure only): ctypes front end of hs_oracle.c.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None

c_int, c_i64, c_dbl, vp = ctypes.c_int, ctypes.c_int64, ctypes.c_double, ctypes.c_void_p


class OrConfig(ctypes.Structure):
    _fields_ = [(n, c_int) for n in ("arch", "L", "d", "V", "H", "P", "N", "conv_w", "qh", "kvh", "hd", "ff",
                                     "gh", "gdk", "gdv", "kv_capacity")] + [("rope_theta", c_dbl), ("eps", c_dbl)]


class OrMat(ctypes.Structure):
    _fields_ = [("off", c_i64), ("stride", c_i64)]


class OrLayer(ctypes.Structure):
    _fields_ = ([("type", c_int)] +
                [(n, c_i64) for n in ("norm1", "conv_w", "conv_b", "A_log", "D", "dt_bias", "gnorm", "norm2")] +
                [(n, OrMat) for n in ("Wz", "Wxbc", "Wdt", "Wq", "Wk", "Wv", "Wo", "Wgz", "Wga", "Wgb", "Wout",
                                      "Wgate", "Wup", "Wdown")])


def build_lib(force: bool = False) -> str:
    src = os.path.join(_HERE, "hs_oracle.c")
    hdr = os.path.join(_HERE, "hs_oracle.h")
    out = os.path.join(_HERE, "libhs_oracle.so")
    newest = max(os.path.getmtime(src), os.path.getmtime(hdr))
    if force or not os.path.exists(out) or os.path.getmtime(out) < newest:
        tmp = out + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC",
                               "-o", tmp, src, "-lm"])
        os.replace(tmp, out)
    return out


def lib():
    global _LIB
    if _LIB is None:
        L = ctypes.CDLL(build_lib())
        L.or_model_create.restype = vp
        L.or_model_create.argtypes = [ctypes.POINTER(OrConfig), vp, ctypes.POINTER(OrLayer), c_i64, c_i64, c_i64]
        L.or_model_destroy.argtypes = [vp]
        L.or_model_set_draft_plan.argtypes = [vp, vp]
        L.or_seq_create.restype = vp
        L.or_seq_create.argtypes = [vp]
        for f in ("or_seq_destroy", "or_seq_reset"):
            getattr(L, f).argtypes = [vp]
        L.or_seq_len.argtypes = [vp]
        L.or_seq_pending.argtypes = [vp]
        L.or_seq_set.argtypes = [vp, c_int, c_int]
        L.or_model_set_literal_draft.argtypes = [vp, c_int]
        for f in ("or_seq_ssm", "or_seq_conv", "or_seq_gdn", "or_seq_k", "or_seq_v", "or_seq_draft_ssm", "or_seq_draft_conv", "or_seq_draft_gdn"):
            getattr(L, f).restype = vp
            getattr(L, f).argtypes = [vp]
        L.or_step_committed.argtypes = [vp, c_int, c_int, vp]
        L.or_prefill.argtypes = [vp, vp, c_int]
        L.or_greedy.argtypes = [vp, c_int, vp]
        L.or_draft_only.argtypes = [vp, c_int, vp, vp]
        L.or_round.argtypes = [vp, c_int, vp, c_int, c_int, vp, vp, vp, vp, vp, vp]
        L.or_rmsnorm.argtypes = [vp, vp, c_int, c_dbl, vp]
        L.or_matvec.argtypes = [vp, OrMat, c_int, c_int, vp, vp]
        L.or_conv_step.restype = c_dbl
        L.or_conv_step.argtypes = [vp, c_dbl, vp, c_dbl]
        L.or_ssm_step.argtypes = [vp, c_int, c_int, c_dbl, c_dbl, c_dbl, vp, vp, vp, vp]
        L.or_ssd_chunk.argtypes = [vp, c_int, c_int, c_int, vp, c_dbl, c_dbl, vp, vp, vp, vp, vp]
        L.or_gdn_step.argtypes = [vp, c_int, c_int, c_dbl, c_dbl, vp, vp, vp, vp]
        L.or_rope.argtypes = [vp, c_int, c_int, c_dbl]
        L.or_attention.argtypes = [vp, vp, vp, c_i64, c_int, c_int, c_int, c_int, vp]
        L.or_argmax_margin.argtypes = [vp, c_int, vp]
        L.or_accept_len.argtypes = [vp, vp, c_int]
        L.or_softmax_t.argtypes = [vp, c_int, c_dbl, vp]
        L.or_sample_cdf.argtypes = [vp, c_int, c_dbl, vp]
        L.or_spec_accept.argtypes = [vp, vp, c_int, c_dbl, vp]
        L.or_residual.argtypes = [vp, vp, c_int, vp]
        L.or_round_sampled.argtypes = [vp, c_int, c_dbl, vp, vp, c_dbl, vp, c_int, c_int, vp, vp, vp, vp]
        _LIB = L
    return _LIB


def _p(a):
    return a.ctypes.data if a is not None else None


def _f64(a):
    return np.ascontiguousarray(a, np.float64)


# ------------------------------------------------------------------ components
def rmsnorm(x, w, eps):
    x = _f64(x); w = np.ascontiguousarray(w, np.float32); out = np.empty_like(x)
    lib().or_rmsnorm(_p(x), _p(w), x.size, eps, _p(out))
    return out


def matvec_bf16(w_bits, x):
    """w_bits: uint16 [rows, cols] bf16 bit patterns."""
    w = np.ascontiguousarray(w_bits, np.uint16); x = _f64(x)
    y = np.empty(w.shape[0], np.float64)
    lib().or_matvec(_p(w), OrMat(0, w.shape[1]), w.shape[0], w.shape[1], _p(x), _p(y))
    return y


def conv_step(win3, cur, taps4, bias):
    """Returns (pre-activation output, shifted window)."""
    w = _f64(win3).copy(); t = np.ascontiguousarray(taps4, np.float32)
    o = lib().or_conv_step(_p(w), float(cur), _p(t), float(bias))
    return o, w


def ssm_step(S, dt, A, D, x, B, C):
    """One head. Returns (S_new [P,N], y [P])."""
    S = _f64(S).copy(); P, N = S.shape
    x, B, C = _f64(x), _f64(B), _f64(C); y = np.empty(P)
    lib().or_ssm_step(_p(S), P, N, dt, A, D, _p(x), _p(B), _p(C), _p(y))
    return S, y


def ssd_chunk(S0, dt, A, D, x, B, C):
    """One head, T positions. x [T,P], B,C [T,N]. Returns (y [T,P], snaps [T,P,N])."""
    S0 = _f64(S0); P, N = S0.shape
    dt, x, B, C = _f64(dt), _f64(x), _f64(B), _f64(C); T = dt.size
    y = np.empty((T, P)); snaps = np.empty((T, P, N))
    lib().or_ssd_chunk(_p(S0), P, N, T, _p(dt), A, D, _p(x), _p(B), _p(C), _p(y), _p(snaps))
    return y, snaps


def gdn_step(S, alpha, beta, q, k, v):
    S = _f64(S).copy(); dv, dk = S.shape
    q, k, v = _f64(q), _f64(k), _f64(v); o = np.empty(dv)
    lib().or_gdn_step(_p(S), dv, dk, alpha, beta, _p(q), _p(k), _p(v), _p(o))
    return S, o


def rope(x, pos, theta=10000.0):
    x = _f64(x).copy()
    lib().or_rope(_p(x), x.size, pos, theta)
    return x


def attention(q, K_bits, V_bits, qh, kvh, hd):
    """q [qh, hd]; K_bits, V_bits uint16 [len, kvh, hd]. Returns [qh, hd]."""
    q = _f64(q); K = np.ascontiguousarray(K_bits, np.uint16); V = np.ascontiguousarray(V_bits, np.uint16)
    out = np.empty((qh, hd))
    lib().or_attention(_p(q), _p(K), _p(V), kvh * hd, K.shape[0], qh, kvh, hd, _p(out))
    return out


def argmax_margin(logits):
    lg = _f64(logits); m = c_dbl()
    i = lib().or_argmax_margin(_p(lg), lg.size, ctypes.byref(m))
    return i, m.value


def accept_len(d, g):
    d = np.ascontiguousarray(d, np.int32); g = np.ascontiguousarray(g, np.int32)
    return lib().or_accept_len(_p(d), _p(g), d.size)


def softmax_t(logits, tau):
    lg = _f64(logits); p = np.empty_like(lg)
    lib().or_softmax_t(_p(lg), lg.size, float(tau), _p(p))
    return p


def sample_cdf(w, u):
    """(index, margin) of the inverse-CDF draw from unnormalised weights w with uniform u."""
    w = _f64(w); m = c_dbl()
    return lib().or_sample_cdf(_p(w), w.size, float(u), ctypes.byref(m)), m.value


def spec_accept(pS, pH, x, u):
    pS, pH = _f64(pS), _f64(pH); m = c_dbl()
    return bool(lib().or_spec_accept(_p(pS), _p(pH), int(x), float(u), ctypes.byref(m))), m.value


def residual(pS, pH):
    pS, pH = _f64(pS), _f64(pH); r = np.empty_like(pS)
    lib().or_residual(_p(pS), _p(pH), pS.size, _p(r))
    return r


# ---------------------------------------------------------------------- model
def _layer_desc(shape, table, l):
    """Describe layer l to the oracle from the blob's offset table ((layer, tid) -> (offset, shape, dtype)).
    Tensor ids follow the blob format: 0 norm1, 1 in-projection, 2 conv taps, 3 conv bias, 4 A_log, 5 D,
    6 dt_bias, 7 gated/out norm, 8 out-projection, 9 W_o, 10 norm2, 11 gate/up interleaved, 12 down."""
    s = shape
    ly = OrLayer()
    ly.type = s.layer_type(l)

    def off(tid):
        return table[(l, tid)][0] if (l, tid) in table else -1

    ly.norm1, ly.conv_w, ly.conv_b = off(0), off(2), off(3)
    ly.A_log, ly.D, ly.dt_bias, ly.gnorm, ly.norm2 = off(4), off(5), off(6), off(7), off(10)
    none = OrMat(-1, 0)
    for n in ("Wz", "Wxbc", "Wdt", "Wq", "Wk", "Wv", "Wo", "Wgz", "Wga", "Wgb", "Wout"):
        setattr(ly, n, none)
    w_in, d = off(1), s.d
    row = lambda r: OrMat(w_in + 2 * d * r, d)
    if ly.type == 0:
        di = s.H * s.P
        convd = di + 2 * s.N
        ly.Wz, ly.Wxbc, ly.Wdt = row(0), row(di), row(di + convd)
        r0 = di + convd + s.H
        ly.Wq, ly.Wk, ly.Wv = row(r0), row(r0 + s.qh * s.hd), row(r0 + (s.qh + s.kvh) * s.hd)
        ly.Wout, ly.Wo = OrMat(off(8), di), OrMat(off(9), s.qh * s.hd)
    elif ly.type == 1:
        nk, nv = s.gh * s.gdk, s.gh * s.gdv
        ly.Wq, ly.Wk, ly.Wv = row(0), row(nk), row(2 * nk)
        ly.Wgz, ly.Wga, ly.Wgb = row(2 * nk + nv), row(2 * nk + 2 * nv), row(2 * nk + 2 * nv + s.gh)
        ly.Wout = OrMat(off(8), nv)
    else:
        ly.Wq, ly.Wk, ly.Wv = row(0), row(s.qh * s.hd), row((s.qh + s.kvh) * s.hd)
        ly.Wo = OrMat(off(9), s.qh * s.hd)
    gu = off(11)
    ly.Wgate, ly.Wup = OrMat(gu, 2 * d), OrMat(gu + 2 * d, 2 * d)
    ly.Wdown = OrMat(off(12), s.ff)
    return ly


class Model:
    def __init__(self, shape, blob: np.ndarray, table, kv_capacity: int, layer_ids=None):
        """layer_ids: optional subset of the blob's layers to stack (used to pin the draft of a
        sequential hybrid against a model whose attention layers were deleted)."""
        s = shape
        ids = list(range(s.L)) if layer_ids is None else list(layer_ids)
        if layer_ids is not None:
            shape = s.replace(L=len(ids))
        self.shape, self.blob, self.cap = shape, blob, kv_capacity
        self.cfg = OrConfig(s.arch, len(ids), s.d, s.V, s.H, s.P, s.N, s.conv_w, s.qh, s.kvh, s.hd, s.ff,
                            s.gh, s.gdk, s.gdv, kv_capacity, s.rope_theta, s.eps)
        layers = (OrLayer * len(ids))(*[_layer_desc(s, table, l) for l in ids])
        self.h = lib().or_model_create(ctypes.byref(self.cfg), _p(blob), layers, table[(-1, 0)][0],
                                       table[(-1, 1)][0], table[(-1, 2)][0])

    def __del__(self):
        if getattr(self, "h", None):
            lib().or_model_destroy(self.h)
            self.h = None

    def new_seq(self) -> "Seq":
        return Seq(self)

    def set_literal_draft(self, on=True):
        """The draft model keeps its own attention-free recurrent state over the whole history (Eq. 4 / Eq. 5 literally)."""
        lib().or_model_set_literal_draft(self.h, int(bool(on)))

    def set_draft_plan(self, plan=None):
        """Per-layer draft plan (0 skip the layer, 1 recurrent pathway only, 2 whole layer); None: component-aware."""
        if plan is None:
            lib().or_model_set_draft_plan(self.h, None)
        else:
            p = np.ascontiguousarray(plan, np.int32)
            assert p.size == self.cfg.L
            lib().or_model_set_draft_plan(self.h, _p(p))


class Seq:
    def __init__(self, model: Model):
        self.m = model
        self.h = lib().or_seq_create(model.h)

    def __del__(self):
        if getattr(self, "h", None):
            lib().or_seq_destroy(self.h)
            self.h = None

    def reset(self):
        lib().or_seq_reset(self.h)

    @property
    def len(self):
        return lib().or_seq_len(self.h)

    @property
    def pending(self):
        return lib().or_seq_pending(self.h)

    def set(self, length, pending):
        lib().or_seq_set(self.h, length, pending)

    def _view(self, fn, shape, dtype):
        ptr = getattr(lib(), fn)(self.h)
        if not ptr:
            return None
        n = int(np.prod(shape))
        buf = (ctypes.c_byte * (n * np.dtype(dtype).itemsize)).from_address(ptr)
        return np.frombuffer(buf, dtype=dtype).reshape(shape)

    def ssm(self):
        s = self.m.shape
        return self._view("or_seq_ssm", (s.L, s.H, s.P, s.N), np.float64) if s.arch == 0 else None

    def conv(self):
        s = self.m.shape
        return self._view("or_seq_conv", (s.L, s.conv_w - 1, s.convd), np.float64)

    def gdn(self):
        s = self.m.shape
        return self._view("or_seq_gdn", (s.L, s.gh, s.gdv, s.gdk), np.float64) if s.arch == 1 else None

    def draft_state(self):
        """(recurrent state, conv window) of the draft model's own history (literal reading of Eq. 4 / Eq. 5)."""
        s = self.m.shape
        rec = (self._view("or_seq_draft_ssm", (s.L, s.H, s.P, s.N), np.float64) if s.arch == 0
               else self._view("or_seq_draft_gdn", (s.L, s.gh, s.gdv, s.gdk), np.float64))
        return rec, self._view("or_seq_draft_conv", (s.L, s.conv_w - 1, s.convd), np.float64)

    def k(self):
        s = self.m.shape
        return self._view("or_seq_k", (s.L, self.m.cap, s.kvh, s.hd), np.uint16)

    def v(self):
        s = self.m.shape
        return self._view("or_seq_v", (s.L, self.m.cap, s.kvh, s.hd), np.uint16)

    def step(self, token, mode=0):
        lg = np.empty(self.m.shape.V)
        rc = lib().or_step_committed(self.h, int(token), mode, _p(lg))
        assert rc == 0, rc
        return lg

    def prefill(self, tokens):
        t = np.ascontiguousarray(tokens, np.int32)
        rc = lib().or_prefill(self.h, _p(t), t.size)
        assert rc == 0, rc
        return self.pending

    def greedy(self, n):
        out = np.empty(n, np.int32)
        rc = lib().or_greedy(self.h, n, _p(out))
        assert rc == 0, rc
        return out

    def draft_only(self, k, want_logits=False):
        d = np.empty(k, np.int32)
        lg = np.empty((k, self.m.shape.V)) if want_logits else None
        rc = lib().or_draft_only(self.h, k, _p(d), _p(lg))
        assert rc == 0, rc
        return (d, lg) if want_logits else d

    def round_sampled(self, k, tau, u_draft, u_acc, u_final, cand_in=None, forced_n=-1, forced_next=-1):
        """One round at temperature tau > 0 (Eq. 6). Returns dict(cand, n, emitted, margins[2k+1])."""
        T = k + 1
        ud, ua = _f64(u_draft), _f64(u_acc)
        assert ud.size >= k and ua.size >= k
        ci = np.ascontiguousarray(cand_in, np.int32) if cand_in is not None else None
        cand, em, mg = np.empty(T, np.int32), np.full(T, -1, np.int32), np.ones(2 * k + 1)
        n = c_int()
        rc = lib().or_round_sampled(self.h, k, float(tau), _p(ud), _p(ua), float(u_final), _p(ci), forced_n, forced_next,
                                    _p(cand), ctypes.byref(n), _p(em), _p(mg))
        assert rc == 0, rc
        return dict(cand=cand, n=n.value, emitted=em[:n.value + 1].copy(), margins=mg)

    def round(self, k, cand_in=None, forced_n=-1, forced_next=-1, want_logits=False):
        """One speculative round. Returns dict(cand, g, margin, logits, n, emitted)."""
        T = k + 1
        ci = np.ascontiguousarray(cand_in, np.int32) if cand_in is not None else None
        cand, g, em = np.empty(T, np.int32), np.empty(T, np.int32), np.full(T, -1, np.int32)
        margin = np.empty(T)
        lg = np.empty((T, self.m.shape.V)) if want_logits else None
        n = c_int()
        rc = lib().or_round(self.h, k, _p(ci), forced_n, forced_next, _p(cand), _p(g), _p(margin), _p(lg),
                            ctypes.byref(n), _p(em))
        assert rc == 0, rc
        return dict(cand=cand, g=g, margin=margin, logits=lg, n=n.value, emitted=em[:n.value + 1].copy())
