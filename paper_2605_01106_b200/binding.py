"""ctypes binding of libhs.so: argument marshalling only, every step runs in the CUDA library.

There is no fallback: if the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None

i32, i64, f32, vp = ctypes.c_int32, ctypes.c_int64, ctypes.c_float, ctypes.c_void_p

HS_FLAG_GRAPHS = 1
HS_FLAG_REPLAY = 2
HS_FLAG_LITERAL_DRAFT = 4
STATE_SSM, STATE_CONV, STATE_GDN, STATE_K, STATE_V, STATE_DRAFT, STATE_DRAFT_CONV = range(7)
EXPORTS = ["hs_query_sizes", "hs_weight_offset", "hs_init_model", "hs_reset", "hs_prefill", "hs_draft", "hs_verify",
           "hs_accept_rollback", "hs_round_host", "hs_export_state", "hs_import_state", "hs_set_context",
           "hs_set_batch", "hs_get_context", "hs_get_logits", "hs_get_round", "hs_launch_count",
           "hs_set_attn_geometry", "hs_set_sampling", "hs_set_draft_plan", "hs_set_option", "hs_profile", "hs_profile_read", "hs_device_status", "hs_clear_status",
           "hs_selftest_wait_timeout", "hs_poke_control", "hs_last_error", "hs_destroy", "hs_argmax_static"]


class HsError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__("libhs error %d: %s" % (code, msg))
        self.code = code


class HsConfig(ctypes.Structure):
    _fields_ = [(n, i32) for n in ("arch", "L", "d", "V", "H", "P", "N", "conv_w", "qh", "kvh", "hd", "ff",
                                   "gh", "gdk", "gdv", "max_batch", "max_k", "kv_capacity")] + \
               [("rope_theta", f32), ("eps", f32), ("flags", i32)]


class HsSizes(ctypes.Structure):
    _fields_ = [(n, i64) for n in ("weights", "snap", "dstate", "conv", "kv", "work")]


class HsBuffers(ctypes.Structure):
    _fields_ = [(n, vp) for n in ("weights", "snap", "dstate", "conv", "kv", "work")]


def load_library(path: str | None = None):
    """Load libhs.so (built in-tree by ``paper_2605_01106_b200.build``). Raises if it is absent."""
    global _LIB
    if _LIB is not None and path is None:
        return _LIB
    path = path or os.path.join(_HERE, "libhs.so")
    if not os.path.exists(path):
        raise FileNotFoundError("%s not found: build it with `python -m paper_2605_01106_b200.build`" % path)
    L = ctypes.CDLL(path)
    cfgp, szp, bufp = ctypes.POINTER(HsConfig), ctypes.POINTER(HsSizes), ctypes.POINTER(HsBuffers)
    L.hs_query_sizes.argtypes = [cfgp, szp]
    L.hs_weight_offset.restype = i64
    L.hs_weight_offset.argtypes = [cfgp, ctypes.c_int, ctypes.c_int]
    L.hs_init_model.argtypes = [cfgp, bufp, szp, vp, ctypes.POINTER(vp)]
    L.hs_reset.argtypes = [vp]
    L.hs_prefill.argtypes = [vp, vp, vp, ctypes.c_int]
    L.hs_draft.argtypes = [vp, ctypes.c_int]
    L.hs_verify.argtypes = [vp, ctypes.c_int, vp]
    L.hs_accept_rollback.argtypes = [vp, vp, vp, vp, vp]
    L.hs_round_host.argtypes = [vp, ctypes.c_int, vp, vp, vp, vp]
    L.hs_export_state.argtypes = [vp, ctypes.c_int, ctypes.c_int, ctypes.c_int, vp, i64]
    L.hs_import_state.argtypes = [vp, ctypes.c_int, ctypes.c_int, ctypes.c_int, vp, i64]
    L.hs_set_context.argtypes = [vp, ctypes.c_int, ctypes.c_int, ctypes.c_int]
    L.hs_set_batch.argtypes = [vp, ctypes.c_int]
    L.hs_get_context.argtypes = [vp, ctypes.c_int, vp, vp]
    L.hs_get_logits.argtypes = [vp, vp, ctypes.c_int]
    L.hs_get_round.argtypes = [vp, vp, vp, vp]
    L.hs_launch_count.restype = i64
    L.hs_launch_count.argtypes = [vp]
    L.hs_set_attn_geometry.argtypes = [vp, ctypes.c_int, ctypes.c_int]
    L.hs_set_draft_plan.argtypes = [vp, vp]
    L.hs_set_sampling.argtypes = [vp, f32, vp, vp, vp]
    L.hs_set_option.argtypes = [vp, ctypes.c_int, ctypes.c_int]
    L.hs_profile.argtypes = [vp, ctypes.c_int]
    L.hs_profile_read.argtypes = [vp, vp, vp, vp]
    L.hs_device_status.argtypes = [vp]
    L.hs_clear_status.argtypes = [vp]
    L.hs_selftest_wait_timeout.argtypes = [vp, ctypes.c_int]
    L.hs_poke_control.argtypes = [vp, ctypes.c_int, ctypes.c_int, i32]
    L.hs_last_error.restype = ctypes.c_char_p
    L.hs_last_error.argtypes = [vp]
    L.hs_destroy.argtypes = [vp]
    L.hs_argmax_static.argtypes = [vp, ctypes.c_int, ctypes.c_int, vp, vp, vp]
    _LIB = L
    return L


def lib():
    return load_library()


def argmax_static(logits_dev, tokens_dev, margins_dev=None, stream=None):
    """hs_argmax_static on torch CUDA tensors: logits [rows, V] float32 (contiguous), tokens [rows] int32,
    margins [rows] float32 or None.  Uses the library's built-in scratch: nothing is allocated.
    Runs on `stream` (torch stream) or torch's current stream; raises HsError on a non-zero status."""
    import torch
    rows, V = logits_dev.shape
    dev = logits_dev.device
    # the C entry point sees raw pointers only: what they point at is checked here, before anything is launched
    if logits_dev.dtype != torch.float32 or not logits_dev.is_contiguous() or not logits_dev.is_cuda:
        raise HsError(-1, "hs_argmax_static: logits must be a contiguous float32 CUDA tensor")
    if tokens_dev.dtype != torch.int32 or not tokens_dev.is_contiguous() or tokens_dev.device != dev or tokens_dev.numel() != rows:
        raise HsError(-1, "hs_argmax_static: tokens must be a contiguous int32 tensor of `rows` elements on the logits' device")
    if margins_dev is not None and (margins_dev.dtype != torch.float32 or not margins_dev.is_contiguous()
                                    or margins_dev.device != dev or margins_dev.numel() != rows):
        raise HsError(-1, "hs_argmax_static: margins must be a contiguous float32 tensor of `rows` elements on the logits' device")
    st = stream or torch.cuda.current_stream(dev)
    rc = lib().hs_argmax_static(logits_dev.data_ptr(), int(V), int(rows), tokens_dev.data_ptr(),
                                margins_dev.data_ptr() if margins_dev is not None else None, vp(st.cuda_stream))
    if rc != 0:
        raise HsError(rc, "hs_argmax_static: %s" % {-1: "invalid argument (null, misaligned or empty)", -2: "more than 64 rows", -5: "CUDA error"}.get(rc, "error"))


def make_config(shape, max_batch=1, max_k=8, kv_capacity=1024, flags=0) -> HsConfig:
    """hs_config from a shape object with fields arch, L, d, V, H, P, N, conv_w, qh, kvh, hd, ff, gh, gdk, gdv,
    rope_theta, eps."""
    s = shape
    return HsConfig(s.arch, s.L, s.d, s.V, s.H, s.P, s.N, s.conv_w, s.qh, s.kvh, s.hd, s.ff, s.gh, s.gdk, s.gdv,
                    max_batch, max_k, kv_capacity, s.rope_theta, s.eps, flags)


def query_sizes(cfg: HsConfig) -> HsSizes:
    sz = HsSizes()
    rc = lib().hs_query_sizes(ctypes.byref(cfg), ctypes.byref(sz))
    if rc != 0:
        raise HsError(rc, "hs_query_sizes: unsupported configuration")
    return sz


def _ptr(a):
    if a is None:
        return None
    if isinstance(a, np.ndarray):
        return a.ctypes.data
    return a.data_ptr()          # torch tensor


class Engine:
    """Owns the torch device buffers of one model instance and forwards to the C ABI.

    weights: uint8 blob (numpy, host) in the library's blob format; it is copied to the device once.
    All methods mirror the C entry points; device-side results stay on the device unless a method
    says it returns host data."""

    GUARD = 4096          # bytes of guard pattern kept behind every buffer handed to the library
    GUARD_BYTE = 0xA5

    def __init__(self, shape, weights: np.ndarray, max_batch=1, max_k=8, kv_capacity=1024, flags=0,
                 device="cuda:0", stream=None):
        import torch
        self.torch = torch
        self.shape = shape
        self.cfg = make_config(shape, max_batch, max_k, kv_capacity, flags)
        self.sizes = query_sizes(self.cfg)
        if weights.nbytes != self.sizes.weights:
            raise HsError(-2, "weight blob has %d bytes, the library expects %d" % (weights.nbytes, self.sizes.weights))
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        # a stream of its own: the legacy default stream cannot be captured into a CUDA graph
        self.stream = stream or torch.cuda.Stream(self.device)

        def alloc(n):
            # the library is told about n bytes; a guard pattern sits right behind them (see check_guards)
            n = max(int(n), 256)
            t = torch.zeros(n + self.GUARD, dtype=torch.uint8, device=self.device)
            t[n:] = self.GUARD_BYTE
            return t

        self.t_weights = alloc(self.sizes.weights)
        self.t_weights[:weights.nbytes].copy_(torch.from_numpy(weights))
        self.t_snap, self.t_dstate, self.t_conv = alloc(self.sizes.snap), alloc(self.sizes.dstate), alloc(self.sizes.conv)
        self.t_kv, self.t_work = alloc(self.sizes.kv), alloc(self.sizes.work)
        self._guarded = (self.t_weights, self.t_snap, self.t_dstate, self.t_conv, self.t_kv, self.t_work)
        self.bufs = HsBuffers(*[t.data_ptr() for t in self._guarded])
        have = HsSizes(*[t.numel() - self.GUARD for t in self._guarded])
        torch.cuda.synchronize(self.device)
        self.h = vp()
        rc = lib().hs_init_model(ctypes.byref(self.cfg), ctypes.byref(self.bufs), ctypes.byref(have),
                                 vp(self.stream.cuda_stream), ctypes.byref(self.h))
        if rc != 0:
            raise HsError(rc, "hs_init_model failed")
        self.max_k, self.max_batch = max_k, max_batch

    def _ck(self, rc):
        if rc != 0:
            raise HsError(rc, lib().hs_last_error(self.h).decode())

    def close(self):
        if getattr(self, "h", None):
            lib().hs_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the round
    def reset(self):
        self._ck(lib().hs_reset(self.h))

    def prefill(self, prompts):
        """prompts: list of int32 arrays (host)."""
        lens = np.array([len(p) for p in prompts], np.int32)
        toks = np.ascontiguousarray(np.concatenate(prompts), np.int32)
        self._ck(lib().hs_prefill(self.h, _ptr(toks), _ptr(lens), len(prompts)))
        self.batch = len(prompts)

    def draft(self, k):
        self._ck(lib().hs_draft(self.h, k))
        self.last_k = k

    def _after_torch(self, *tensors):
        # device tensors produced on torch's current stream must be complete before this stream reads them
        if any(t is not None for t in tensors):
            self.stream.wait_stream(self.torch.cuda.current_stream(self.device))

    def verify(self, k, cand_dev=None, wait=True):
        if wait:
            self._after_torch(cand_dev)
        self._ck(lib().hs_verify(self.h, k, _ptr(cand_dev)))
        self.last_k = k

    def accept_rollback(self, forced_n_dev=None, forced_next_dev=None, readback=False, wait=True):
        """Returns (n_acc [batch], emitted [batch][k+1]) as numpy when readback, else None.
        wait=False skips the stream dependency on torch's current stream (the caller guarantees that
        the device tensors are complete)."""
        if wait:
            self._after_torch(forced_n_dev, forced_next_dev)
        if not readback:
            self._ck(lib().hs_accept_rollback(self.h, _ptr(forced_n_dev), _ptr(forced_next_dev), None, None))
            return None
        b, T = self.batch, self.last_k + 1
        n, em = np.empty(b, np.int32), np.empty((b, T), np.int32)
        self._ck(lib().hs_accept_rollback(self.h, _ptr(forced_n_dev), _ptr(forced_next_dev), _ptr(n), _ptr(em)))
        return n, em

    def round_host(self, k, forced_n=None, forced_next=None):
        """One whole round with host buffers. Returns (n_acc, emitted) numpy arrays."""
        b = self.batch
        fn = np.ascontiguousarray(forced_n, np.int32) if forced_n is not None else None
        fx = np.ascontiguousarray(forced_next, np.int32) if forced_next is not None else None
        n, em = np.empty(b, np.int32), np.empty((b, k + 1), np.int32)
        self._ck(lib().hs_round_host(self.h, k, _ptr(fn), _ptr(fx), _ptr(n), _ptr(em)))
        self.last_k = k
        return n, em

    def round(self, k, forced_n_dev=None, forced_next_dev=None, cand_dev=None, readback=True):
        if cand_dev is None:
            self.draft(k)
        self.verify(k, cand_dev)
        self.last_k = k
        return self.accept_rollback(forced_n_dev, forced_next_dev, readback)

    # ---- hooks
    batch = 1
    last_k = 0

    def set_batch(self, b):
        self._ck(lib().hs_set_batch(self.h, b))
        self.batch = b

    def set_context(self, seq, kv_len, pending):
        self._ck(lib().hs_set_context(self.h, seq, kv_len, pending))
        self.batch = max(self.batch, seq + 1)

    def get_context(self, seq=0):
        a, b = i32(), i32()
        self._ck(lib().hs_get_context(self.h, seq, ctypes.byref(a), ctypes.byref(b)))
        return a.value, b.value

    def state_shape(self, kind, rows=None):
        s = self.shape
        if kind in (STATE_SSM,):
            return (s.H, s.P, s.N), np.float32
        if kind == STATE_GDN:
            return (s.gh, s.gdv, s.gdk), np.float32
        if kind == STATE_DRAFT:
            return ((s.H, s.P, s.N) if s.arch == 0 else (s.gh, s.gdv, s.gdk)), np.float32
        if kind in (STATE_CONV, STATE_DRAFT_CONV):
            return (s.conv_w - 1, s.convd), np.float32
        return (rows, s.kvh, s.hd), np.uint16

    def export_state(self, layer, seq, kind, rows=None):
        shape, dt = self.state_shape(kind, rows)
        out = np.empty(shape, dt)
        self._ck(lib().hs_export_state(self.h, layer, seq, kind, _ptr(out), out.nbytes))
        return out

    def import_state(self, layer, seq, kind, arr):
        _, dt = self.state_shape(kind, 1)
        a = np.ascontiguousarray(arr, dt)
        self._ck(lib().hs_import_state(self.h, layer, seq, kind, _ptr(a), a.nbytes))

    def get_logits(self, rows):
        out = np.empty((rows, self.shape.V), np.float32)
        self._ck(lib().hs_get_logits(self.h, _ptr(out), rows))
        return out

    def get_round(self, k=None):
        T = (self.last_k if k is None else k) + 1
        c, g, m = np.empty((self.batch, T), np.int32), np.empty((self.batch, T), np.int32), np.empty((self.batch, T), np.float32)
        self._ck(lib().hs_get_round(self.h, _ptr(c), _ptr(g), _ptr(m)))
        return c, g, m

    PROF_NAMES = ("gemv", "mixer", "attention", "argmax", "embed", "accept")

    def set_attn_geometry(self, chunk, tiles=1):
        """Fix the KV split of verify-mode attention (chunk keys x tiles per CTA); chunk = 0: automatic."""
        self._ck(lib().hs_set_attn_geometry(self.h, int(chunk), int(tiles)))

    def set_sampling(self, temperature, u_draft=None, u_accept=None, u_final=None):
        """Temperature > 0: speculative sampling (Eq. 6) with the given device tensors of uniforms (float32,
        [max_batch, max_k], [max_batch, max_k], [max_batch]); the engine keeps them alive.  0: greedy."""
        self._sampling = (u_draft, u_accept, u_final)
        if temperature > 0:
            for t, n in ((u_draft, self.max_batch * self.max_k), (u_accept, self.max_batch * self.max_k), (u_final, self.max_batch)):
                if t is None or t.dtype != self.torch.float32 or not t.is_contiguous() or t.numel() != n or t.device != self.device:
                    raise HsError(-1, "sampling needs contiguous float32 device tensors [max_batch, max_k] x2 and [max_batch]")
        self._ck(lib().hs_set_sampling(self.h, float(temperature), _ptr(u_draft), _ptr(u_accept), _ptr(u_final)))

    def set_draft_plan(self, plan=None):
        """Per-layer draft plan (0 skip, 1 recurrent pathway only, 2 whole layer), or None for the component-aware draft."""
        p = None if plan is None else np.ascontiguousarray(plan, np.int32)
        if p is not None and p.size != self.shape.L:
            raise HsError(-1, "draft plan needs one entry per layer")
        self._ck(lib().hs_set_draft_plan(self.h, _ptr(p)))

    OPT_CLUSTER_REDUCE, OPT_GEMM_MMA, OPT_GEMM_TC, OPT_PDL, OPT_ATTN_SMALL, OPT_ATTN_STREAM, OPT_TC_MIN_ROWS = range(7)

    def set_option(self, option, value):
        """Switch a kernel choice (process-wide) on or off; see hs_set_option."""
        self._ck(lib().hs_set_option(self.h, int(option), int(value)))

    def profile(self, enable):
        self._ck(lib().hs_profile(self.h, int(enable)))

    def profile_read(self):
        """{category: (ms, launches, algorithmic bytes)} accumulated since profile(True)."""
        n = len(self.PROF_NAMES)
        ms, cnt, by = np.zeros(n), np.zeros(n, np.int64), np.zeros(n)
        self._ck(lib().hs_profile_read(self.h, _ptr(ms), _ptr(cnt), _ptr(by)))
        return {k: (float(ms[i]), int(cnt[i]), float(by[i])) for i, k in enumerate(self.PROF_NAMES)}

    def launch_count(self):
        return lib().hs_launch_count(self.h)

    def device_status(self):
        return lib().hs_device_status(self.h)

    def clear_status(self):
        self._ck(lib().hs_clear_status(self.h))

    def selftest_wait_timeout(self, polls=1000):
        self._ck(lib().hs_selftest_wait_timeout(self.h, int(polls)))

    CTRL_KV_LEN, CTRL_SLOT = 0, 1

    def poke_control(self, seq, word, value):
        """Overwrite a device control word without validation (self-test of the kernels' range checks)."""
        self._ck(lib().hs_poke_control(self.h, int(seq), int(word), int(value)))

    def check_guards(self):
        """True if the guard bytes behind every buffer the library was given are untouched (synchronises)."""
        self.torch.cuda.synchronize(self.device)
        return all(bool((t[t.numel() - self.GUARD:] == self.GUARD_BYTE).all().item()) for t in self._guarded)
