"""Seeded synthetic inputs for the hybrid speculative-decoding hot path.

This module only *generates data*: model shapes, random weight bytes in the
documented blob format, prompts, accept patterns and injected contexts.  It
holds none of the method's arithmetic and is the only code that both the CUDA
library's tests and the CPU oracle's tests use.

Everything is a pure function of (seed, tensor id, element index) through a
splitmix-style counter generator; the bulk fills run in a small C helper
(``gen.c``) and the same word stream is re-implemented in numpy for the small
tensors, so a slice can be regenerated anywhere.
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess
from dataclasses import dataclass, field, asdict

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None

ARCH_PARALLEL = 0
ARCH_SEQUENTIAL = 1

LAYER_PAR = 0   # Mamba-2 + attention summed in one block
LAYER_GDN = 1   # Gated DeltaNet layer of a sequential hybrid
LAYER_ATT = 2   # softmax-attention layer of a sequential hybrid


def build_lib(force: bool = False) -> str:
    """Compile gen.c into libhsin.so next to it (gcc, OpenMP) if stale."""
    src = os.path.join(_HERE, "gen.c")
    out = os.path.join(_HERE, "libhsin.so")
    if force or not os.path.exists(out) or os.path.getmtime(out) < os.path.getmtime(src):
        tmp = out + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, src, "-lm"])
        os.replace(tmp, out)
    return out


def _lib():
    global _LIB
    if _LIB is None:
        lib = ctypes.CDLL(build_lib())
        u64, i64, vp = ctypes.c_uint64, ctypes.c_int64, ctypes.c_void_p
        lib.hsin_base.restype = u64
        lib.hsin_base.argtypes = [u64, u64]
        lib.hsin_words.argtypes = [vp, i64, u64, u64, i64]
        lib.hsin_normal_bf16.argtypes = [vp, i64, u64, u64, ctypes.c_double, i64]
        lib.hsin_grid_bf16.argtypes = [vp, i64, u64, u64, ctypes.c_float, i64]
        lib.hsin_grid_f32.argtypes = [vp, i64, u64, u64, ctypes.c_float, i64]
        _LIB = lib
    return _LIB


# ----------------------------------------------------------------------------
# word stream (numpy twin of gen.c)
# ----------------------------------------------------------------------------
_GAMMA = np.uint64(0x9E3779B97F4A7C15)


def _fin64(z: np.ndarray) -> np.ndarray:
    z = z.astype(np.uint64, copy=True)
    with np.errstate(over="ignore"):
        z ^= z >> np.uint64(30)
        z *= np.uint64(0xBF58476D1CE4E5B9)
        z ^= z >> np.uint64(27)
        z *= np.uint64(0x94D049BB133111EB)
        z ^= z >> np.uint64(31)
    return z


def _base(seed: int, tid: int) -> np.uint64:
    with np.errstate(over="ignore"):
        s = _fin64(np.array([seed], np.uint64) + _GAMMA)
        t = np.array([tid], np.uint64) * np.uint64(0xD1B54A32D192ED03)
        return _fin64((s ^ t) + _GAMMA)[0]


def words(seed: int, tid: int, n: int, first: int = 0) -> np.ndarray:
    """n raw 64-bit words of stream (seed, tid), element indices first..first+n-1."""
    idx = np.arange(first + 1, first + n + 1, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return _fin64(_base(seed, tid) + idx * _GAMMA)


def uniform01(seed: int, tid: int, n: int, first: int = 0) -> np.ndarray:
    """float64 uniforms in (0,1)."""
    return ((words(seed, tid, n, first) >> np.uint64(11)).astype(np.float64) + 0.5) / 9007199254740992.0


def normal_bf16(n: int, seed: int, tid: int, std: float) -> np.ndarray:
    """n samples of N(0, std^2) rounded to bf16 (returned as uint16 bit patterns)."""
    out = np.empty(n, np.uint16)
    _lib().hsin_normal_bf16(out.ctypes.data, n, seed, tid, std, 0)
    return out


def grid_bf16(n: int, seed: int, tid: int, scale: float, first: int = 0) -> np.ndarray:
    out = np.empty(n, np.uint16)
    _lib().hsin_grid_bf16(out.ctypes.data, n, seed, tid, scale, first)
    return out


def grid_f32(n: int, seed: int, tid: int, scale: float, first: int = 0) -> np.ndarray:
    out = np.empty(n, np.float32)
    _lib().hsin_grid_f32(out.ctypes.data, n, seed, tid, scale, first)
    return out


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def f32_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bf16 bit patterns (finite inputs)."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32).astype(np.uint64)
    u = u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))
    return (u >> np.uint64(16)).astype(np.uint16)


# ----------------------------------------------------------------------------
# model shapes
# ----------------------------------------------------------------------------
@dataclass
class ModelShape:
    name: str
    arch: int
    L: int
    d: int
    V: int
    # Mamba-2 branch (parallel hybrids)
    H: int = 0
    P: int = 0
    N: int = 0
    # softmax attention
    qh: int = 0
    kvh: int = 0
    hd: int = 0
    ff: int = 0
    # Gated DeltaNet (sequential hybrids)
    gh: int = 0
    gdk: int = 0
    gdv: int = 0
    conv_w: int = 4
    rope_theta: float = 10000.0
    eps: float = 1e-5
    # workload
    batch: int = 1
    prompt_len: int = 64
    gen_tokens: int = 32
    ks: tuple = (2,)

    @property
    def d_inner(self) -> int:
        return self.H * self.P

    @property
    def convd(self) -> int:
        if self.arch == ARCH_PARALLEL:
            return self.H * self.P + 2 * self.N
        return 2 * self.gh * self.gdk + self.gh * self.gdv

    def layer_type(self, l: int) -> int:
        if self.arch == ARCH_PARALLEL:
            return LAYER_PAR
        return LAYER_ATT if l % 4 == 3 else LAYER_GDN

    def replace(self, **kw) -> "ModelShape":
        d = asdict(self)
        d.update(kw)
        return ModelShape(**d)


CONFIGS = {
    # the five workloads (tiny, 0.5B-class, 3B-class, sequential, batch-64 long context)
    "cfg1_tiny": ModelShape("cfg1_tiny", ARCH_PARALLEL, L=2, d=256, V=4096, H=8, P=64, N=64,
                            qh=4, kvh=2, hd=64, ff=1024, batch=1, prompt_len=64, gen_tokens=32, ks=(2,)),
    "cfg2_0p5b": ModelShape("cfg2_0p5b", ARCH_PARALLEL, L=36, d=1024, V=32768, H=32, P=64, N=128,
                            qh=8, kvh=2, hd=128, ff=4096, batch=1, prompt_len=512, gen_tokens=256,
                            ks=(1, 2, 4, 8)),
    "cfg3_3b": ModelShape("cfg3_3b", ARCH_PARALLEL, L=32, d=2560, V=65536, H=80, P=64, N=256,
                          qh=20, kvh=4, hd=128, ff=10240, batch=1, prompt_len=2048, gen_tokens=256,
                          ks=(2, 4)),
    "cfg4_seq": ModelShape("cfg4_seq", ARCH_SEQUENTIAL, L=24, d=1024, V=32768, qh=8, kvh=2, hd=128,
                           ff=4096, gh=16, gdk=64, gdv=64, batch=1, prompt_len=1024, gen_tokens=128,
                           ks=(2, 4)),
    "cfg5_b64": ModelShape("cfg5_b64", ARCH_PARALLEL, L=36, d=1024, V=32768, H=32, P=64, N=128,
                           qh=8, kvh=2, hd=128, ff=4096, batch=64, prompt_len=16384, gen_tokens=128,
                           ks=(4,)),
    # small sequential stack used by tests only (8 layers, attention at l % 4 == 3)
    "test_seq": ModelShape("test_seq", ARCH_SEQUENTIAL, L=8, d=256, V=2048, qh=4, kvh=2, hd=64,
                           ff=512, gh=4, gdk=64, gdv=64, batch=1, prompt_len=48, gen_tokens=24, ks=(2, 4)),
}


# ----------------------------------------------------------------------------
# weight blob
# ----------------------------------------------------------------------------
# tensor ids inside a layer (also the order of storage); id 7 is the gated-norm
# weight of the Mamba branch or the per-head output-norm weight of a DeltaNet layer
T_NORM1, T_W_IN, T_CONV_W, T_CONV_B, T_A_LOG, T_D, T_DT_BIAS, T_GNORM, T_W_OUT, T_W_O, T_NORM2, T_W_GU, T_W_DOWN = range(13)
N_LAYER_TENSORS = 13
G_EMBED, G_LM_HEAD, G_FINAL_NORM = range(3)
ALIGN = 256


def in_proj_rows(s: ModelShape, ltype: int) -> int:
    if ltype == LAYER_PAR:
        return 2 * s.d_inner + 2 * s.N + s.H + (s.qh + 2 * s.kvh) * s.hd
    if ltype == LAYER_GDN:
        return 2 * s.gh * s.gdk + 2 * s.gh * s.gdv + 2 * s.gh
    return (s.qh + 2 * s.kvh) * s.hd


def layer_tensors(s: ModelShape, ltype: int):
    """(tensor id, shape, dtype) for every tensor a layer of this type stores, in storage order."""
    bf, f4 = "bf16", "f32"
    t = [(T_NORM1, (s.d,), f4), (T_W_IN, (in_proj_rows(s, ltype), s.d), bf)]
    if ltype == LAYER_PAR:
        t += [(T_CONV_W, (s.convd, s.conv_w), f4), (T_CONV_B, (s.convd,), f4),
              (T_A_LOG, (s.H,), f4), (T_D, (s.H,), f4), (T_DT_BIAS, (s.H,), f4),
              (T_GNORM, (s.d_inner,), f4), (T_W_OUT, (s.d, s.d_inner), bf), (T_W_O, (s.d, s.qh * s.hd), bf)]
    elif ltype == LAYER_GDN:
        t += [(T_CONV_W, (s.convd, s.conv_w), f4), (T_CONV_B, (s.convd,), f4),
              (T_GNORM, (s.gdv,), f4), (T_W_OUT, (s.d, s.gh * s.gdv), bf)]
    else:
        t += [(T_W_O, (s.d, s.qh * s.hd), bf)]
    t += [(T_NORM2, (s.d,), f4), (T_W_GU, (2 * s.ff, s.d), bf), (T_W_DOWN, (s.d, s.ff), bf)]
    return t


def _nbytes(shape, dtype):
    return int(np.prod(shape)) * (2 if dtype == "bf16" else 4)


def _up(x):
    return (x + ALIGN - 1) // ALIGN * ALIGN


def blob_layout(s: ModelShape):
    """Byte offset of every tensor: {(layer, tid): (offset, shape, dtype)}, layer = -1 for globals.
    Returns (table, total_bytes)."""
    table = {}
    off = 0
    for tid, shape, dt in [(G_EMBED, (s.V, s.d), "bf16"), (G_LM_HEAD, (s.V, s.d), "bf16"),
                           (G_FINAL_NORM, (s.d,), "f32")]:
        table[(-1, tid)] = (off, shape, dt)
        off = _up(off + _nbytes(shape, dt))
    for l in range(s.L):
        for tid, shape, dt in layer_tensors(s, s.layer_type(l)):
            table[(l, tid)] = (off, shape, dt)
            off = _up(off + _nbytes(shape, dt))
    return table, off


def make_weights(s: ModelShape, seed: int = 0, small_init: str = "unit"):
    """Random-init weight blob.

    Matrices and embeddings ~ N(0, 0.02) rounded to bf16; A_log ~ U(log 1, log 16);
    dt_bias = softplus^-1(exp(U(log 1e-3, log 1e-1))); conv taps ~ U(-0.5, 0.5).
    small_init = "unit": norm weights 1, D 1, conv bias 0.
    small_init = "jitter": those get a +-10 % / +-0.1 seeded perturbation so that a
    parity test notices a kernel that drops one of them.
    Returns (blob uint8[total], table)."""
    table, total = blob_layout(s)
    blob = np.zeros(total, np.uint8)
    lib = _lib()
    for (l, tid), (off, shape, dt) in table.items():
        n = int(np.prod(shape))
        rid = (l + 1) * 64 + tid
        view = blob[off:off + _nbytes(shape, dt)]
        if dt == "bf16":
            lib.hsin_normal_bf16(view.ctypes.data, n, seed, rid, 0.02, 0)
            continue
        u = uniform01(seed, rid, n)
        jit = small_init == "jitter"
        if l >= 0 and tid == T_A_LOG:
            v = math.log(1.0) + u * (math.log(16.0) - math.log(1.0))
        elif l >= 0 and tid == T_DT_BIAS:
            dt0 = np.exp(math.log(1e-3) + u * (math.log(1e-1) - math.log(1e-3)))
            v = dt0 + np.log(-np.expm1(-dt0))
        elif l >= 0 and tid == T_CONV_W:
            v = u - 0.5
        elif l >= 0 and tid == T_CONV_B:
            v = (u - 0.5) * 0.2 if jit else np.zeros(n)
        else:  # norm weights and D
            v = 1.0 + (u - 0.5) * 0.2 if jit else np.ones(n)
        view.view(np.float32)[:] = v.astype(np.float32)
    return blob, table


def tensor_view(blob: np.ndarray, table, layer: int, tid: int) -> np.ndarray:
    off, shape, dt = table[(layer, tid)]
    raw = blob[off:off + _nbytes(shape, dt)]
    return raw.view(np.uint16 if dt == "bf16" else np.float32).reshape(shape)


# ----------------------------------------------------------------------------
# prompts, accept pattern, injected contexts
# ----------------------------------------------------------------------------
def make_prompt(V: int, length: int, seed: int = 1, seq: int = 0) -> np.ndarray:
    """i.i.d. uniform token ids in [0, V)."""
    return (words(seed, seq, length) % np.uint64(V)).astype(np.int32)


def context_lengths(batch: int, lo: int, hi: int, seed: int = 1) -> np.ndarray:
    """Per-sequence context lengths, uniform in [lo, hi]."""
    w = words(seed, 1 << 20, batch)
    return (lo + (w % np.uint64(hi - lo + 1))).astype(np.int32)


ALPHA_NUM = int(0.68 * (1 << 53))


def forced_accept(k: int, n_rounds: int, seq: int = 0, seed: int = 2, alpha_num: int = ALPHA_NUM) -> np.ndarray:
    """Truncated-geometric accept lengths: position i of round r succeeds iff
    word(seed, seq, r*64+i) >> 11 < alpha_num; n = leading successes, capped at k."""
    out = np.empty(n_rounds, np.int32)
    if k == 0:
        out[:] = 0
        return out
    w = words(seed, seq, n_rounds * 64).reshape(n_rounds, 64)[:, :k] >> np.uint64(11)
    ok = w < np.uint64(alpha_num)
    fail = ~ok
    first_fail = np.where(fail.any(axis=1), fail.argmax(axis=1), k)
    out[:] = first_fail
    return out


DRAFT_SKIP, DRAFT_LINEAR, DRAFT_FULL = 0, 1, 2


def draft_plan(s: ModelShape, kind: str = "component") -> np.ndarray:
    """Per-layer draft plans (data only).  "component": the recurrent pathway of every layer (attention suppressed);
    "layerskip33": every third layer skipped as a whole (l % 3 == 1), the others kept whole - uniformly selected
    layers, about 33 %; "full": every layer whole (the draft is the full model: every draft is accepted)."""
    if kind == "component":
        return np.full(s.L, DRAFT_LINEAR, np.int32)
    if kind == "full":
        return np.full(s.L, DRAFT_FULL, np.int32)
    if kind == "layerskip33":
        return np.array([DRAFT_SKIP if l % 3 == 1 else DRAFT_FULL for l in range(s.L)], np.int32)
    raise ValueError(kind)


def expected_tokens_per_round(alpha: float, k: int) -> float:
    return (1.0 - alpha ** (k + 1)) / (1.0 - alpha)


# stream ids of injected contexts: (kind, layer, seq) -> tid
def _ctx_tid(kind: int, layer: int, seq: int) -> int:
    return (1 << 30) + (kind << 26) + (layer << 16) + seq


CTX_K, CTX_V, CTX_SSM, CTX_CONV, CTX_GDN = range(5)


def injected_kv(s: ModelShape, layer: int, seq: int, length: int, which: int, seed: int = 3) -> np.ndarray:
    """bf16 bits [length, kvh, hd] of synthetic K (which=CTX_K) or V rows for one layer and sequence."""
    n = length * s.kvh * s.hd
    return grid_bf16(n, seed, _ctx_tid(which, layer, seq), 1.0).reshape(length, s.kvh, s.hd)


def injected_state(s: ModelShape, layer: int, seq: int, kind: int, seed: int = 3) -> np.ndarray:
    """float32 synthetic recurrent state of one layer and sequence.
    CTX_SSM: [H, P, N]; CTX_CONV: [conv_w-1, convd]; CTX_GDN: [gh, gdv, gdk]."""
    if kind == CTX_SSM:
        shape, scale = (s.H, s.P, s.N), 0.5
    elif kind == CTX_CONV:
        shape, scale = (s.conv_w - 1, s.convd), 1.0
    else:
        shape, scale = (s.gh, s.gdv, s.gdk), 0.5
    return grid_f32(int(np.prod(shape)), seed, _ctx_tid(kind, layer, seq), scale).reshape(shape)
