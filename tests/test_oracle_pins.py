"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU).

Each test names the passage or the textbook fact it checks.  A mistake in the
oracle (dropped term, wrong sign, transposed operand, wrong index) must fail at
least one of these before the oracle is trusted as the yardstick of the CUDA path.
"""
import itertools
import os

import numpy as np
import pytest

import hs_inputs as hi
import oracle

RNG = np.random.default_rng(1234)
GOLD = os.path.join(os.path.dirname(__file__), "golden")


def bf16_round(x):
    return hi.bf16_to_f32(hi.f32_to_bf16(np.asarray(x, np.float32))).astype(np.float64)


# --------------------------------------------------------------------------- components
def test_matvec_rmsnorm_textbook():
    W = hi.normal_bf16(37 * 96, 5, 1, 0.5).reshape(37, 96)
    x = RNG.standard_normal(96)
    np.testing.assert_allclose(oracle.matvec_bf16(W, x), hi.bf16_to_f32(W).astype(np.float64) @ x, rtol=1e-12, atol=1e-12)
    w = RNG.uniform(0.5, 1.5, 96).astype(np.float32)
    got = oracle.rmsnorm(x, w, 1e-5)
    np.testing.assert_allclose(got, x / np.sqrt((x * x).mean() + 1e-5) * w, rtol=1e-12)
    # unit weight, eps -> 0: output has unit RMS and is invariant to the input's scale
    one = np.ones(96, np.float32)
    assert abs(np.sqrt((oracle.rmsnorm(x, one, 0.0) ** 2).mean()) - 1.0) < 1e-12
    np.testing.assert_allclose(oracle.rmsnorm(7.5 * x, one, 0.0), oracle.rmsnorm(x, one, 0.0), rtol=1e-12)


def test_conv_equals_direct_causal_convolution():
    # the rolling-window step applied to a sequence == causal convolution with zero left padding
    T, taps, bias = 11, RNG.uniform(-0.5, 0.5, 4).astype(np.float32), 0.3
    x = RNG.standard_normal(T)
    win, got = np.zeros(3), []
    for t in range(T):
        o, win = oracle.conv_step(win, x[t], taps, bias)
        got.append(o)
    xp = np.concatenate([np.zeros(3), x])
    want = [bias + sum(float(taps[j]) * xp[t + j] for j in range(4)) for t in range(T)]
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-12)
    # the newest input is weighted by the last tap (np.convolve flips the kernel)
    np.testing.assert_allclose(got, bias + np.convolve(x, taps[::-1].astype(np.float64))[:T], rtol=1e-12, atol=1e-12)
    np.testing.assert_array_equal(win, x[-3:])


def test_ssm_closed_form_constant_inputs():
    # constant dt, x, B from S_0 = 0: S_t = dt x(x)B (1 - a^t)/(1 - a), a = exp(dt A)
    P, N, dt, A = 4, 6, 0.3, -1.7
    x, B, C = RNG.standard_normal(P), RNG.standard_normal(N), RNG.standard_normal(N)
    S = np.zeros((P, N))
    a = np.exp(dt * A)
    for t in range(1, 8):
        S, y = oracle.ssm_step(S, dt, A, 0.0, x, B, C)
        np.testing.assert_allclose(S, dt * np.outer(x, B) * (1 - a ** t) / (1 - a), rtol=1e-12)
        np.testing.assert_allclose(y, S @ C, rtol=1e-12)


def test_ssm_no_decay_is_linear_attention_sum_and_C_picks_column():
    # A -> 0-, dt = 1: S_t = sum_j x_j (x) B_j ; C = e_n reads column n ; D adds D x
    P, N, T = 3, 5, 6
    xs, Bs = RNG.standard_normal((T, P)), RNG.standard_normal((T, N))
    S = np.zeros((P, N))
    for t in range(T):
        e = np.zeros(N); e[t % N] = 1.0
        S, y = oracle.ssm_step(S, 1.0, -0.0, 2.0, xs[t], Bs[t], e)
        want = sum(np.outer(xs[j], Bs[j]) for j in range(t + 1))
        np.testing.assert_allclose(S, want, rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(y, want[:, t % N] + 2.0 * xs[t], rtol=1e-12, atol=1e-14)


def test_ssm_decay_only():
    # x = 0: the state only decays by exp(dt A); the state layout is [P][N] (y_p uses row p)
    S0 = RNG.standard_normal((2, 3))
    S, y = oracle.ssm_step(S0, 0.5, -2.0, 0.0, np.zeros(2), np.ones(3), np.array([1.0, 0, 0]))
    np.testing.assert_allclose(S, np.exp(-1.0) * S0, rtol=1e-14)
    np.testing.assert_allclose(y, np.exp(-1.0) * S0[:, 0], rtol=1e-14)


@pytest.mark.parametrize("T", [1, 2, 3, 5, 9])
def test_chunked_ssd_equals_recurrence(T):
    # one-chunk SSD form == T applications of the recurrence (and T = 1 is the recurrence itself)
    P, N, A, D = 4, 4, -0.9, 0.7
    S0 = RNG.standard_normal((P, N))
    dt = RNG.uniform(0.01, 0.5, T)
    x, B, C = RNG.standard_normal((T, P)), RNG.standard_normal((T, N)), RNG.standard_normal((T, N))
    y, snaps = oracle.ssd_chunk(S0, dt, A, D, x, B, C)
    S = S0
    for i in range(T):
        S, yi = oracle.ssm_step(S, dt[i], A, D, x[i], B[i], C[i])
        np.testing.assert_allclose(snaps[i], S, rtol=1e-5, atol=1e-12)
        np.testing.assert_allclose(y[i], yi, rtol=1e-5, atol=1e-12)


def test_gdn_associative_memory():
    # alpha = beta = 1, orthonormal keys: after writing (k_i, v_i), S k_j = v_j exactly; rewriting overwrites
    dk, dv, r = 8, 5, 4
    Q, _ = np.linalg.qr(RNG.standard_normal((dk, dk)))
    keys, vals = Q[:, :r].T, RNG.standard_normal((r, dv))
    S = np.zeros((dv, dk))
    for i in range(r):
        S, o = oracle.gdn_step(S, 1.0, 1.0, keys[i], keys[i], vals[i])
        np.testing.assert_allclose(o, vals[i] / np.sqrt(dk), rtol=1e-10, atol=1e-12)   # o = S q / sqrt(dk), q = k_i
    for j in range(r):
        np.testing.assert_allclose(S @ keys[j], vals[j], rtol=1e-10, atol=1e-12)
    new = RNG.standard_normal(dv)
    S, _ = oracle.gdn_step(S, 1.0, 1.0, keys[0], keys[1], new)
    np.testing.assert_allclose(S @ keys[1], new, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(S @ keys[2], vals[2], rtol=1e-10, atol=1e-12)


def test_gdn_gates():
    dk, dv = 6, 3
    S0 = RNG.standard_normal((dv, dk))
    q, k, v = RNG.standard_normal(dk), RNG.standard_normal(dk), RNG.standard_normal(dv)
    S, _ = oracle.gdn_step(S0, 0.3, 0.0, q, k, v)           # beta = 0: decay only
    np.testing.assert_allclose(S, 0.3 * S0, rtol=1e-14)
    S, _ = oracle.gdn_step(S0, 0.0, 0.8, q, k, v)           # alpha = 0: S = beta v k^T
    np.testing.assert_allclose(S, 0.8 * np.outer(v, k), rtol=1e-14)
    # general step against the matrix form S' (I - beta k k^T) + beta v k^T
    S, o = oracle.gdn_step(S0, 0.9, 0.4, q, k, v)
    want = 0.9 * S0 @ (np.eye(dk) - 0.4 * np.outer(k, k)) + 0.4 * np.outer(v, k)
    np.testing.assert_allclose(S, want, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(o, want @ q / np.sqrt(dk), rtol=1e-12, atol=1e-14)


def test_rope_properties():
    hd = 16
    x, y = RNG.standard_normal(hd), RNG.standard_normal(hd)
    np.testing.assert_array_equal(oracle.rope(x, 0), x)                    # position 0 is the identity
    d0 = oracle.rope(x, 7) @ oracle.rope(y, 3)
    np.testing.assert_allclose(oracle.rope(x, 107) @ oracle.rope(y, 103), d0, rtol=1e-9)   # depends on m - n only
    np.testing.assert_allclose(np.linalg.norm(oracle.rope(x, 12345)), np.linalg.norm(x), rtol=1e-12)
    # pair (i, i + hd/2) turns by pos * theta^(-2i/hd): check pair 0 (angle = pos) and pair 3
    e = np.zeros(hd); e[0] = 1.0
    r = oracle.rope(e, 2)
    np.testing.assert_allclose([r[0], r[hd // 2]], [np.cos(2.0), np.sin(2.0)], rtol=1e-12)
    e = np.zeros(hd); e[3] = 1.0
    r = oracle.rope(e, 5)
    ang = 5 * 10000.0 ** (-2 * 3 / hd)
    np.testing.assert_allclose([r[3], r[3 + hd // 2]], [np.cos(ang), np.sin(ang)], rtol=1e-12)


def test_attention_special_cases_and_gqa_brute_force():
    qh, kvh, hd, n = 4, 2, 8, 13
    q = RNG.standard_normal((qh, hd))
    K = hi.f32_to_bf16(RNG.standard_normal((n, kvh, hd)).astype(np.float32))
    V = hi.f32_to_bf16(RNG.standard_normal((n, kvh, hd)).astype(np.float32))
    Kf, Vf = hi.bf16_to_f32(K).astype(np.float64), hi.bf16_to_f32(V).astype(np.float64)
    # single key: output = its value row
    o = oracle.attention(q, K[:1], V[:1], qh, kvh, hd)
    for h in range(qh):
        np.testing.assert_allclose(o[h], Vf[0, h // 2], rtol=1e-14)
    # all keys equal: uniform weights -> mean of V
    Keq = np.repeat(K[:1], n, axis=0)
    o = oracle.attention(q, Keq, V, qh, kvh, hd)
    for h in range(qh):
        np.testing.assert_allclose(o[h], Vf[:, h // 2].mean(axis=0), rtol=1e-12)
    # grouped-query result == per-q-head softmax attention with kv heads repeated
    o = oracle.attention(q, K, V, qh, kvh, hd)
    for h in range(qh):
        s = Kf[:, h // (qh // kvh)] @ q[h] / np.sqrt(hd)
        p = np.exp(s - s.max()); p /= p.sum()
        np.testing.assert_allclose(o[h], p @ Vf[:, h // (qh // kvh)], rtol=1e-12, atol=1e-14)


def test_argmax_tiebreak_and_margin():
    lg = np.array([0.1, 0.7, 0.7, -1.0, 0.5])
    i, m = oracle.argmax_margin(lg)
    assert i == 1 and m == 0.0                       # lowest index wins a tie, margin 0
    i, m = oracle.argmax_margin(np.array([0.25, -3.0, 1.5, 1.0]))
    assert i == 2 and m == 0.5
    # decisions are taken on float32-rounded logits: a difference below float32 resolution is a tie
    i, m = oracle.argmax_margin(np.array([1.0, 1.0 + 1e-12]))
    assert i == 0 and m == 0.0


@pytest.mark.parametrize("k", [1, 2, 3, 5, 8])
def test_accept_len_brute_force(k):
    # all match patterns in {0,1}^k: n = number of leading matches (tokens up to the first rejection, Sec. 3.3)
    for pat in itertools.product([0, 1], repeat=k):
        g = np.arange(10, 10 + k, dtype=np.int32)
        d = np.where(np.array(pat) == 1, g, g + 1000).astype(np.int32)
        want = k if all(pat) else pat.index(0)
        assert oracle.accept_len(d, g) == want


# --------------------------------------------------------------------------- seeded inputs
def test_word_stream_numpy_equals_c():
    import ctypes
    out = np.empty(1000, np.uint64)
    hi._lib().hsin_words(out.ctypes.data, 1000, 7, 99, 5)
    np.testing.assert_array_equal(out, hi.words(7, 99, 1000, first=5))


def test_weight_statistics():
    w = hi.bf16_to_f32(hi.normal_bf16(400000, 0, 3, 0.02)).astype(np.float64)
    assert abs(w.mean()) < 2e-4 and abs(w.std() - 0.02) < 2e-4
    assert abs((np.abs(w) < 0.02).mean() - 0.6827) < 5e-3


def _golden_eq1():
    rows = [l.split() for l in open(os.path.join(GOLD, "eq1_tokens_per_round.txt")) if not l.startswith("#")]
    return {int(k): float(v) for k, v in rows}


def test_forced_accept_pattern_matches_eq1_numerator():
    # mean emitted tokens per round of the truncated-geometric pattern -> (1 - a^(k+1))/(1 - a) (Eq. 1)
    gold = _golden_eq1()
    for k, want in gold.items():
        assert abs(hi.expected_tokens_per_round(0.68, k) - want) < 1e-6
        n = hi.forced_accept(k, 200000, seq=3)
        assert n.min() >= 0 and n.max() <= k
        assert abs((n + 1).mean() - want) < 0.012, (k, (n + 1).mean(), want)


# --------------------------------------------------------------------------- model-level pins
@pytest.fixture(scope="module")
def tiny():
    s = hi.CONFIGS["cfg1_tiny"]
    blob, table = hi.make_weights(s, 0, "jitter")
    return s, blob, table


@pytest.fixture(scope="module")
def tseq():
    s = hi.CONFIGS["test_seq"]
    blob, table = hi.make_weights(s, 0, "jitter")
    return s, blob, table


def _decode_spec(model, prompt, k, n_tokens, forced=None):
    q = model.new_seq(); q.prefill(prompt)
    out, ns, r = [q.pending], [], 0
    while len(out) < n_tokens:
        res = q.round(k, forced_n=-1 if forced is None else int(forced[r]))
        out += list(res["emitted"]); ns.append(res["n"]); r += 1
    return np.array(out), ns, q      # may overshoot n_tokens by up to k


@pytest.mark.parametrize("cfg", ["tiny", "tseq"])
@pytest.mark.parametrize("k", [0, 1, 2, 4, 8])
def test_speculative_equals_plain_greedy(cfg, k, request):
    # lossless under greedy decoding (Sec. 3.3): token for token identical, bit-exact in the oracle;
    # k = 0 is ordinary autoregressive decoding
    s, blob, table = request.getfixturevalue(cfg)
    m = oracle.Model(s, blob, table, 160)
    prompt = hi.make_prompt(s.V, s.prompt_len)
    a = m.new_seq(); a.prefill(prompt)
    ref = a.greedy(s.gen_tokens)
    out, ns, _ = _decode_spec(m, prompt, k, s.gen_tokens)
    np.testing.assert_array_equal(out[: s.gen_tokens], ref)
    if k >= 2 and cfg == "tiny":
        assert min(ns) < k and max(ns) == k      # both a rejection and a full accept occur


@pytest.mark.parametrize("cfg", ["tiny", "tseq"])
def test_rollback_equals_recompute(cfg, request):
    # after rounds, committed state and KV rows == those of re-prefilling the accepted prefix from scratch
    s, blob, table = request.getfixturevalue(cfg)
    m = oracle.Model(s, blob, table, 160)
    prompt = hi.make_prompt(s.V, s.prompt_len)
    out, ns, q = _decode_spec(m, prompt, 4, 20)
    q2 = m.new_seq(); q2.reset()
    consumed = np.concatenate([prompt, out])[: q.len]
    q2.prefill(consumed)
    assert q2.len == q.len and q2.pending == q.pending
    for a, b in ((q.ssm(), q2.ssm()), (q.gdn(), q2.gdn()), (q.conv(), q2.conv())):
        if a is not None:
            np.testing.assert_array_equal(a, b)
    np.testing.assert_array_equal(q.k()[:, : q.len], q2.k()[:, : q.len])
    np.testing.assert_array_equal(q.v()[:, : q.len], q2.v()[:, : q.len])


def test_forced_accept_keeps_state_consistent(tiny):
    # with a forced accept length the emitted drafts are kept; the state is the full model over what was emitted
    s, blob, table = tiny
    m = oracle.Model(s, blob, table, 200)
    prompt = hi.make_prompt(s.V, 32)
    forced = hi.forced_accept(4, 16)
    out, ns, q = _decode_spec(m, prompt, 4, 24, forced=forced)
    assert ns == list(forced[: len(ns)])
    q2 = m.new_seq()
    q2.prefill(np.concatenate([prompt, out])[: q.len])
    np.testing.assert_array_equal(q.ssm(), q2.ssm())
    np.testing.assert_array_equal(q.conv(), q2.conv())
    assert q.pending == q2.pending


def test_draft_equals_full_with_attention_output_zeroed(tiny):
    # Eq. 4: the parallel draft is the full model with the attention output zeroed (here: W_o = 0)
    s, blob, table = tiny
    z = blob.copy()
    for l in range(s.L):
        hi.tensor_view(z, table, l, hi.T_W_O)[:] = 0
    m, mz = oracle.Model(s, blob, table, 64), oracle.Model(s, z, table, 64)
    a, b = m.new_seq(), mz.new_seq()
    toks = hi.make_prompt(s.V, 12, seq=5)
    k_before = a.k().copy()
    for t in toks:
        np.testing.assert_array_equal(a.step(t, mode=1), b.step(t, mode=0))
    # the draft touched neither the cache nor the length; the full model's attention does change the logits
    assert a.len == 0 and np.array_equal(a.k(), k_before)
    c = m.new_seq()
    full = [c.step(t, mode=0) for t in toks]
    assert np.abs(full[-1] - b.step(int(toks[0]), mode=0)).max() > 0


def test_sequential_draft_equals_stack_without_attention_layers(tseq):
    # Eq. 5: attention layers are the identity in the draft (whole layer bypassed by the residual)
    s, blob, table = tseq
    m = oracle.Model(s, blob, table, 64)
    lin = [l for l in range(s.L) if s.layer_type(l) == hi.LAYER_GDN]
    m_lin = oracle.Model(s, blob, table, 64, layer_ids=lin)
    a, b = m.new_seq(), m_lin.new_seq()
    for t in hi.make_prompt(s.V, 10, seq=6):
        np.testing.assert_array_equal(a.step(t, mode=1), b.step(t, mode=0))
    assert a.len == 0


def _f(blob, table, l, tid):
    v = hi.tensor_view(blob, table, l, tid)
    return hi.bf16_to_f32(v).astype(np.float64) if v.dtype == np.uint16 else v.astype(np.float64)


def _rms(x, w, eps):
    return x / np.sqrt((x * x).mean() + eps) * w


def test_block_composition_special_cases(tiny):
    # with the mixers silenced (W_out = W_o = 0) one layer is the textbook pre-norm SwiGLU residual block;
    # with W_down = 0 as well the stack is the identity and logits = W_lm rmsnorm(E[token])
    s, blob, table = tiny
    s1 = s.replace(L=1)
    b1 = blob.copy()
    hi.tensor_view(b1, table, 0, hi.T_W_OUT)[:] = 0
    hi.tensor_view(b1, table, 0, hi.T_W_O)[:] = 0
    tok = 77
    e = _f(b1, table, -1, hi.G_EMBED)[tok]
    Wlm, wf = _f(b1, table, -1, hi.G_LM_HEAD), _f(b1, table, -1, hi.G_FINAL_NORM)
    gu, Wd, w2 = _f(b1, table, 0, hi.T_W_GU), _f(b1, table, 0, hi.T_W_DOWN), _f(b1, table, 0, hi.T_NORM2)
    u = _rms(e, w2, s.eps)
    g, up = gu[0::2] @ u, gu[1::2] @ u                     # even rows gate, odd rows up
    h = e + Wd @ (g / (1 + np.exp(-g)) * up)
    got = oracle.Model(s1, b1, table, 8).new_seq().step(tok)
    np.testing.assert_allclose(got, Wlm @ _rms(h, wf, s.eps), rtol=1e-10, atol=1e-12)
    hi.tensor_view(b1, table, 0, hi.T_W_DOWN)[:] = 0
    got = oracle.Model(s1, b1, table, 8).new_seq().step(tok)
    np.testing.assert_allclose(got, Wlm @ _rms(e, wf, s.eps), rtol=1e-10, atol=1e-12)


def test_first_token_ssm_branch_closed_form(tiny):
    # first token from zero state, one layer, attention and MLP silenced: conv sees only the newest tap,
    # S_1 = dt x(x)B, y = (B.C) dt x + D x ; checks the in-projection row blocks z | x | B | C | dt
    s, blob, table = tiny
    s1 = s.replace(L=1)
    b1 = blob.copy()
    hi.tensor_view(b1, table, 0, hi.T_W_O)[:] = 0
    hi.tensor_view(b1, table, 0, hi.T_W_DOWN)[:] = 0
    tok, di, N, H, P = 123, s.d_inner, s.N, s.H, s.P
    e = _f(b1, table, -1, hi.G_EMBED)[tok]
    u = _rms(e, _f(b1, table, 0, hi.T_NORM1), s.eps)
    Win = _f(b1, table, 0, hi.T_W_IN)
    z, xbc, dtr = Win[:di] @ u, Win[di:2 * di + 2 * N] @ u, Win[2 * di + 2 * N: 2 * di + 2 * N + H] @ u
    cw, cb = _f(b1, table, 0, hi.T_CONV_W), _f(b1, table, 0, hi.T_CONV_B)
    pre = cb + cw[:, 3] * xbc
    act = pre / (1 + np.exp(-pre))
    x, B, C = act[:di].reshape(H, P), act[di:di + N], act[di + N:]
    dt = np.log1p(np.exp(dtr + _f(b1, table, 0, hi.T_DT_BIAS)))
    D = _f(b1, table, 0, hi.T_D)
    y = ((B @ C) * dt[:, None] * x + D[:, None] * x).reshape(-1)
    g = y * (z / (1 + np.exp(-z)))
    h = e + _f(b1, table, 0, hi.T_W_OUT) @ _rms(g, _f(b1, table, 0, hi.T_GNORM), s.eps)
    want = _f(b1, table, -1, hi.G_LM_HEAD) @ _rms(h, _f(b1, table, -1, hi.G_FINAL_NORM), s.eps)
    q = oracle.Model(s1, b1, table, 8).new_seq()
    np.testing.assert_allclose(q.step(tok, mode=1), want, rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(q.ssm()[0], dt[:, None, None] * x[:, :, None] * B[None, None, :], rtol=1e-10, atol=1e-14)
    np.testing.assert_allclose(q.conv()[0, 2], xbc, rtol=1e-12)            # newest raw input is the last window row
    assert not q.conv()[0, :2].any()


def test_attention_branch_first_two_tokens(tiny):
    # attention only (W_out = W_down = 0), one layer: token 0 attends to itself -> o = v (bf16-rounded);
    # checks q | k | v row blocks, RoPE on the cached key, cache layout [position][kv head][dim]
    s, blob, table = tiny
    s1 = s.replace(L=1)
    b1 = blob.copy()
    hi.tensor_view(b1, table, 0, hi.T_W_OUT)[:] = 0
    hi.tensor_view(b1, table, 0, hi.T_W_DOWN)[:] = 0
    di, N, H = s.d_inner, s.N, s.H
    r0 = 2 * di + 2 * N + H
    Win = _f(b1, table, 0, hi.T_W_IN)
    Wq, Wk, Wv = Win[r0:r0 + s.qh * s.hd], Win[r0 + s.qh * s.hd: r0 + (s.qh + s.kvh) * s.hd], Win[r0 + (s.qh + s.kvh) * s.hd:]
    E, Wo = _f(b1, table, -1, hi.G_EMBED), _f(b1, table, 0, hi.T_W_O)
    Wlm, wf, w1 = _f(b1, table, -1, hi.G_LM_HEAD), _f(b1, table, -1, hi.G_FINAL_NORM), _f(b1, table, 0, hi.T_NORM1)
    q = oracle.Model(s1, b1, table, 8).new_seq()
    t0, t1 = 11, 2222
    u0 = _rms(E[t0], w1, s.eps)
    v0 = bf16_round(Wv @ u0)
    o0 = np.repeat(v0.reshape(s.kvh, s.hd), s.qh // s.kvh, axis=0).reshape(-1)
    np.testing.assert_allclose(q.step(t0), Wlm @ _rms(E[t0] + Wo @ o0, wf, s.eps), rtol=1e-9, atol=1e-11)
    np.testing.assert_array_equal(hi.bf16_to_f32(q.v()[0, 0]).reshape(-1), v0.astype(np.float32))
    # second token: two keys, causal; brute-force softmax with RoPE at positions 0 and 1
    u1 = _rms(E[t1], w1, s.eps)
    k0 = bf16_round(np.concatenate([oracle.rope(r, 0) for r in (Wk @ u0).reshape(s.kvh, s.hd)]))
    k1 = bf16_round(np.concatenate([oracle.rope(r, 1) for r in (Wk @ u1).reshape(s.kvh, s.hd)]))
    v1 = bf16_round(Wv @ u1)
    qq = np.stack([oracle.rope(r, 1) for r in (Wq @ u1).reshape(s.qh, s.hd)])
    o = []
    for h in range(s.qh):
        kh = h // (s.qh // s.kvh)
        sc = np.array([qq[h] @ k0.reshape(s.kvh, s.hd)[kh], qq[h] @ k1.reshape(s.kvh, s.hd)[kh]]) / np.sqrt(s.hd)
        p = np.exp(sc - sc.max()); p /= p.sum()
        o.append(p[0] * v0.reshape(s.kvh, s.hd)[kh] + p[1] * v1.reshape(s.kvh, s.hd)[kh])
    want = Wlm @ _rms(E[t1] + Wo @ np.concatenate(o), wf, s.eps)
    np.testing.assert_allclose(q.step(t1), want, rtol=1e-9, atol=1e-11)


def test_gdn_layer_first_token_closed_form(tseq):
    # one DeltaNet layer from zero state, MLP silenced: S_1 = beta v k^T, o = beta v (k.q)/sqrt(dk)
    s, blob, table = tseq
    s1 = s.replace(L=1)
    b1 = blob.copy()
    hi.tensor_view(b1, table, 0, hi.T_W_DOWN)[:] = 0
    tok, nk, nv, gh, dk, dv = 99, s.gh * s.gdk, s.gh * s.gdv, s.gh, s.gdk, s.gdv
    e = _f(b1, table, -1, hi.G_EMBED)[tok]
    u = _rms(e, _f(b1, table, 0, hi.T_NORM1), s.eps)
    Win = _f(b1, table, 0, hi.T_W_IN)
    raw = Win[:2 * nk + nv] @ u
    z, ga, gb = Win[2 * nk + nv:2 * nk + 2 * nv] @ u, Win[2 * nk + 2 * nv:2 * nk + 2 * nv + gh] @ u, Win[2 * nk + 2 * nv + gh:] @ u
    pre = _f(b1, table, 0, hi.T_CONV_B) + _f(b1, table, 0, hi.T_CONV_W)[:, 3] * raw
    act = pre / (1 + np.exp(-pre))
    qv, kv, vv = act[:nk].reshape(gh, dk), act[nk:2 * nk].reshape(gh, dk), act[2 * nk:].reshape(gh, dv)
    qn = qv / np.sqrt((qv * qv).sum(1, keepdims=True) + 1e-6)
    kn = kv / np.sqrt((kv * kv).sum(1, keepdims=True) + 1e-6)
    beta = 1 / (1 + np.exp(-gb))
    o = beta[:, None] * vv * (kn * qn).sum(1, keepdims=True) / np.sqrt(dk)
    wn = _f(b1, table, 0, hi.T_GNORM)
    o = np.stack([_rms(o[h], wn, s.eps) for h in range(gh)]) * (z / (1 + np.exp(-z))).reshape(gh, dv)
    h1 = e + _f(b1, table, 0, hi.T_W_OUT) @ o.reshape(-1)
    want = _f(b1, table, -1, hi.G_LM_HEAD) @ _rms(h1, _f(b1, table, -1, hi.G_FINAL_NORM), s.eps)
    q = oracle.Model(s1, b1, table, 8).new_seq()
    np.testing.assert_allclose(q.step(tok, mode=1), want, rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(q.gdn()[0], beta[:, None, None] * vv[:, :, None] * kn[:, None, :], rtol=1e-10, atol=1e-14)


def test_second_token_ssm_decay_closed_form(tiny):
    # two tokens through one parallel layer from zero state, attention and MLP silenced.  The second token is the
    # first one whose state update has a non-zero previous state, so it is the one that fixes the decay term of the
    # Mamba-2 recurrence inside the layer: S_2 = exp(dt_2 * (-exp(A_log_h))) S_1 + dt_2 x_2 (x) B_2 per head h -
    # the sign, the exponential and the head index of A_log - and the conv window carrying the first raw input.
    s, blob, table = tiny
    s1 = s.replace(L=1)
    b1 = blob.copy()
    hi.tensor_view(b1, table, 0, hi.T_W_O)[:] = 0
    hi.tensor_view(b1, table, 0, hi.T_W_DOWN)[:] = 0
    di, N, H, P = s.d_inner, s.N, s.H, s.P
    E = _f(b1, table, -1, hi.G_EMBED)
    Win = _f(b1, table, 0, hi.T_W_IN)
    w1, wg = _f(b1, table, 0, hi.T_NORM1), _f(b1, table, 0, hi.T_GNORM)
    cw, cb = _f(b1, table, 0, hi.T_CONV_W), _f(b1, table, 0, hi.T_CONV_B)
    A_log, D, dtb = _f(b1, table, 0, hi.T_A_LOG), _f(b1, table, 0, hi.T_D), _f(b1, table, 0, hi.T_DT_BIAS)
    Wout, Wlm, wf = _f(b1, table, 0, hi.T_W_OUT), _f(b1, table, -1, hi.G_LM_HEAD), _f(b1, table, -1, hi.G_FINAL_NORM)
    assert len(set(np.round(A_log, 6))) == H              # distinct per head: a wrong head index cannot hide
    toks = (123, 3001)
    raws, S, want_logits = [], np.zeros((H, P, N)), None
    for t, tok in enumerate(toks):
        u = _rms(E[tok], w1, s.eps)
        z, xbc, dtr = Win[:di] @ u, Win[di:2 * di + 2 * N] @ u, Win[2 * di + 2 * N: 2 * di + 2 * N + H] @ u
        raws.append(xbc)
        pre = cb + cw[:, 3] * raws[t] + (cw[:, 2] * raws[t - 1] if t >= 1 else 0.0)   # taps 0, 1 still see zeros
        act = pre / (1 + np.exp(-pre))
        x, B, C = act[:di].reshape(H, P), act[di:di + N], act[di + N:]
        dt = np.log1p(np.exp(dtr + dtb))
        decay = np.exp(dt * -np.exp(A_log))                                           # one scalar per head
        S = decay[:, None, None] * S + dt[:, None, None] * x[:, :, None] * B[None, None, :]
        y = (S @ C + D[:, None] * x).reshape(-1)
        g = y * (z / (1 + np.exp(-z)))
        h = E[tok] + Wout @ _rms(g, wg, s.eps)
        want_logits = Wlm @ _rms(h, wf, s.eps)
    q = oracle.Model(s1, b1, table, 8).new_seq()
    q.step(toks[0], mode=1)
    got = q.step(toks[1], mode=1)
    np.testing.assert_allclose(q.ssm()[0], S, rtol=1e-10, atol=1e-14)
    np.testing.assert_allclose(got, want_logits, rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(q.conv()[0, 1:], np.stack(raws), rtol=1e-12)
    # the pin has teeth: the decay moves the state by far more than the tolerance (a dropped or mis-signed A would fail)
    no_decay = S / decay[:, None, None]
    assert np.abs(no_decay - S).max() > 1e-3 * np.abs(S).max()


def test_second_token_gdn_alpha_closed_form(tseq):
    # two tokens through one Gated DeltaNet layer from zero state, MLP silenced.  From a zero state the decay gate
    # alpha never acts; the second token fixes alpha = sigmoid(W_a u) with its own row block of the in-projection:
    # S_2 = alpha_2 S_1 + beta_2 (v_2 - alpha_2 S_1 k_2) k_2^T ,  o_2 = S_2 q_2 / sqrt(d_k)
    s, blob, table = tseq
    s1 = s.replace(L=1)
    b1 = blob.copy()
    hi.tensor_view(b1, table, 0, hi.T_W_DOWN)[:] = 0
    nk, nv, gh, dk, dv = s.gh * s.gdk, s.gh * s.gdv, s.gh, s.gdk, s.gdv
    E = _f(b1, table, -1, hi.G_EMBED)
    Win = _f(b1, table, 0, hi.T_W_IN)
    w1, wn = _f(b1, table, 0, hi.T_NORM1), _f(b1, table, 0, hi.T_GNORM)
    cw, cb = _f(b1, table, 0, hi.T_CONV_W), _f(b1, table, 0, hi.T_CONV_B)
    Wout, Wlm, wf = _f(b1, table, 0, hi.T_W_OUT), _f(b1, table, -1, hi.G_LM_HEAD), _f(b1, table, -1, hi.G_FINAL_NORM)
    toks = (99, 1500)
    raws, S, want_logits, alphas = [], np.zeros((gh, dv, dk)), None, None
    for t, tok in enumerate(toks):
        u = _rms(E[tok], w1, s.eps)
        raw = Win[:2 * nk + nv] @ u
        z = Win[2 * nk + nv:2 * nk + 2 * nv] @ u
        ga = Win[2 * nk + 2 * nv:2 * nk + 2 * nv + gh] @ u          # decay-gate rows come before the beta rows
        gb = Win[2 * nk + 2 * nv + gh:2 * nk + 2 * nv + 2 * gh] @ u
        raws.append(raw)
        pre = cb + cw[:, 3] * raws[t] + (cw[:, 2] * raws[t - 1] if t >= 1 else 0.0)
        act = pre / (1 + np.exp(-pre))
        qv, kv, vv = act[:nk].reshape(gh, dk), act[nk:2 * nk].reshape(gh, dk), act[2 * nk:].reshape(gh, dv)
        qn = qv / np.sqrt((qv * qv).sum(1, keepdims=True) + 1e-6)
        kn = kv / np.sqrt((kv * kv).sum(1, keepdims=True) + 1e-6)
        alphas, beta = 1 / (1 + np.exp(-ga)), 1 / (1 + np.exp(-gb))
        o = np.empty((gh, dv))
        for h in range(gh):
            Sd = alphas[h] * S[h]
            S[h] = Sd + beta[h] * np.outer(vv[h] - Sd @ kn[h], kn[h])
            o[h] = S[h] @ qn[h] / np.sqrt(dk)
        o = np.stack([_rms(o[h], wn, s.eps) for h in range(gh)]) * (z / (1 + np.exp(-z))).reshape(gh, dv)
        h1 = E[tok] + Wout @ o.reshape(-1)
        want_logits = Wlm @ _rms(h1, wf, s.eps)
    q = oracle.Model(s1, b1, table, 8).new_seq()
    q.step(toks[0], mode=1)
    got = q.step(toks[1], mode=1)
    np.testing.assert_allclose(q.gdn()[0], S, rtol=1e-10, atol=1e-14)
    np.testing.assert_allclose(got, want_logits, rtol=1e-9, atol=1e-11)
    # alpha acts visibly: with alpha = 1 (no decay) or with the beta rows used for alpha the state would differ
    assert np.abs(alphas - 1.0).min() > 1e-3 and len(set(np.round(alphas, 6))) == gh


# --------------------------------------------------------------------------- draft strategies (Sec. 4.2)
@pytest.mark.parametrize("cfg", ["tiny", "tseq"])
def test_draft_plans_reduce_to_known_models(cfg, request):
    # a per-layer draft plan generalises the component-aware draft: all layers "recurrent pathway only" IS that draft
    # (Eq. 4 / Eq. 5); all layers whole is the full model; layers skipped as a whole are layers deleted from the stack
    s, blob, table = request.getfixturevalue(cfg)
    toks = hi.make_prompt(s.V, 6, seq=9)
    m, mp = oracle.Model(s, blob, table, 64), oracle.Model(s, blob, table, 64)
    mp.set_draft_plan(hi.draft_plan(s, "component"))
    a, b = m.new_seq(), mp.new_seq()
    for t in toks:
        np.testing.assert_array_equal(a.step(t, mode=1), b.step(t, mode=1))
    # whole layers: the draft step at position 0 equals the full model's first step
    mp.set_draft_plan(hi.draft_plan(s, "full"))
    np.testing.assert_array_equal(mp.new_seq().step(int(toks[0]), mode=1), m.new_seq().step(int(toks[0]), mode=0))
    # skipped layers == a stack without them (every kept layer whole), first token
    plan = hi.draft_plan(s, "layerskip33")
    assert (plan == hi.DRAFT_SKIP).sum() >= s.L // 3 and (plan == hi.DRAFT_FULL).sum() >= 1
    mp.set_draft_plan(plan)
    kept = [l for l in range(s.L) if plan[l] != hi.DRAFT_SKIP]
    m_kept = oracle.Model(s, blob, table, 64, layer_ids=kept)
    np.testing.assert_array_equal(mp.new_seq().step(int(toks[0]), mode=1), m_kept.new_seq().step(int(toks[0]), mode=0))
    mp.set_draft_plan(None)
    np.testing.assert_array_equal(mp.new_seq().step(int(toks[0]), mode=1), m.new_seq().step(int(toks[0]), mode=1))


@pytest.mark.parametrize("cfg", ["tiny", "tseq"])
@pytest.mark.parametrize("kind", ["layerskip33", "full"])
def test_any_draft_plan_is_lossless(cfg, kind, request):
    # whatever the draft proposes, greedy verification emits the full model's own greedy sequence (Sec. 3.3); with the
    # full model as its own draft every draft is accepted (n = k in every round)
    s, blob, table = request.getfixturevalue(cfg)
    m = oracle.Model(s, blob, table, 200)
    prompt = hi.make_prompt(s.V, s.prompt_len)
    ref_seq = m.new_seq(); ref_seq.prefill(prompt)
    ref = ref_seq.greedy(s.gen_tokens)
    m.set_draft_plan(hi.draft_plan(s, kind))
    out, ns, q = _decode_spec(m, prompt, 4, s.gen_tokens)
    np.testing.assert_array_equal(out[: s.gen_tokens], ref)
    if kind == "full":
        assert min(ns) == 4
    # rollback == recompute also holds with drafts that wrote scratch KV rows beyond the committed length
    q2 = m.new_seq(); q2.prefill(np.concatenate([prompt, out])[: q.len])
    np.testing.assert_array_equal(q.k()[:, : q.len], q2.k()[:, : q.len])
    for x, y in ((q.ssm(), q2.ssm()), (q.gdn(), q2.gdn()), (q.conv(), q2.conv())):
        if x is not None:
            np.testing.assert_array_equal(x, y)


# --------------------------------------------------------------------------- speculative sampling (Eq. 6)
def test_softmax_temperature_and_inverse_cdf():
    lg = RNG.standard_normal(9)
    for tau in (0.3, 0.6, 1.0, 2.5):
        p = oracle.softmax_t(lg, tau)
        e = np.exp(lg / tau)
        np.testing.assert_allclose(p, e / e.sum(), rtol=1e-12)
    w = np.array([0.0, 0.2, 0.0, 0.5, 0.3])
    # thresholds inside each positive weight's interval pick it; zero weights are never picked; monotone in u
    for u, want in ((0.0, 1), (0.19, 1), (0.21, 3), (0.69, 3), (0.71, 4), (0.999999, 4)):
        j, m = oracle.sample_cdf(w, u)
        assert j == want
    j, m = oracle.sample_cdf(w, 0.45)
    assert j == 3 and abs(m - 0.25) < 1e-12          # 0.45 is 0.25 away from both boundaries (0.2 and 0.7)
    assert oracle.sample_cdf(np.zeros(4), 0.3)[0] == -1
    # frequencies over a fine grid of u reproduce the weights (weights need not be normalised)
    us = (np.arange(20000) + 0.5) / 20000
    picks = np.array([oracle.sample_cdf(7.0 * w, u)[0] for u in us])
    np.testing.assert_allclose(np.bincount(picks, minlength=5) / us.size, w, atol=1e-4)


def test_speculative_sampling_is_lossless_in_distribution():
    # Eq. 6: a draft x ~ P_S accepted with probability min(1, P_H(x)/P_S(x)) and otherwise replaced by a draw from
    # norm(max(0, P_H - P_S)) is distributed exactly as P_H.  Integrate over a stratified grid of the three uniforms.
    V = 6
    pS = oracle.softmax_t(RNG.standard_normal(V), 0.7)
    pH = oracle.softmax_t(RNG.standard_normal(V), 0.7)
    G = 60
    us = (np.arange(G) + 0.5) / G
    r = oracle.residual(pS, pH)
    np.testing.assert_allclose(r, np.maximum(0.0, pH - pS), rtol=0, atol=0)
    out = np.zeros(V)
    for ud in us:
        x, _ = oracle.sample_cdf(pS, ud)
        acc_frac = np.mean([oracle.spec_accept(pS, pH, x, ua)[0] for ua in us])
        np.testing.assert_allclose(acc_frac, min(1.0, pH[x] / pS[x]), atol=1.0 / G)
        out[x] += acc_frac / G
        res = np.bincount([oracle.sample_cdf(r, uf)[0] for uf in us], minlength=V) / G
        out += (1.0 - acc_frac) / G * res
    np.testing.assert_allclose(out, pH, atol=3.0 / G)
    # identical distributions: every draft is accepted whatever u
    assert all(oracle.spec_accept(pH, pH, x, u)[0] for x in range(V) for u in (0.0, 0.5, 0.999999))


@pytest.mark.parametrize("cfg", ["tiny", "tseq"])
def test_sampled_round_reduces_to_greedy_at_low_temperature(cfg, request):
    # tau -> 0: the draws collapse onto the argmax, so a sampled round emits what the greedy round emits
    s, blob, table = request.getfixturevalue(cfg)
    m = oracle.Model(s, blob, table, 160)
    prompt = hi.make_prompt(s.V, s.prompt_len)
    a, b = m.new_seq(), m.new_seq()
    a.prefill(prompt); b.prefill(prompt)
    for r in range(4):
        u = hi.uniform01(5, 77 + r, 2 * 4 + 1)
        ga = a.round(4)
        gb = b.round_sampled(4, 1e-4, u[:4], u[4:8], u[8])
        np.testing.assert_array_equal(ga["cand"], gb["cand"])
        assert ga["n"] == gb["n"]
        np.testing.assert_array_equal(ga["emitted"], gb["emitted"])
    np.testing.assert_array_equal(a.ssm() if a.ssm() is not None else a.gdn(), b.ssm() if b.ssm() is not None else b.gdn())


def test_sampled_round_state_is_consistent_and_first_token_follows_p_h(tiny):
    # (i) after sampled rounds the state is the full model over the emitted tokens (rollback == recompute);
    # (ii) with the full model as its own draft (plan: every layer whole) P_S = P_H: every draft is accepted
    s, blob, table = tiny
    m = oracle.Model(s, blob, table, 200)
    prompt = hi.make_prompt(s.V, 24)
    q = m.new_seq(); q.prefill(prompt)
    out, ns = [q.pending], []
    # (the random-init model's logits are small, so the temperature that makes P_S and P_H differ visibly is small too)
    for r in range(10):
        u = hi.uniform01(6, r, 9)
        res = q.round_sampled(4, 0.01, u[:4], u[4:8], u[8])
        out += list(res["emitted"]); ns.append(res["n"])
    assert len(set(ns)) >= 3, ns
    q2 = m.new_seq(); q2.prefill(np.concatenate([prompt, out])[: q.len])
    np.testing.assert_array_equal(q.ssm(), q2.ssm())
    np.testing.assert_array_equal(q.k()[:, : q.len], q2.k()[:, : q.len])
    m.set_draft_plan(hi.draft_plan(s, "full"))
    q3 = m.new_seq(); q3.prefill(prompt)
    for r in range(3):
        u = hi.uniform01(6, 100 + r, 9)
        assert q3.round_sampled(4, 0.01, u[:4], u[4:8], u[8])["n"] == 4


# --------------------------------------------------------------------------- whose state the draft starts from
@pytest.mark.parametrize("cfg", ["tiny", "tseq"])
def test_literal_draft_state_is_the_attention_free_models_own_history(cfg, request):
    # Eq. 4 / Eq. 5 read literally: h^S is computed from h^S at every position, so the draft model M_S carries a state
    # of its own.  (i) That state equals the state of a stand-alone attention-free model (W_o = 0 in a parallel hybrid,
    # attention layers deleted in a sequential one) that consumed the same tokens; (ii) the emitted tokens are still the
    # full model's greedy tokens; (iii) the drafts differ from the shared-state reading once there is history.
    s, blob, table = request.getfixturevalue(cfg)
    prompt = hi.make_prompt(s.V, s.prompt_len)
    m = oracle.Model(s, blob, table, 200)
    ref_seq = m.new_seq(); ref_seq.prefill(prompt)
    ref = ref_seq.greedy(s.gen_tokens)
    shared = m.new_seq(); shared.prefill(prompt)
    d_shared = shared.draft_only(4)
    m.set_literal_draft(True)
    out, ns, q = _decode_spec(m, prompt, 4, s.gen_tokens)
    np.testing.assert_array_equal(out[: s.gen_tokens], ref)                       # (ii)
    consumed = np.concatenate([prompt, out])[: q.len]
    if s.arch == hi.ARCH_PARALLEL:
        z = blob.copy()
        for l in range(s.L):
            hi.tensor_view(z, table, l, hi.T_W_O)[:] = 0
        alone = oracle.Model(s, z, table, 200).new_seq()
        for tok in consumed:
            alone.step(int(tok), mode=0)
        rec_alone, conv_alone = alone.ssm(), alone.conv()
    else:
        lin = [l for l in range(s.L) if s.layer_type(l) == hi.LAYER_GDN]
        alone = oracle.Model(s, blob, table, 200, layer_ids=lin).new_seq()
        for tok in consumed:
            alone.step(int(tok), mode=0)
        rec_alone, conv_alone = alone.gdn(), alone.conv()
    rec, conv = q.draft_state()
    if s.arch == hi.ARCH_SEQUENTIAL:
        rec, conv = rec[lin], conv[lin]
    np.testing.assert_array_equal(rec, rec_alone)                                  # (i)
    np.testing.assert_array_equal(conv, conv_alone)
    lit = m.new_seq(); lit.prefill(prompt)
    d_lit = lit.draft_only(4)
    full_state = q.ssm() if s.arch == hi.ARCH_PARALLEL else q.gdn()[lin]
    assert np.abs(full_state - rec).max() > 1e-6 if s.arch == hi.ARCH_PARALLEL else True   # (iii) two different states
    m.set_literal_draft(False)
    assert d_shared.shape == d_lit.shape
