"""Parity of the CUDA library with the CPU oracle at the full sizes of the five workloads, in the launch
configuration the benchmark times (CUDA graphs on).  Contexts too long to prefill on the CPU are injected:
the same seeded recurrent state, conv window and KV rows are given to both sides (prefill itself is compared
on the small configurations).  Every comparison is round by round: candidates, argmax, accept length,
emitted tokens bit-exact where the oracle's margin exceeds 1e-2, logits within 2e-2, states within 1e-3."""
import numpy as np
import pytest

import hs_inputs as hi

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    import oracle
    from paper_2605_01106_b200 import build, binding
    build.build()
    import harness
    return dict(torch=torch, oracle=oracle, hs=binding, harness=harness)


_W = {}


def make(env, name, batch, max_k, cap, checked, ctx_lens, small_init="jitter", flags=0):
    s = hi.CONFIGS[name]
    if (name, small_init) not in _W:
        _W.clear()                                     # one large blob at a time
        _W[(name, small_init)] = hi.make_weights(s, 0, small_init)
    blob, table = _W[(name, small_init)]
    eng = env["hs"].Engine(s, blob, max_batch=batch, max_k=max_k, kv_capacity=cap, flags=env["hs"].HS_FLAG_GRAPHS | flags)
    model = env["oracle"].Model(s, blob, table, cap)
    seqs = []
    for b in range(batch):
        q = model.new_seq() if b in checked else None
        pending = int(hi.make_prompt(s.V, 1, seq=1000 + b)[0])
        env["harness"].inject_context(eng, q, s, b, int(ctx_lens[b]), pending)
        seqs.append(q)
    eng.set_batch(batch)
    return s, eng, model, seqs


def test_cfg2_full_size_all_k(env):
    s, eng, model, seqs = make(env, "cfg2_0p5b", 1, 8, 640, {0}, [512])
    rep = None
    for k, rounds in ((1, 2), (2, 3), (4, 2), (8, 1)):
        forced = [hi.forced_accept(k, rounds, seq=k)]
        rep = env["harness"].run_rounds(eng, seqs, s, k, rounds, forced=forced, rep=rep)
    print(rep)
    assert eng.device_status() == 0 and rep.rounds == 8


def test_cfg2_full_size_real_acceptance(env):
    s, eng, model, seqs = make(env, "cfg2_0p5b", 1, 2, 600, {0}, [512])
    rep = env["harness"].run_rounds(eng, seqs, s, 2, 3)
    print(rep)
    assert eng.device_status() == 0


@pytest.mark.parametrize("name,ctx", [("cfg2_0p5b", 512), ("cfg4_seq", 1024)])
def test_full_size_rollback_by_replay(env, name, ctx):
    s, eng, model, seqs = make(env, name, 2, 4, ctx + 100, {0, 1}, [ctx, ctx - 37], flags=env["hs"].HS_FLAG_REPLAY)
    rep = env["harness"].run_rounds(eng, seqs, s, 2, 2, forced=[[0, 2], [1, 0]])
    rep = env["harness"].run_rounds(eng, seqs, s, 4, 2, forced=[[4, 1], [2, 3]], rep=rep)
    print(rep)
    assert eng.device_status() == 0 and rep.rounds == 4


def test_cfg2_attention_geometries(env):
    # the split of the KV cache over CTAs (keys per tile x tiles per CTA) is a launch-time choice: every
    # setting, including several tiles per CTA (running softmax), ragged last tiles and more than one
    # cluster per sequence, must reproduce the oracle on two sequences of different context length
    s, eng, model, seqs = make(env, "cfg2_0p5b", 2, 4, 1024, {0, 1}, [700, 333])
    with pytest.raises(RuntimeError):
        eng.set_attn_geometry(40, 1)
    rep = None
    for chunk, tiles in ((32, 2), (32, 4), (48, 2), (64, 2), (64, 8), (96, 1), (128, 2), (128, 1), (0, 0)):
        seqs = [model.new_seq(), model.new_seq()]
        for b, n in enumerate((700, 333)):
            env["harness"].inject_context(eng, seqs[b], s, b, n, 11 + b)
        eng.set_batch(2)
        eng.set_attn_geometry(chunk, tiles)
        rep = env["harness"].run_rounds(eng, seqs, s, 4, 1, forced=[[2], [4]], rep=rep)
        assert eng.device_status() == 0, (chunk, tiles)
    print(rep)
    assert rep.rounds == 9


def test_cfg2_projection_kernel_choices(env):
    # which kernel a projection runs on is a matter of its activation-row count (CUDA cores up to 3 rows, the
    # warp-level tensor path, tcgen05 from a threshold on): every choice must reproduce the oracle.  Threshold 17 keeps
    # 6 and 10 rows on the warp-level path (one and two groups of eight rows), 2 sends even the two-row draft steps
    # through tcgen05 (16- and 32-row tiles, K split over clusters), 0 restores the automatic threshold.
    s, eng, model, seqs = make(env, "cfg2_0p5b", 2, 8, 700, {0, 1}, [512, 77])
    with pytest.raises(RuntimeError):
        eng.set_option(eng.OPT_TC_MIN_ROWS, 18)
    rep = None
    try:
        for thr, ks in ((17, (2, 4)), (2, (0, 2, 8)), (0, (1, 4))):
            eng.set_option(eng.OPT_TC_MIN_ROWS, thr)
            for k in ks:
                forced = [hi.forced_accept(k, 1, seq=thr + k + b) for b in range(2)]
                rep = env["harness"].run_rounds(eng, seqs, s, k, 1, forced=forced, rep=rep)
                assert eng.device_status() == 0, (thr, k)
    finally:
        eng.set_option(eng.OPT_TC_MIN_ROWS, 0)          # the choice is process-wide
    print(rep)
    assert rep.rounds == 7


def test_streaming_attention_edge_cases(env):
    # the streaming form (128-key tiles walked with two buffers, warp-local running softmax, ranges merged by the last
    # CTA to arrive) on the small sequential stack, where attention is a launch of its own: contexts that end exactly on
    # a tile boundary (the new rows then form a ninth key group), one key short of and one past it, a single short
    # range, several tiles per CTA, one and two 16-row query tiles (k = 4: 10 rows, k = 8: 18 rows)
    lens = [1152, 1151, 1153, 640, 77, 1279]
    s, eng, model, seqs = make(env, "test_seq", len(lens), 8, 1500, set(range(len(lens))), lens)
    rep = None
    for tiles, k in ((-1, 4), (-2, 8), (-4, 4), (-16, 8), (-3, 1)):
        eng.set_attn_geometry(128, tiles)
        forced = [hi.forced_accept(k, 1, seq=40 + b - tiles) for b in range(len(lens))]
        rep = env["harness"].run_rounds(eng, seqs, s, k, 1, forced=forced, rep=rep)
        assert eng.device_status() == 0, (tiles, k)
    with pytest.raises(RuntimeError):
        eng.set_attn_geometry(64, -2)
    print(rep)
    assert rep.rounds == 5


def test_streaming_attention_batched_parallel_hybrid(env):
    # a batch large enough that the verify attention of the parallel hybrid runs as its own launch in the streaming form
    # (chosen automatically); three sequences carry their context on both sides, the others run beside them
    lens = [1152, 1151, 640] + [1000 + 7 * b for b in range(21)]
    s, eng, model, seqs = make(env, "cfg1_tiny", len(lens), 4, 1400, {0, 1, 2}, lens)
    forced = [hi.forced_accept(4, 2, seq=b) for b in range(len(lens))]
    rep = env["harness"].run_rounds(eng, seqs, s, 4, 2, forced=forced)
    forced = [hi.forced_accept(2, 2, seq=50 + b) for b in range(len(lens))]
    rep = env["harness"].run_rounds(eng, seqs, s, 2, 2, forced=forced, rep=rep)
    print(rep)
    assert eng.device_status() == 0 and rep.rounds == 4


def test_cfg4_sequential_full_size(env):
    s, eng, model, seqs = make(env, "cfg4_seq", 1, 4, 1100, {0}, [1024])
    rep = env["harness"].run_rounds(eng, seqs, s, 2, 2, forced=[hi.forced_accept(2, 2, seq=1)])
    rep = env["harness"].run_rounds(eng, seqs, s, 4, 1, forced=[hi.forced_accept(4, 1, seq=2)], rep=rep)
    print(rep)
    assert eng.device_status() == 0


def test_cfg3_3b_batch1(env):
    # perturbed small parameters (norm weights, D, conv bias): a kernel that dropped one of them at this shape
    # (N = 256, 80 heads, 20 query heads) would be noticed
    s, eng, model, seqs = make(env, "cfg3_3b", 1, 4, 2100, {0}, [2048])
    rep = env["harness"].run_rounds(eng, seqs, s, 2, 1, forced=[[1]])
    rep = env["harness"].run_rounds(eng, seqs, s, 4, 1, forced=[[2]], rep=rep)
    print(rep)
    assert eng.device_status() == 0


def test_cfg3_3b_batch8_two_checked(env):
    s, eng, model, seqs = make(env, "cfg3_3b", 8, 4, 2100, {0, 5}, [2048] * 8)
    forced = [hi.forced_accept(4, 1, seq=b) for b in range(8)]
    rep = env["harness"].run_rounds(eng, seqs, s, 4, 1, forced=forced)
    forced = [hi.forced_accept(2, 1, seq=20 + b) for b in range(8)]
    rep = env["harness"].run_rounds(eng, seqs, s, 2, 1, forced=forced, rep=rep)
    print(rep)
    assert eng.device_status() == 0


def test_cfg5_batch64_ragged_sampled(env):
    # 64 sequences with contexts uniform in [4096, 16384]; four of them carry a full seeded context on both
    # sides and are compared, the others run beside them with their own accept pattern (ragged rollback)
    s = hi.CONFIGS["cfg5_b64"]
    lens = hi.context_lengths(64, 4096, 16384)
    checked = {0, 17, 38, 63}
    s, eng, model, seqs = make(env, "cfg5_b64", 64, 4, 16384 + 32, checked, lens)
    forced = [hi.forced_accept(4, 2, seq=b) for b in range(64)]
    rep = env["harness"].run_rounds(eng, seqs, s, 4, 2, forced=forced)
    print(rep, sorted(set(int(x) for x in lens))[:3])
    for b in range(64):
        kv, _ = eng.get_context(b)
        assert kv == lens[b] + int((np.array(forced[b]) + 1).sum())
    assert len(rep.n_hist) >= 2 and eng.device_status() == 0


def test_cfg5_batch64_two_sequences_128_tokens(env):
    # the long run of the batch-64 workload: 64 ragged sequences decode 128 tokens each (k = 4, seeded accept
    # pattern, about 48 rounds); two of them carry their full context on the CPU side as well and are compared
    # round by round over the whole generation, states every eighth round
    s = hi.CONFIGS["cfg5_b64"]
    lens = hi.context_lengths(64, 4096, 16384)
    rounds = 48
    s, eng, model, seqs = make(env, "cfg5_b64", 64, 4, 16384 + 5 * (rounds + 2), {5, 41}, lens)
    forced = [hi.forced_accept(4, rounds, seq=100 + b) for b in range(64)]
    rep = env["harness"].run_rounds(eng, seqs, s, 4, rounds, forced=forced, check_states_every=8)
    print(rep)
    assert rep.tokens >= 2 * 110 and eng.device_status() == 0
    for b in (5, 41):
        kv, _ = eng.get_context(b)
        assert kv == lens[b] + int((np.array(forced[b]) + 1).sum())
