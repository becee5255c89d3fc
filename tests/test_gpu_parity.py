"""Parity of the CUDA library (through the C ABI) with the CPU oracle on a B200."""
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


_WEIGHTS = {}


def weights(name, small_init="jitter"):
    key = (name, small_init)
    if key not in _WEIGHTS:
        _WEIGHTS[key] = hi.make_weights(hi.CONFIGS[name], 0, small_init)
    return _WEIGHTS[key]


def setup(env, name, prompt_lens, max_k, cap, flags=0, seed_seq0=0):
    s = hi.CONFIGS[name]
    blob, table = weights(name)
    eng = env["hs"].Engine(s, blob, max_batch=len(prompt_lens), max_k=max_k, kv_capacity=cap, flags=flags)
    model = env["oracle"].Model(s, blob, table, cap)
    prompts = [hi.make_prompt(s.V, n, seq=seed_seq0 + b) for b, n in enumerate(prompt_lens)]
    seqs = []
    for p in prompts:
        q = model.new_seq()
        q.prefill(p)
        seqs.append(q)
    eng.prefill(prompts)
    return s, eng, model, seqs


@pytest.mark.parametrize("name", ["cfg1_tiny", "test_seq"])
def test_prefill_matches_oracle(env, name):
    s, eng, model, seqs = setup(env, name, [hi.CONFIGS[name].prompt_len], max_k=4, cap=256)
    env["harness"].compare_states(eng, seqs, s)
    assert eng.device_status() == 0


@pytest.mark.parametrize("name", ["cfg1_tiny", "test_seq"])
@pytest.mark.parametrize("k", [0, 1, 2, 4, 8])
def test_rounds_real_acceptance(env, name, k):
    s, eng, model, seqs = setup(env, name, [hi.CONFIGS[name].prompt_len], max_k=8, cap=512)
    rounds = 32 if k == 2 else 10
    rep = env["harness"].run_rounds(eng, seqs, s, k, rounds)
    print(name, k, rep)
    assert rep.tokens >= rounds
    assert eng.device_status() == 0


def test_cfg1_workload_32_tokens_lossless(env):
    # config 1 as specified: 64-token prompt, k = 2, 32 generated tokens; output == plain greedy of the oracle
    s, eng, model, seqs = setup(env, "cfg1_tiny", [64], max_k=2, cap=256)
    ref_seq = model.new_seq()
    ref_seq.prefill(hi.make_prompt(s.V, 64))
    ref = ref_seq.greedy(48)
    out = [eng.get_context(0)[1]]
    hist = {}
    listed = 0
    while len(out) < 32:
        eng.draft(2); eng.verify(2)
        _, g, margin = eng.get_round(2)
        n, em = eng.accept_rollback(readback=True)
        hist[int(n[0])] = hist.get(int(n[0]), 0) + 1
        out += list(em[0, : n[0] + 1])
    assert np.array_equal(np.array(out[:32]), ref[:32]), (out, ref)
    assert len(hist) >= 2, hist        # both rejections and full accepts occur


@pytest.mark.parametrize("name,batch", [("cfg1_tiny", 3), ("test_seq", 2)])
def test_batched_ragged_forced_pattern(env, name, batch):
    lens = [40, 23, 57][:batch]
    s, eng, model, seqs = setup(env, name, lens, max_k=4, cap=256)
    forced = [hi.forced_accept(4, 12, seq=b) for b in range(batch)]
    rep = env["harness"].run_rounds(eng, seqs, s, 4, 12, forced=forced)
    print(rep)
    assert len(rep.n_hist) >= 3
    assert eng.device_status() == 0


def test_graph_replay_matches(env):
    s, eng, model, seqs = setup(env, "cfg1_tiny", [64], max_k=4, cap=256, flags=env["hs"].HS_FLAG_GRAPHS)
    rep = env["harness"].run_rounds(eng, seqs, s, 4, 12)
    rep = env["harness"].run_rounds(eng, seqs, s, 2, 6, rep=rep)
    print(rep)
    assert eng.launch_count() > 0 and eng.device_status() == 0


def test_draft_leaves_cache_and_committed_state_untouched(env):
    s, eng, model, seqs = setup(env, "cfg1_tiny", [32], max_k=4, cap=128)
    hs = env["hs"]
    before = [eng.export_state(l, 0, hs.STATE_SSM) for l in range(s.L)]
    kb = eng.export_state(0, 0, hs.STATE_K, rows=128)
    ctx = eng.get_context(0)
    eng.draft(4)
    assert eng.get_context(0)[0] == ctx[0]
    for l in range(s.L):
        assert np.array_equal(eng.export_state(l, 0, hs.STATE_SSM), before[l])
    assert np.array_equal(eng.export_state(0, 0, hs.STATE_K, rows=128), kb)


def test_call_order_and_capacity_errors(env):
    s, eng, model, seqs = setup(env, "cfg1_tiny", [16], max_k=2, cap=24)
    hs = env["hs"]
    with pytest.raises(hs.HsError) as e:
        eng.accept_rollback()
    assert e.value.code == -4
    with pytest.raises(hs.HsError) as e:
        eng.verify(2)
    assert e.value.code == -4
    with pytest.raises(hs.HsError) as e:
        eng.draft(3)
    assert e.value.code == -1
    eng.round(2); eng.round(2)                     # kv_len now <= 22
    with pytest.raises(hs.HsError) as e:
        for _ in range(3):
            eng.round(2)
    assert e.value.code == -3
    assert eng.device_status() == 0                # the host refused before any kernel overran the cache
