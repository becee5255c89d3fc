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
    if flags & env["hs"].HS_FLAG_LITERAL_DRAFT:
        model.set_literal_draft(True)
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


@pytest.mark.parametrize("flags", [2, 3])
@pytest.mark.parametrize("name,k", [("cfg1_tiny", 4), ("cfg1_tiny", 8), ("test_seq", 2), ("test_seq", 4)])
def test_rollback_by_replay_matches_oracle(env, name, k, flags):
    # HS_FLAG_REPLAY: verify keeps an update log instead of per-position snapshots and the accepted updates are
    # replayed into the committed state; every round's state, conv window, KV rows, tokens and accept length must be
    # the oracle's (whose rollback == recompute property is pinned on the CPU), with and without graph replay
    s, eng, model, seqs = setup(env, name, [hi.CONFIGS[name].prompt_len], max_k=8, cap=512, flags=flags)
    rep = env["harness"].run_rounds(eng, seqs, s, k, 8)
    forced = [hi.forced_accept(k, 8, seq=7)]
    rep = env["harness"].run_rounds(eng, seqs, s, k, 8, forced=forced, rep=rep)      # every accept length 0..k occurs
    print(name, k, flags, rep)
    assert len(rep.n_hist) >= 2 and eng.device_status() == 0


def test_rollback_by_replay_ragged_batch_and_async(env):
    lens = [40, 23, 57]
    s, eng, model, seqs = setup(env, "cfg1_tiny", lens, max_k=4, cap=512, flags=3)
    forced = [hi.forced_accept(4, 10, seq=b) for b in range(3)]
    rep = env["harness"].run_rounds(eng, seqs, s, 4, 10, forced=forced)
    assert len(rep.n_hist) >= 3
    env["harness"].run_rounds_async(eng, seqs, [2, 0, 4, 0, 0, 2, 4, 1] * 2)
    env["harness"].compare_states(eng, seqs, s, kv_rows=None)
    assert eng.device_status() == 0
    # the snapshot buffer of this mode is one state per sequence plus the log: smaller than k + 1 snapshots
    hs = env["hs"]
    a = hs.query_sizes(hs.make_config(s, 3, 4, 512, flags=0)).snap
    b = hs.query_sizes(hs.make_config(s, 3, 4, 512, flags=2)).snap
    assert b < a / 3


@pytest.mark.parametrize("flags", [0, 1])
@pytest.mark.parametrize("kind", ["layerskip33", "full"])
@pytest.mark.parametrize("name", ["cfg1_tiny", "test_seq"])
def test_draft_plans_match_oracle(env, name, kind, flags):
    # per-layer draft plans (layers skipped whole / kept whole, Sec. 4.2): candidates, accept lengths, tokens and states
    # against the oracle running the same plan; with every layer kept whole the draft is the full model and every
    # draft is accepted.  The draft's attention writes scratch KV rows beyond kv_len that verification overwrites.
    s, eng, model, seqs = setup(env, name, [hi.CONFIGS[name].prompt_len], max_k=4, cap=512, flags=flags)
    plan = hi.draft_plan(s, kind)
    eng.set_draft_plan(plan); model.set_draft_plan(plan)
    rep = env["harness"].run_rounds(eng, seqs, s, 4, 6)
    rep = env["harness"].run_rounds(eng, seqs, s, 2, 4, rep=rep)
    print(name, kind, flags, rep)
    if kind == "full":
        assert set(rep.n_hist) == {2, 4}, rep.n_hist
    with pytest.raises(env["hs"].HsError):
        eng.set_draft_plan([3] * s.L)
    eng.set_draft_plan(None); model.set_draft_plan(None)
    env["harness"].run_rounds(eng, seqs, s, 2, 3, rep=rep)
    assert eng.device_status() == 0


@pytest.mark.parametrize("flags", [0, 1])
@pytest.mark.parametrize("name,tau", [("cfg1_tiny", 0.01), ("cfg1_tiny", 0.05), ("test_seq", 0.02)])
def test_speculative_sampling_matches_oracle(env, name, tau, flags):
    # temperature > 0 (Eq. 6): draft draws, accept tests and the correction / bonus draw happen on the device with the
    # uniforms the oracle gets; tokens, accept lengths and states must agree wherever the oracle's margins are wide
    s, eng, model, seqs = setup(env, name, [hi.CONFIGS[name].prompt_len, 19], max_k=4, cap=512, flags=flags)
    rep, full = env["harness"].run_rounds_sampled(eng, seqs, s, 4, 10, tau)
    rep, full2 = env["harness"].run_rounds_sampled(eng, seqs, s, 2, 6, tau, seed=12, rep=rep)
    print(name, tau, flags, rep, "rounds compared in full:", full + full2)
    assert full + full2 >= 8                    # most rounds are decided by the device and compared as such
    assert eng.device_status() == 0
    # back to greedy: the next rounds are the oracle's greedy rounds
    env["harness"].run_rounds(eng, seqs, s, 2, 3)


def test_sampling_with_the_full_model_as_draft_accepts_everything(env):
    # P_S = P_H when the draft plan keeps every layer whole: Eq. 6 accepts with probability 1
    s, eng, model, seqs = setup(env, "cfg1_tiny", [33], max_k=4, cap=256, flags=1)
    plan = hi.draft_plan(s, "full")
    eng.set_draft_plan(plan); model.set_draft_plan(plan)
    rep, full = env["harness"].run_rounds_sampled(eng, seqs, s, 4, 6, 0.02)
    assert set(rep.n_hist) == {4}, rep.n_hist
    with pytest.raises(env["hs"].HsError):           # no uniforms given
        eng.set_sampling(0.5)


def test_prefill_ragged_batch_matches_oracle(env):
    # prompts of different lengths go through prefill together, chunk by chunk; shorter ones drop out of later passes
    lens = [9, 31, 30, 30, 5]
    s, eng, model, seqs = setup(env, "cfg1_tiny", lens, max_k=4, cap=128)
    env["harness"].compare_states(eng, seqs, s, kv_rows=None)
    s, eng, model, seqs = setup(env, "test_seq", [17, 17, 4], max_k=8, cap=128, flags=1)
    env["harness"].compare_states(eng, seqs, s, kv_rows=None)
    assert eng.device_status() == 0


@pytest.mark.parametrize("flags", [4, 5, 7])
@pytest.mark.parametrize("name", ["cfg1_tiny", "test_seq"])
def test_literal_draft_state_matches_oracle(env, name, flags):
    # HS_FLAG_LITERAL_DRAFT: the draft model keeps its own attention-free state over the whole history (Eq. 4 / Eq. 5
    # read literally): prefill runs it over the prompt, a round advances it over the consumed tokens.  Candidates,
    # accept lengths, tokens, the full model's state AND the draft model's own state and conv window follow the oracle,
    # with real acceptance, forced accept lengths (every n from 0 to k), k = 0 rounds, ragged prompts, graphs, replay.
    lens = [hi.CONFIGS[name].prompt_len, 7, 22]
    s, eng, model, seqs = setup(env, name, lens, max_k=4, cap=512, flags=flags)
    env["harness"].compare_states(eng, seqs, s)
    rep = env["harness"].run_rounds(eng, seqs, s, 4, 5)
    forced = [hi.forced_accept(4, 8, seq=30 + b) for b in range(3)]
    rep = env["harness"].run_rounds(eng, seqs, s, 4, 8, forced=forced, rep=rep)
    rep = env["harness"].run_rounds(eng, seqs, s, 0, 2, rep=rep)
    rep = env["harness"].run_rounds(eng, seqs, s, 2, 3, rep=rep)
    print(name, flags, rep)
    assert len(rep.n_hist) >= 3 and eng.device_status() == 0
    env["harness"].run_rounds_async(eng, seqs, [2, 0, 4, 1, 0, 2])
    env["harness"].compare_states(eng, seqs, s, kv_rows=None)
    with pytest.raises(env["hs"].HsError):           # this reading goes with attention-free draft plans only
        eng.set_draft_plan(hi.draft_plan(s, "full"))


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


def test_order_and_argument_errors_leave_the_state_alone(env):
    # a second verify (or a draft) between verify and accept_rollback would start from snapshots that already hold
    # the verified positions: refused; a forced accept length beyond k and token ids outside the vocabulary are
    # refused on the host before anything is enqueued
    s, eng, model, seqs = setup(env, "cfg1_tiny", [16], max_k=2, cap=128)
    hs = env["hs"]
    L = hs.lib()
    eng.draft(2); eng.verify(2)
    for call in (lambda: eng.verify(2), lambda: eng.draft(2), lambda: eng.round_host(2)):
        with pytest.raises(hs.HsError) as e:
            call()
        assert e.value.code == -4
    eng.accept_rollback(readback=True)
    for o in seqs:
        o.round(2)
    with pytest.raises(hs.HsError) as e:
        eng.round_host(2, forced_n=[3])
    assert e.value.code == -1
    with pytest.raises(hs.HsError) as e:
        eng.round_host(2, forced_n=[1], forced_next=[s.V])
    assert e.value.code == -1
    bad = np.array([5, s.V, 7], np.int32); lens = np.array([3], np.int32)
    assert L.hs_prefill(eng.h, bad.ctypes.data, lens.ctypes.data, 1) == -1
    bad[1] = -2
    assert L.hs_prefill(eng.h, bad.ctypes.data, lens.ctypes.data, 1) == -1
    # nothing of the refused calls ran: the next round still agrees with the oracle
    env["harness"].run_rounds(eng, seqs, s, 2, 2)
    assert eng.device_status() == 0


def test_out_of_range_candidate_is_not_used_as_an_address(env):
    # candidates supplied on the device cannot be checked by the host: the gather clamps them and reports
    s, eng, model, seqs = setup(env, "cfg1_tiny", [16], max_k=2, cap=128)
    torch, hs = env["torch"], env["hs"]
    cand = torch.tensor([[3, 2 ** 30, -5]], dtype=torch.int32, device=eng.device)
    eng.verify(2, cand)
    eng.accept_rollback(readback=True)
    assert eng.device_status() == -7
    eng.clear_status()
    assert eng.device_status() == 0 and eng.check_guards()


@pytest.mark.parametrize("flags", [0, 1])
@pytest.mark.parametrize("name", ["cfg1_tiny", "test_seq"])
def test_rounds_back_to_back_without_host_reads(env, name, flags):
    # 24 rounds, k = 0 (verify directly after accept) mixed with k = 2 and 4, the library's own acceptance, and no
    # host read or synchronisation between rounds: the control words (kv_len, snapshot slot) written by the accept
    # kernel of one round are read by the first mixer / attention kernels of the next as early as the launch mode
    # lets them start.  Afterwards every consumed token (all KV rows), the recurrent state, the conv window,
    # kv_len and the pending token must be the oracle's.
    s, eng, model, seqs = setup(env, name, [hi.CONFIGS[name].prompt_len], max_k=4, cap=512, flags=flags)
    ks = [2, 0, 0, 2, 4, 0, 2, 2, 0, 4, 0, 0] * 2
    env["harness"].run_rounds_async(eng, seqs, ks)
    env["harness"].compare_states(eng, seqs, s, kv_rows=None)
    assert eng.get_context(0)[0] >= hi.CONFIGS[name].prompt_len + len(ks)      # at least one token per round
    assert eng.device_status() == 0


def test_bounded_wait_runs_out_and_reports(env):
    # every wait on a copy barrier gives up after a fixed number of polls; here nothing ever completes the barrier:
    # the kernel must end by itself, the status word must say HS_ERR_TIMEOUT, and the handle must stay usable
    s, eng, model, seqs = setup(env, "cfg1_tiny", [16], max_k=2, cap=128)
    eng.selftest_wait_timeout(2000)
    assert eng.device_status() == -6
    eng.clear_status()
    assert eng.device_status() == 0
    env["harness"].run_rounds(eng, seqs, s, 2, 2)
    assert eng.device_status() == 0


@pytest.mark.parametrize("name", ["cfg1_tiny", "test_seq"])
def test_control_words_out_of_range_are_not_used_as_addresses(env, name):
    # The kernels that turn a device control word into an address check it first.  A self-test hook plants a bad word
    # for one of two sequences (no host-side validation; the sequence is chosen so that even an unchecked access would
    # stay inside the buffer): the blocks of that sequence must touch neither cache nor state,
    # the status word must name the error, the guard bytes behind every buffer must be intact, and after a reset the
    # handle must reproduce the oracle again.
    k, cap = 4, 64
    lens = [24, 17]
    s, eng, model, seqs = setup(env, name, lens, max_k=k, cap=cap)
    for seq, word, value, want in ((0, eng.CTRL_KV_LEN, cap - 2, -3),   # the k + 1 new rows would not fit: HS_ERR_CAPACITY
                                   (1, eng.CTRL_KV_LEN, -5, -7),        # a negative cache length: HS_ERR_DEVICE
                                   (0, eng.CTRL_SLOT, k + 3, -7)):      # a snapshot slot beyond the k + 1 that exist
        eng.poke_control(seq, word, value)
        eng.draft(k)
        eng.verify(k)
        assert eng.device_status() == want, (word, value)
        assert eng.check_guards()
        eng.accept_rollback()
        eng.reset()
        assert eng.device_status() == 0
        prompts = [hi.make_prompt(s.V, n, seq=b) for b, n in enumerate(lens)]
        seqs = []
        for p in prompts:
            q = model.new_seq()
            q.prefill(p)
            seqs.append(q)
        eng.prefill(prompts)
        env["harness"].run_rounds(eng, seqs, s, k, 2)
        assert eng.device_status() == 0
    with pytest.raises(RuntimeError):
        eng.poke_control(0, 7, 0)
    with pytest.raises(RuntimeError):
        eng.poke_control(2, eng.CTRL_SLOT, 0)

