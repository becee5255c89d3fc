"""Round-by-round comparison of the CUDA library with the CPU oracle on the same seeded inputs.

Tolerances (those the workload definition states): token ids, accept lengths and KV/state indices bit-exact wherever the
oracle's top-2 logit margin exceeds 1e-2 (narrower positions are listed, and the GPU is re-synchronised to
the oracle there); logits within 2e-2 absolute; recurrent states within 1e-3 of the state's magnitude.
"""
from __future__ import annotations

import numpy as np

import hs_inputs as hi
import oracle
from paper_2605_01106_b200 import binding as hs

MARGIN = 1e-2
LOGIT_TOL = 2e-2
STATE_TOL = 1e-3


class Report:
    def __init__(self):
        self.listed = []          # (round, seq, phase, position, margin)
        self.n_hist = {}
        self.max_logit_err = 0.0
        self.max_state_err = 0.0
        self.rounds = 0
        self.tokens = 0

    def __repr__(self):
        return "Report(rounds=%d tokens=%d listed=%d n_hist=%s max_logit_err=%.2e max_state_err=%.2e)" % (
            self.rounds, self.tokens, len(self.listed), dict(sorted(self.n_hist.items())), self.max_logit_err,
            self.max_state_err)


def compare_states(eng, seqs, shape, rep=None, kv_rows=None):
    """Committed recurrent state, conv window and KV rows of every sequence against the oracle (and, with the literal
    draft state, the draft model's own committed state and window)."""
    worst = 0.0
    literal = bool(eng.cfg.flags & hs.HS_FLAG_LITERAL_DRAFT)
    for b, o in enumerate(seqs):
        if o is None:
            continue
        kv_len, pending = eng.get_context(b)
        assert kv_len == o.len, ("kv_len", b, kv_len, o.len)
        assert pending == o.pending, ("pending", b, pending, o.pending)
        ssm, gdn, conv = o.ssm(), o.gdn(), o.conv()
        for l in range(shape.L):
            t = shape.layer_type(l)
            if t != hi.LAYER_ATT:
                want = ssm[l] if t == hi.LAYER_PAR else gdn[l]      # the oracle indexes its arrays by layer
                got = eng.export_state(l, b, hs.STATE_SSM if t == hi.LAYER_PAR else hs.STATE_GDN)
                err = np.abs(got - want).max() / max(np.abs(want).max(), 1e-30)
                assert err <= STATE_TOL, ("state", l, b, err)
                worst = max(worst, err)
                gotc = eng.export_state(l, b, hs.STATE_CONV)
                errc = np.abs(gotc - conv[l]).max() / max(np.abs(conv[l]).max(), 1e-30)
                assert errc <= STATE_TOL, ("conv", l, b, errc)
                if literal:
                    drec, dconv = o.draft_state()
                    gotd = eng.export_state(l, b, hs.STATE_DRAFT)
                    errd = np.abs(gotd - drec[l]).max() / max(np.abs(drec[l]).max(), 1e-30)
                    assert errd <= STATE_TOL, ("draft model's own state", l, b, errd)
                    gotdc = eng.export_state(l, b, hs.STATE_DRAFT_CONV)
                    errdc = np.abs(gotdc - dconv[l]).max() / max(np.abs(dconv[l]).max(), 1e-30)
                    assert errdc <= STATE_TOL, ("draft model's own conv window", l, b, errdc)
                    worst = max(worst, errd)
        n = o.len if kv_rows is None else min(kv_rows, o.len)
        for l in range(shape.L):
            if shape.layer_type(l) == hi.LAYER_GDN or n == 0:
                continue
            for kind, ref in ((hs.STATE_K, o.k()), (hs.STATE_V, o.v())):
                got = hi.bf16_to_f32(eng.export_state(l, b, kind, rows=o.len)[-n:]).astype(np.float64)
                want = hi.bf16_to_f32(ref[l, o.len - n:o.len]).astype(np.float64)
                # bf16 rows: equal up to one rounding step of the larger magnitude
                assert (np.abs(got - want) <= np.abs(want) * 2.0 ** -7 + 1e-3).all(), ("kv", l, b, kind)
                # most rows are bit-identical; a value flips to the neighbouring bf16 only when it sits within the
                # arithmetic difference (about 1e-4 relative: fp32 activations enter the tensor-core projections
                # as bf16 head + remainder) of a rounding boundary
                assert (got == want).mean() > 0.75, ("kv exact fraction", l, b, kind, (got == want).mean())
    # nothing was written behind any of the buffers the library was given
    assert eng.check_guards(), "guard bytes behind a library buffer were overwritten"
    if rep is not None:
        rep.max_state_err = max(rep.max_state_err, worst)
    return worst


def run_rounds_async(eng, seqs, ks):
    """Rounds with the library's own acceptance and NO host read between them: every call is only enqueued, so
    consecutive passes follow each other on the device as closely as the launch mode allows.  ks: draft length
    of each round (0 = plain autoregressive step).  The oracle sequences take the same rounds; the caller compares
    afterwards (compare_states with kv_rows=None covers kv_len, pending, recurrent state and every KV row, i.e.
    every consumed token)."""
    for k in ks:
        eng.draft(k)
        eng.verify(k)
        eng.accept_rollback(readback=False)
    emitted = []
    for o in seqs:
        toks = []
        for k in ks:
            toks += list(o.round(k)["emitted"])
        emitted.append(toks)
    return emitted


def run_rounds(eng, seqs, shape, k, rounds, forced=None, rep=None, check_states_every=1, check_logits=True,
               torch=None):
    """seqs: oracle sequences, one per active GPU sequence, already holding the same context; an entry may be
    None for a sequence that runs on the GPU without being compared (then `forced` is required).
    forced: None (real acceptance) or int array [batch][rounds] of forced accept lengths."""
    import torch as _torch
    torch = torch or _torch
    rep = rep or Report()
    B, T, V = len(seqs), k + 1, shape.V
    dev = eng.device
    for r in range(rounds):
        # ---- oracle: draft (with logits, for the margins), then the whole round on those candidates
        ora = []
        for b, o in enumerate(seqs):
            if o is None:
                assert forced is not None
                ora.append(None)
                continue
            if k > 0:
                d, dlg = o.draft_only(k, want_logits=True)
                dm = np.array([oracle.argmax_margin(dlg[i])[1] for i in range(k)])
            else:
                d, dm = np.zeros(0, np.int32), np.zeros(0)
            cand = np.concatenate([[o.pending], d]).astype(np.int32)
            fn = -1 if forced is None else int(forced[b][r])
            res = o.round(k, cand_in=cand, forced_n=fn, want_logits=check_logits)
            res["draft_margin"] = dm
            ora.append(res)
        # ---- GPU draft; candidates must agree where the oracle's draft margin is wide
        eng.draft(k)
        eng.last_k = k
        # get_round reads cand before verify: phase is 'drafted'
        gc, _, _ = eng.get_round(k)
        resync = False
        for b in range(B):
            if ora[b] is None:
                continue
            for i in range(T):
                if gc[b, i] != ora[b]["cand"][i]:
                    m = ora[b]["draft_margin"][i - 1] if i > 0 else np.inf
                    assert m <= MARGIN, ("draft token differs at a wide margin", r, b, i, m, gc[b], ora[b]["cand"])
                    rep.listed.append((r, b, "draft", i, float(m)))
                    resync = True
                    break
        cand_all = np.stack([o["cand"] if o is not None else gc[b] for b, o in enumerate(ora)]).astype(np.int32)
        eng.verify(k, torch.from_numpy(cand_all).to(dev) if resync else None)
        gc, gg, gm = eng.get_round(k)
        assert np.array_equal(gc, cand_all)
        force_accept = resync
        for b in range(B):
            if ora[b] is None:
                continue
            for i in range(T):
                if gg[b, i] != ora[b]["g"][i]:
                    m = ora[b]["margin"][i]
                    assert m <= MARGIN, ("verify argmax differs at a wide margin", r, b, i, m)
                    rep.listed.append((r, b, "verify", i, float(m)))
                    force_accept = True
        if check_logits:
            lg = eng.get_logits(B * T).reshape(B, T, V)
            for b in range(B):
                if ora[b] is None:
                    continue
                err = np.abs(lg[b] - ora[b]["logits"]).max()
                assert err <= LOGIT_TOL, ("logits", r, b, err)
                rep.max_logit_err = max(rep.max_logit_err, float(err))
        # ---- accept / rollback (forced to the oracle's decision when the pattern is forced or a listed
        #      narrow-margin position made the GPU's own decision differ)
        fn_dev = fx_dev = None
        if forced is not None or force_accept:
            fn_dev = torch.tensor([o["n"] if o is not None else int(forced[b][r]) for b, o in enumerate(ora)],
                                  dtype=torch.int32, device=dev)
        if force_accept:
            fx_dev = torch.tensor([int(o["emitted"][-1]) if o is not None else -1 for o in ora], dtype=torch.int32, device=dev)
        n, em = eng.accept_rollback(fn_dev, fx_dev, readback=True)
        for b in range(B):
            if ora[b] is None:
                assert n[b] == forced[b][r]
                continue
            assert n[b] == ora[b]["n"], ("accept length", r, b, n[b], ora[b]["n"])
            want = ora[b]["emitted"]
            assert np.array_equal(em[b, : n[b] + 1], want), ("emitted", r, b, em[b], want)
            assert (em[b, n[b] + 1:] == -1).all()
            rep.n_hist[int(n[b])] = rep.n_hist.get(int(n[b]), 0) + 1
            rep.tokens += int(n[b]) + 1
        rep.rounds += 1
        if check_states_every and (r % check_states_every == 0 or r == rounds - 1):
            compare_states(eng, seqs, shape, rep, kv_rows=2 * T + 2)
    return rep


# a draw or an accept test whose uniform lies closer than this to a decision boundary (in the oracle's double
# arithmetic) may come out differently in float32: such rounds are listed and the GPU is given the oracle's outcome
CDF_MARGIN = 5e-3
ACCEPT_MARGIN = 2e-2


def run_rounds_sampled(eng, seqs, shape, k, rounds, tau, seed=11, rep=None):
    """Rounds at temperature tau > 0 (Eq. 6) with the same float32 uniforms on both sides.  The library draws the
    drafts, decides the accept length and draws the correction / bonus token on the device; everything must equal the
    oracle's round wherever the oracle's decision margins are wide.  Returns (report, rounds compared in full)."""
    import torch
    rep = rep or Report()
    B, T, dev, mk = len(seqs), k + 1, eng.device, eng.max_k
    ud = torch.zeros((eng.max_batch, mk), dtype=torch.float32, device=dev)
    ua = torch.zeros((eng.max_batch, mk), dtype=torch.float32, device=dev)
    uf = torch.zeros((eng.max_batch,), dtype=torch.float32, device=dev)
    eng.set_sampling(tau, ud, ua, uf)
    full = 0
    for r in range(rounds):
        u = np.stack([hi.uniform01(seed, 1000 * b + r, 2 * mk + 1).astype(np.float32) for b in range(B)])
        u = np.minimum(u, np.float32(1.0 - 2.0 ** -24))            # keep [0, 1) after rounding to float32
        with torch.cuda.stream(eng.stream):
            ud[:B].copy_(torch.from_numpy(u[:, :mk]).to(dev)); ua[:B].copy_(torch.from_numpy(u[:, mk:2 * mk]).to(dev))
            uf[:B].copy_(torch.from_numpy(u[:, 2 * mk]).to(dev))
        ora = [o.round_sampled(k, tau, u[b, :k].astype(np.float64), u[b, mk:mk + k].astype(np.float64), float(u[b, 2 * mk]))
               for b, o in enumerate(seqs)]
        eng.draft(k)
        eng.last_k = k
        gc, _, _ = eng.get_round(k)
        resync = False
        for b in range(B):
            mg = ora[b]["margins"]
            for i in range(1, T):
                if gc[b, i] != ora[b]["cand"][i]:
                    assert mg[i - 1] <= CDF_MARGIN, ("draft draw differs at a wide margin", r, b, i, mg[i - 1])
                    rep.listed.append((r, b, "draft draw", i, float(mg[i - 1])))
                    resync = True
                    break
        cand_all = np.stack([o["cand"] for o in ora]).astype(np.int32)
        eng.verify(k, torch.from_numpy(cand_all).to(dev) if resync else None)
        narrow = resync
        for b in range(B):
            mg, n = ora[b]["margins"], ora[b]["n"]
            if any(mg[k + i] <= ACCEPT_MARGIN for i in range(min(n + 1, k))) or mg[2 * k] <= CDF_MARGIN:
                narrow = True
                rep.listed.append((r, b, "accept / final draw", n, float(min(mg[k:].min(), mg[2 * k]))))
        if narrow:       # hand the GPU the oracle's outcome for this round (states stay comparable)
            fn = torch.tensor([o["n"] for o in ora], dtype=torch.int32, device=dev)
            fx = torch.tensor([int(o["emitted"][-1]) for o in ora], dtype=torch.int32, device=dev)
            n, em = eng.accept_rollback(fn, fx, readback=True)
        else:
            n, em = eng.accept_rollback(readback=True)
            full += 1
        for b in range(B):
            assert n[b] == ora[b]["n"], ("accept length", r, b, n[b], ora[b]["n"], ora[b]["margins"])
            assert np.array_equal(em[b, : n[b] + 1], ora[b]["emitted"]), ("emitted", r, b, em[b], ora[b]["emitted"], ora[b]["margins"])
            rep.n_hist[int(n[b])] = rep.n_hist.get(int(n[b]), 0) + 1
            rep.tokens += int(n[b]) + 1
        rep.rounds += 1
        compare_states(eng, seqs, shape, rep, kv_rows=2 * T + 2)
    eng.set_sampling(0.0)
    return rep, full


def inject_context(eng, oseq, shape, b, kv_len, pending, seed=3):
    """Give GPU sequence b and the oracle sequence `oseq` (or None: GPU only, recurrent state only) the same
    synthetic context: seeded recurrent state, conv window and kv_len KV rows per layer, plus the pending token."""
    s = shape
    for l in range(s.L):
        t = s.layer_type(l)
        if t != hi.LAYER_ATT:
            kind, ctx = (hs.STATE_SSM, hi.CTX_SSM) if t == hi.LAYER_PAR else (hs.STATE_GDN, hi.CTX_GDN)
            st = hi.injected_state(s, l, b, ctx, seed)
            cv = hi.injected_state(s, l, b, hi.CTX_CONV, seed)
            eng.import_state(l, b, kind, st)
            eng.import_state(l, b, hs.STATE_CONV, cv)
            if oseq is not None:
                (oseq.ssm() if t == hi.LAYER_PAR else oseq.gdn())[l] = st
                oseq.conv()[l] = cv
        if t != hi.LAYER_GDN and oseq is not None and kv_len > 0:
            K = hi.injected_kv(s, l, b, kv_len, hi.CTX_K, seed)
            V = hi.injected_kv(s, l, b, kv_len, hi.CTX_V, seed)
            eng.import_state(l, b, hs.STATE_K, K)
            eng.import_state(l, b, hs.STATE_V, V)
            oseq.k()[l, :kv_len] = K
            oseq.v()[l, :kv_len] = V
    eng.set_context(b, kv_len, pending)
    if oseq is not None:
        oseq.set(kv_len, pending)
