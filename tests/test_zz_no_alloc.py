"""The allocation-free argmax entry point (hs_argmax_static) against the model's own argmax.

Some users of the library cannot allocate device memory at the point where they need a result: they
run inside somebody else's memory plan, or they must not trigger the synchronisation an allocation
can bring.  For them the library keeps the argmax kernel's scratch in a built-in device array.  This
test feeds that entry point the logits of a verify pass and expects exactly the tokens and margins the
verify pass itself produced (same kernel, so the comparison is bit-exact), twice in a row so that a
stale counter or partial left behind by the first call would show, and checks the size limit.
The file name makes pytest collect it after every other test file.
"""
import numpy as np
import pytest

import hs_inputs as hi

pytestmark = pytest.mark.gpu


def test_static_argmax_matches_verify_twice_and_rejects_oversize():
    import torch
    from paper_2605_01106_b200 import build, binding as hs
    build.build()
    s = hi.CONFIGS["cfg1_tiny"]
    blob, _ = hi.make_weights(s, 0, "jitter")
    eng = hs.Engine(s, blob, max_batch=2, max_k=4, kv_capacity=128)
    eng.prefill([hi.make_prompt(s.V, 20, seq=0), hi.make_prompt(s.V, 13, seq=1)])
    dev = eng.device
    for call, k in enumerate((4, 2)):                      # two calls in a row, different row counts
        eng.draft(k)
        eng.verify(k)
        _, g, margin = eng.get_round(k)                    # what the existing entry points decided
        rows = 2 * (k + 1)
        logits = torch.from_numpy(eng.get_logits(rows)).to(dev)
        eng.accept_rollback()
        tok = torch.full((rows,), -7, dtype=torch.int32, device=dev)
        mar = torch.full((rows,), -1.0, dtype=torch.float32, device=dev)
        # number of allocation events so far (frees of other tests' buffers do not change it)
        before = torch.cuda.memory_stats(dev)["allocation.all.allocated"]
        hs.argmax_static(logits, tok, mar)
        torch.cuda.synchronize(dev)
        assert torch.cuda.memory_stats(dev)["allocation.all.allocated"] == before
        assert np.array_equal(tok.cpu().numpy(), g.reshape(-1)), (call, tok.cpu().numpy(), g)
        assert np.array_equal(mar.cpu().numpy(), margin.reshape(-1)), call
        # and against a plain definition: first index of the maximum, top1 - top2
        lg = logits.cpu().numpy()
        assert np.array_equal(tok.cpu().numpy(), lg.argmax(axis=1).astype(np.int32))
        top2 = np.sort(lg, axis=1)[:, -2:]
        assert np.array_equal(mar.cpu().numpy(), top2[:, 1] - top2[:, 0])
    # margins are optional
    tok2 = torch.zeros(rows, dtype=torch.int32, device=dev)
    hs.argmax_static(logits, tok2, None)
    torch.cuda.synchronize(dev)
    assert np.array_equal(tok2.cpu().numpy(), tok.cpu().numpy())
    # more rows than the built-in scratch holds: a clear error, nothing launched
    big = torch.zeros((65, 8), dtype=torch.float32, device=dev)
    with pytest.raises(hs.HsError) as e:
        hs.argmax_static(big, torch.zeros(65, dtype=torch.int32, device=dev))
    assert e.value.code == -2
    assert eng.device_status() == 0


def test_static_argmax_ties_odd_widths_and_misaligned_views():
    """The device-side tie rule (lowest id wins, margin 0 when the maximum is not unique), row widths that are not
    a multiple of four or smaller than the number of blocks that share a row, rows without any finite value, and
    the refusal of a logits view that does not start on a 16-byte boundary - all through the C entry point."""
    import torch
    from paper_2605_01106_b200 import build, binding as hs
    build.build()
    dev = torch.device("cuda:0")
    g = torch.Generator(device="cpu").manual_seed(5)

    def run(lg):
        rows = lg.shape[0]
        tok = torch.full((rows,), -7, dtype=torch.int32, device=dev)
        mar = torch.full((rows,), -1.0, dtype=torch.float32, device=dev)
        hs.argmax_static(lg, tok, mar)
        torch.cuda.synchronize(dev)
        return tok.cpu().numpy(), mar.cpu().numpy()

    # ties: the maximum duplicated inside one block's slice, across slices (ids 5, 1000 and 4000 of 4096 lie in
    # different 128-wide slices), at the very last id, and a constant row
    V = 4096
    lg = torch.randn(6, V, generator=g).clamp_(-3, 3)
    lg[0, [5, 6]] = 9.0
    lg[1, [4000, 1000, 5]] = 9.0
    lg[2, [V - 1, 77]] = 9.0
    lg[3, :] = 0.25
    lg[4, 2049] = 9.0                                     # unique maximum: margin is top1 - top2
    lg[5, [0, V - 1]] = 9.0
    tok, mar = run(lg.to(dev))
    assert list(tok) == [5, 5, 77, 0, 2049, 0], tok
    assert list(mar[[0, 1, 2, 3, 5]]) == [0.0] * 5
    assert mar[4] == 9.0 - float(lg[4][lg[4] < 9.0].max())
    # widths that are not a multiple of four (scalar path) and narrower than the 32 blocks of a row
    for V in (7, 30, 33, 1001):
        lg = torch.randn(5, V, generator=g)
        lg[1, V - 1] = 50.0
        lg[2, [V // 2, V - 2]] = 50.0
        tok, mar = run(lg.to(dev))
        ref = lg.numpy()
        assert np.array_equal(tok, ref.argmax(axis=1).astype(np.int32)), (V, tok)
        top2 = np.sort(ref, axis=1)[:, -2:]
        assert np.array_equal(mar, top2[:, 1] - top2[:, 0]), V
    # a row with no finite value: id 0 (always a valid token), margin 0
    lg = torch.full((2, 64), float("-inf"))
    lg[1, :] = float("nan")
    tok, mar = run(lg.to(dev))
    assert list(tok) == [0, 0] and list(mar) == [0.0, 0.0]
    # a view that starts one float into a larger tensor is only 4-byte aligned: with V % 4 == 0 it is refused on the
    # host (the kernel would read it 128 bits at a time), with an odd V it is served by the scalar path
    big = torch.randn(4 * 64 + 1, generator=g).to(dev)
    view = big[1:].view(4, 64)
    assert view.data_ptr() % 16 == 4
    tok = torch.zeros(4, dtype=torch.int32, device=dev)
    with pytest.raises(hs.HsError) as e:
        hs.argmax_static(view, tok)
    assert e.value.code == -1
    view7 = big[1:1 + 4 * 7].view(4, 7)
    hs.argmax_static(view7, tok)
    torch.cuda.synchronize(dev)
    assert np.array_equal(tok.cpu().numpy(), view7.cpu().numpy().argmax(axis=1).astype(np.int32))
    # the binding refuses tensors the C entry point could not interpret
    for bad in (lambda: hs.argmax_static(view.half(), tok), lambda: hs.argmax_static(big[: 4 * 64].view(4, 64).t(), tok),
                lambda: hs.argmax_static(big[: 4 * 64].view(4, 64), tok[:3])):
        with pytest.raises(hs.HsError):
            bad()
