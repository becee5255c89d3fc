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
