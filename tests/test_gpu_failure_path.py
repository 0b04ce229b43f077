"""The device-side failure path, exercised without provoking a fault: a bounded wait that nothing
satisfies must give up after its budget, leave the time-out bit in the status word, and leave the
context usable (the next forward still matches the oracle)."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import oracle  # noqa: E402
from synth.inputs import CONFIGS, make_inputs  # noqa: E402

pytestmark = pytest.mark.gpu

RLX_OK, RLX_ERR_DEVICE_TIMEOUT = 0, 5


@pytest.fixture(scope="module")
def rlx():
    import paper_2609_37916_b200 as pkg
    from paper_2609_37916_b200.build import build
    build()
    return pkg


def test_bounded_wait_expires_and_is_reported(rlx):
    inp = make_inputs(CONFIGS["c0"])
    c = inp.cfg
    enc = rlx.Encoder.from_config(c, max_batch=c.batch, max_seq=c.seq)
    ws = enc.alloc_workspace(c.batch, c.seq)
    w = rlx.upload_weights(inp.params, inp.layers)
    out = torch.empty((c.batch, c.hidden), dtype=torch.float32, device="cuda")
    ids, mask = torch.from_numpy(inp.ids).cuda(), torch.from_numpy(inp.mask).cuda()
    enc.forward(ids, mask, w, out, ws)
    assert enc.last_device_status(ws) == RLX_OK

    waited = torch.zeros(1, dtype=torch.int64, device="cuda")
    status_word = ws.view(torch.int32)[:1]          # the sticky status word is the first word of the workspace
    rlx.binding.selftest_bounded_wait(2000, status_word, waited)      # 2 ms budget, nothing ever arrives
    torch.cuda.synchronize()
    assert 2_000_000 <= int(waited.item()) < 50_000_000               # gave up after the budget, not much later
    assert enc.last_device_status(ws) == RLX_ERR_DEVICE_TIMEOUT
    assert enc.last_device_status(ws) == RLX_OK                       # reading clears the sticky word

    # the context is intact: the same forward again, against the oracle
    enc.forward(ids, mask, w, out, ws)
    torch.cuda.synchronize()
    assert enc.last_device_status(ws) == RLX_OK
    ref = oracle.encoder_forward(c, inp.ids, inp.mask, inp.params, inp.layers)
    got = out.double().cpu().numpy()
    assert np.abs(got - ref).max() <= 2e-2
    enc.close()


def test_selftest_rejects_unbounded_budgets(rlx):
    word = torch.zeros(1, dtype=torch.int32, device="cuda")
    for bad in (0, 100001):
        with pytest.raises(rlx.RlxError):
            rlx.binding.selftest_bounded_wait(bad, word)
    with pytest.raises(rlx.RlxError):
        rlx.binding.selftest_bounded_wait(10, None)
