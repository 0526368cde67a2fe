"""The report path of the bounded device-side waits, without hanging or faulting anything: a status
word written from the host, and the library's own self-test kernel, whose wait for a barrier that
nobody signals runs out after a short limit.  Both must surface as ATF_ERR_TIMEOUT exactly once."""
import pytest
import torch

import atf_inputs as gen

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def atf():
    import paper_2608_02947_b200 as m
    m.lib()
    return m


def test_status_word_is_reported_once_and_cleared(atf):
    ws = atf.ensure_workspace(1 << 20, torch.device("cuda", torch.cuda.current_device()))
    torch.cuda.synchronize()
    atf.binding.check_status()
    words = ws[:8].view(torch.int32)
    words[0], words[1] = 1, 7
    torch.cuda.synchronize()
    with pytest.raises(atf.AtfError) as e:
        atf.binding.check_status()
    assert e.value.code == 5 and "site 7" in str(e.value)
    atf.binding.check_status()  # cleared by the report
    # the same through the call that takes the workspace explicitly
    other = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    other[:8].view(torch.int32)[0] = 1
    with pytest.raises(atf.AtfError) as e:
        atf.binding.check_status(other)
    assert e.value.code == 5
    atf.binding.check_status(other)


def test_a_wait_that_runs_out_is_reported(atf):
    atf.ensure_workspace(1 << 20, torch.device("cuda", torch.cuda.current_device()))
    atf.binding.check_status()
    atf.binding.selftest_bounded_wait(300)  # gives up after 0.3 ms and returns; the context stays usable
    torch.cuda.synchronize()
    with pytest.raises(atf.AtfError) as e:
        atf.binding.check_status()
    assert e.value.code == 5 and "site 99" in str(e.value)
    atf.binding.check_status()
    # and the library still computes afterwards
    w = gen.tiny(N=300)
    Q, K, V = gen.prefill_inputs(w, device="cuda")
    O, LSE = atf.atf_prefill(Q, K, V, table=None)
    torch.cuda.synchronize()
    atf.binding.check_status()
    assert torch.isfinite(O.float()).all() and torch.isfinite(LSE).all()


def test_every_window_covering_the_prompt_makes_all_modes_one(atf):
    """k = infinity: table = NULL, an all-N table in exact mode and the same table in coarse mode are the same
    computation, bit for bit, with the full term count."""
    w = gen.Workload("allN", 1, 4, 2, 128, 700, 5e5, 2.0, None, gen.SEED0 + 90)
    Q, K, V = gen.prefill_inputs(w, device="cuda")
    W = torch.full((w.d // 2,), w.N, dtype=torch.int64)
    outs = []
    for table, mode in ((None, atf.ATF_MODE_EXACT), (W, atf.ATF_MODE_EXACT), (W, atf.ATF_MODE_COARSE)):
        kept = torch.zeros(w.B * w.Hq, dtype=torch.int64, device="cuda")
        O, LSE = atf.atf_prefill(Q, K, V, table=table, mode=mode, kept_terms=kept)
        torch.cuda.synchronize()
        assert kept.cpu().tolist() == [(w.d // 2) * w.N * (w.N + 1) // 2] * (w.B * w.Hq)
        outs.append((O.clone(), LSE.clone()))
    for O, LSE in outs[1:]:
        assert torch.equal(O.view(torch.int16), outs[0][0].view(torch.int16)) and torch.equal(LSE, outs[0][1])
