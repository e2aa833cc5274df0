"""QA-bank lookup kernel against its CPU definition, through the C ABI."""
import numpy as np
import pytest

from oracle import qa_bank as qa
from paper_2601_11553_b200 import percache as pcb

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n,dim,nq", [(1, 1024, 1), (37, 64, 3), (5000, 1024, 1), (5000, 1024, 8), (20011, 384, 5)])
def test_qa_top1_matches_definition(n, dim, nq):
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(n + dim + nq)
    bank = rng.standard_normal((n, dim)).astype(np.float32)
    src = rng.integers(0, n, size=nq)
    noise = np.linspace(0.0, 1.5, nq)[:, None]                   # from exact copies to unrelated vectors
    queries = (bank[src] * rng.uniform(0.5, 2.0, size=(nq, 1)) + noise * rng.standard_normal((nq, dim))).astype(np.float32)
    if n > 40:
        bank[n // 2] = bank[3] * 2.0                              # an exact cosine tie between rows 3 and n // 2
        queries[0] = bank[3]
    idx, best, hit, scores = qa.top1(bank, queries, 0.85)
    g_idx, g_best, g_hit = pcb.qa_top1(torch.from_numpy(bank).cuda(), torch.from_numpy(queries).cuda(), 0.85)
    assert np.max(np.abs(g_best - best)) < 2e-6
    for q in range(nq):
        # fp32 decides the arg-max on the GPU: accept an entry whose exact score is within rounding of the best
        assert scores[q, g_idx[q]] >= best[q] - 2e-6
        if abs(best[q] - 0.85) > 1e-5:
            assert g_hit[q] == hit[q]
    if n > 40:
        assert g_idx[0] == 3                                      # lowest index among exactly equal scores


def test_qa_top1_argument_errors():
    torch = pytest.importorskip("torch")
    bank = torch.zeros((4, 8), dtype=torch.float32).cuda()
    with pytest.raises(pcb.PerCacheError) as e:
        pcb.qa_top1(bank, torch.zeros((9, 8), dtype=torch.float32).cuda(), 0.5)
    assert e.value.code == pcb.E_CAPACITY
    with pytest.raises(pcb.PerCacheError) as e:
        pcb.qa_top1(torch.zeros((4, 6), dtype=torch.float32).cuda(), torch.zeros((1, 6), dtype=torch.float32).cuda(), 0.5)
    assert e.value.code == pcb.E_INVAL
