"""CUDA all-token aggregation (a benchmark of the V x k gather-sum; not used by verify) against the oracle:
|A_{k,delta}(x)| identical for every token except where the cut lies within WINDOW of the bound, the
aggregated mass to REL where the cut agrees."""
import numpy as np
import pytest
import torch

import lantern_inputs as li
import oracle
import paper_2410_03355_b200 as lt
from parity import REL, WINDOW

pytestmark = pytest.mark.gpu


def rows_of(inp):
    t = torch.from_numpy(inp.target_logits[:, :, 0])          # [C, rows, V]: the root contexts
    if inp.dtype == li.BF16:
        t = t.view(torch.int16).view(torch.bfloat16)
    return t.contiguous().cuda()


@pytest.mark.parametrize("V,k,rows,dtype,unc,T,delta", [
    (1024, 16, 8, li.F32, False, 1.0, 0.05),
    (1024, 16, 8, li.BF16, True, 1.0, 0.05),
    (1000, 300, 5, li.BF16, True, 0.8, 0.1),        # k a multiple of 4: 16-byte table loads
    (1000, 301, 5, li.BF16, True, 1.0, 0.1),        # k not a multiple of 4: scalar table loads
    (16384, 1000, 2, li.BF16, True, 1.0, 0.4),      # the chain workload's row shape
    (2048, 2048, 3, li.F32, True, 1.0, 2.0),        # the bound never binds: a product with B_k's 0/1 matrix
    (512, 32, 6, li.BF16, False, 1.0, 0.0),         # delta = 0: q itself
    (8, 1, 4, li.F32, False, 1.0, 0.3),
])
def test_aggregate_against_oracle(V, k, rows, dtype, unc, T, delta):
    cb = li.codebook_gaussian(V, 8, seed=31)
    table = oracle.build_neighbors(cb, k)[0]        # every row is read: the oracle builds the whole table
    inp = li.verify_inputs(rows, 0, V, dtype=dtype, has_uncond=unc, cfg_scale=3.0 if unc else 1.0, T=T,
                           sigma_target=1.0, sigma_draft=1.0, rho=0.9, seed=3 + V + k)
    want, m_want, margin = oracle.aggregate_all(inp.target_logits[0, :, 0], inp.target_logits[1, :, 0] if unc else None,
                                                dtype, inp.cfg_scale, T, table, delta)
    agg, m, status = lt.aggregate_all(rows_of(inp), inp.cfg_scale, T, torch.from_numpy(table).cuda(), delta)
    torch.cuda.synchronize()
    agg, m = agg.cpu().numpy(), m.cpu().numpy()
    assert not status.cpu().numpy().any()
    far = margin >= WINDOW
    assert np.array_equal(m[far], m_want[far])
    same = m == m_want
    assert same.mean() > 0.99
    assert (np.abs(agg[same] - want[same]) <= REL * want[same] + 1e-30).all()
    if delta == 0.0 or k == 1:
        assert not m.any()


def test_aggregate_status_and_arguments():
    V, k = 1024, 16
    table = oracle.build_neighbors(li.codebook_gaussian(V, 8, seed=31), k)[0]
    inp = li.verify_inputs(4, 0, V, dtype=li.F32, has_uncond=False, cfg_scale=1.0, sigma_target=1.0,
                           sigma_draft=1.0, rho=0.0, seed=9)
    inp.target_logits[0, 1, 0, 5] = np.nan
    bad = table.copy()
    bad[7, 3] = V + 4
    agg, m, status = lt.aggregate_all(rows_of(inp), 1.0, 1.0, torch.from_numpy(bad).cuda(), 0.1)
    st = status.cpu().numpy()
    assert st[1] == lt.ST_NONFINITE and torch.isnan(agg[1]).all() and (m[1] == -1).all()
    assert st[0] == lt.ST_BAD_TABLE and st[2] == lt.ST_BAD_TABLE
    with pytest.raises(lt.LanternError):
        lt.aggregate_all(rows_of(inp), 1.0, 0.0, torch.from_numpy(table).cuda(), 0.1)      # T must be positive
