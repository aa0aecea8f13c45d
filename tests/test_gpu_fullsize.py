"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The calls are made exactly as bench.py makes them (device-generated inputs, the library's own
neighbour table, outputs without trace for the headline call).  The oracle then recomputes a
seeded sample of sequences one by one from the device bytes copied back, on neighbour rows that
the oracle builds itself for the sampled sequences' drafted tokens (and that are compared with
the library's rows first); every sequence is also checked for the properties that hold at any size.
"""
import numpy as np
import pytest
import torch

import lantern_inputs as li
import lantern_inputs.device as lid
import oracle
import paper_2410_03355_b200 as lt
from parity import assert_parity, compare, near_ceiling, oracle_table

pytestmark = pytest.mark.gpu


_codebooks = {}


def _table(name):
    c = li.CONFIGS[name]
    cbh = _codebooks.setdefault(name, li.config_codebook(name))
    cb = torch.from_numpy(cbh).cuda()
    ws = torch.empty(max(lt.build_workspace_bytes(c["V"], c["D"], c["k"]), 16), dtype=torch.uint8, device="cuda")
    return lt.build_neighbors(cb, c["k"], with_dist=False, workspace=ws)[0]


def _oracle_rows(name, host_inp, table):
    """The oracle's own neighbour rows for every token the sampled sequences draft, checked against the library's."""
    return oracle_table(_codebooks[name], li.CONFIGS[name]["k"], host_inp.draft_tokens, table)


def _take(out: lt.VerifyOutputs, rows) -> lt.VerifyOutputs:
    idx = torch.as_tensor(rows, device=out.accept_len.device)
    pick = lambda t: None if t is None else t[idx]
    return lt.VerifyOutputs(accept_len=pick(out.accept_len), next_token=pick(out.next_token),
                            accept_path=pick(out.accept_path), status=pick(out.status), node_qa=pick(out.node_qa),
                            node_px=pick(out.node_px), node_m=pick(out.node_m))


def _properties(d, out, N, V):
    al = out.accept_len.cpu().numpy()
    tok = out.next_token.cpu().numpy()
    path = out.accept_path.cpu().numpy()
    assert int((out.status != 0).sum()) == 0
    assert al.min() >= 0 and al.max() <= N
    assert tok.min() >= 0 and tok.max() < V
    par = None if d["tree_parents"] is None else d["tree_parents"].cpu().numpy()
    for b in range(0, al.shape[0], max(1, al.shape[0] // 512)):
        prev = -1
        for j in range(al[b]):
            node = path[b, j]
            assert (par[b, node] if par is not None else node - 1) == prev
            prev = node
        assert np.all(path[b, al[b]:] == -1)


@pytest.mark.parametrize("workload,sample", [("batch_chain", 96), ("stress", 64)])
def test_bench_sized_call_against_sampled_oracle(workload, sample):
    import bench
    w = bench.WORKLOADS[workload]
    cfg = li.CONFIGS[w["config"]]
    B, N, V, delta = w["B"], cfg["N"], cfg["V"], cfg["delta"]
    table = _table(w["config"])
    d = lid.config_verify_inputs_device(w["config"], B=B, seed=bench.rank_seed(li.BASE_SEED, 0))
    out = lt.verify(d["target_logits"], d["draft_logits"], d["cfg_scale"], d["T"], d["draft_tokens"],
                    d["tree_parents"], table, delta, d["uniforms"], trace=True)
    torch.cuda.synchronize()
    _properties(d, out, N, V)
    rows = np.sort(np.random.default_rng(11).choice(B, size=min(sample, B), replace=False))
    host = lid.to_host(d, rows=rows)
    res = compare(host, _oracle_rows(w["config"], host, table), delta, _take(out, rows))
    assert_parity(res)
    assert res["nodes_tested"] >= len(rows)
    assert res["near"] <= near_ceiling(len(rows)), res
    # the headline call is made without trace outputs: same decisions
    out2 = lt.verify(d["target_logits"], d["draft_logits"], d["cfg_scale"], d["T"], d["draft_tokens"],
                     d["tree_parents"], table, delta, d["uniforms"])
    torch.cuda.synchronize()
    assert torch.equal(out.accept_len, out2.accept_len) and torch.equal(out.next_token, out2.next_token)
    assert torch.equal(out.accept_path, out2.accept_path)


@pytest.mark.parametrize("workload,sample,divergence,top_k", [
    ("batch_chain", 64, oracle.DIV_JSD, 0),
    ("batch_chain", 64, oracle.DIV_TVD, 1000),       # Appendix B.2's text-conditional setting
    ("stress", 48, oracle.DIV_JSD, 2000),
])
def test_bench_sized_variants_against_sampled_oracle(workload, sample, divergence, top_k):
    """The calls `bench.py --divergence jsd` / `--top-k K` time, checked on a seeded sample of their sequences."""
    import bench
    from parity import DIV_NAME
    w = bench.WORKLOADS[workload]
    cfg = li.CONFIGS[w["config"]]
    B, N, V, delta = w["B"], cfg["N"], cfg["V"], cfg["delta"]
    table = _table(w["config"])
    d = lid.config_verify_inputs_device(w["config"], B=B, seed=bench.rank_seed(li.BASE_SEED, 0))
    out = lt.verify(d["target_logits"], d["draft_logits"], d["cfg_scale"], d["T"], d["draft_tokens"],
                    d["tree_parents"], table, delta, d["uniforms"], trace=True, divergence=DIV_NAME[divergence],
                    top_k=top_k)
    torch.cuda.synchronize()
    _properties(d, out, N, V)
    rows = np.sort(np.random.default_rng(13).choice(B, size=min(sample, B), replace=False))
    host = lid.to_host(d, rows=rows)
    res = compare(host, _oracle_rows(w["config"], host, table), delta, _take(out, rows), divergence=divergence,
                  top_k=top_k)
    assert_parity(res)
    assert res["nodes_tested"] >= len(rows)
    assert res["near"] <= near_ceiling(len(rows)), res
