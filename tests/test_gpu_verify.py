"""CUDA verification step against the oracle (tests/parity.py states the comparison rule)."""
import dataclasses

import numpy as np
import pytest
import torch

import lantern_inputs as li
import oracle
import paper_2410_03355_b200 as lt
from parity import assert_parity, compare, near_ceiling, oracle_table, run_gpu, to_device

pytestmark = pytest.mark.gpu

_tables = {}


class LazyOracleTable:
    """Host table of a full-size configuration: rows are built by the ORACLE for the tokens a call drafts
    and compared with the library's rows (`dev`) before the call's decisions are."""

    def __init__(self, cb, k, dev):
        self.cb, self.k, self.dev = cb, k, dev

    def for_tokens(self, tokens):
        return oracle_table(self.cb, self.k, tokens, self.dev)


def table_for(name, V=None, k=None):
    """(host table, device table) for a configuration's codebook.  On small V both are the oracle's full
    table; on the full V the device table is the library's and the host side builds, per call, the
    oracle's rows for the drafted tokens."""
    c = li.CONFIGS[name]
    V = V or c["V"]
    k = k or c["k"]
    key = (c["codebook"], c["D"], V, k)
    if key not in _tables:
        cb = li.config_codebook(name, V=V)
        if V <= 2048:
            host = oracle.build_neighbors(cb, k)[0]
            dev = torch.from_numpy(host).cuda()
        else:
            dev = lt.build_neighbors(torch.from_numpy(cb).cuda(), k, with_dist=False)[0]
            torch.cuda.synchronize()
            host = LazyOracleTable(cb, k, dev)
        _tables[key] = (host, dev)
    return _tables[key]


def check(inp, host, dev, delta, min_tested=1):
    if isinstance(host, LazyOracleTable):
        host = host.for_tokens(inp.draft_tokens)
    gpu = run_gpu(inp, dev, delta)
    res = compare(inp, host, delta, gpu)
    assert_parity(res)
    assert res["nodes_tested"] >= min_tested
    assert res["near"] <= near_ceiling(inp.B), res
    return res


# ------------------------------------------------------------------ small shapes, many cases
@pytest.mark.parametrize("V,k,N,B,dtype,unc", [
    (1024, 16, 4, 64, li.F32, False),        # the tiny configuration's shape
    (1024, 16, 4, 64, li.BF16, True),
    (8, 1, 1, 33, li.F32, False),            # smallest legal vocabulary, k = 1
    (8, 8, 3, 17, li.BF16, False),
    (1000, 300, 7, 40, li.BF16, True),       # V not a power of two, ragged last chunk
    (8192, 1000, 5, 12, li.F32, True),       # largest fp32 + guidance shape
    (8200, 64, 3, 9, li.BF16, True),         # just over one chunk per thread
    (2048, 2048, 2, 6, li.BF16, True),       # k = V: two scan rounds of the neighbour row
])
def test_chain_shapes(V, k, N, B, dtype, unc):
    cb = li.codebook_gaussian(V, 8, seed=31)
    host = oracle.build_neighbors(cb, k)[0]
    dev = torch.from_numpy(host).cuda()
    for seed, delta, T in [(1, 0.1, 1.0), (2, 0.4, 0.8), (3, 0.0, 1.3)]:
        inp = li.verify_inputs(B, N, V, dtype=dtype, has_uncond=unc, cfg_scale=3.0 if unc else 1.0, T=T,
                               sigma_target=1.5, sigma_draft=0.8, rho=0.8, peaked_frac=0.1, seed=seed)
        check(inp, host, dev, delta, min_tested=B)


@pytest.mark.parametrize("depth,N", [(6, 60), (3, 25), (1, 12)])
def test_trees(depth, N):
    V, k = 2048, 100
    cb = li.codebook_gaussian(V, 8, seed=32)
    host = oracle.build_neighbors(cb, k)[0]
    dev = torch.from_numpy(host).cuda()
    n_sib = 0
    for seed in range(4):
        par = li.tree_parents(24, N, depth=depth, seed=seed)
        inp = li.verify_inputs(24, N, V, dtype=li.BF16, has_uncond=True, cfg_scale=2.0, sigma_target=1.0,
                               sigma_draft=1.0, rho=0.9, parents=par, seed=100 + seed)
        for delta in (0.0, 0.05, 0.3):
            res = check(inp, host, dev, delta, min_tested=24)
            n_sib += res["nodes_tested"]
    assert n_sib > 24 * 4 * 3 * 1.5        # sibling rounds were exercised


def test_long_chain_and_wide_tree():
    """Draft lengths far beyond the paper's settings: the plan's per-sequence arrays, the breadth-first ranks
    and the dead marks over hundreds of contexts (a rejection at depth d strikes the N - d contexts behind it)."""
    V, k = 256, 16
    cb = li.codebook_gaussian(V, 8, seed=39)
    host = oracle.build_neighbors(cb, k)[0]
    dev = torch.from_numpy(host).cuda()
    inp = li.verify_inputs(5, 300, V, dtype=li.BF16, has_uncond=True, cfg_scale=1.5, sigma_target=1.0, sigma_draft=0.15,
                           rho=0.95, seed=61)
    res = check(inp, host, dev, 0.3, min_tested=5)
    assert res["accept_mean"] > 3
    wide = li.verify_inputs(6, 200, V, dtype=li.F32, has_uncond=False, cfg_scale=1.0, sigma_draft=0.6,
                            parents=li.tree_parents(6, 200, depth=6, seed=4), seed=62)
    check(wide, host, dev, 0.1, min_tested=6)
    inp = li.verify_inputs(2, 1024, V, dtype=li.BF16, has_uncond=False, cfg_scale=1.0, sigma_draft=0.05, seed=63)
    check(inp, host, dev, 0.5, min_tested=2)          # the longest supported chain


def test_deep_explicit_trees():
    """Trees whose depth is of the order of their size: the longest chain written as a tree (every level holds
    one node), and a spine with a leaf hanging off every spine node (the plan's depths, level order, subtree sizes
    and pre-order positions over hundreds of levels)."""
    V, k = 256, 16
    cb = li.codebook_gaussian(V, 8, seed=39)
    host = oracle.build_neighbors(cb, k)[0]
    dev = torch.from_numpy(host).cuda()
    inp = li.verify_inputs(2, 1024, V, dtype=li.BF16, has_uncond=False, cfg_scale=1.0, sigma_draft=0.05, seed=63)
    a = run_gpu(inp, dev, 0.5)
    b = run_gpu(dataclasses.replace(inp, tree_parents=li.chain_parents(2, 1024)), dev, 0.5)
    for f in ("accept_len", "next_token", "accept_path", "status"):
        assert torch.equal(getattr(a, f), getattr(b, f)), f
    assert int(a.accept_len.min()) > 20
    # spine nodes 0, 2, 4, ... (each the child of the spine node before), node 2j + 1 a second child of spine node 2j - 2
    N = 600
    par = np.empty((3, N), np.int32)
    for i in range(N):
        par[:, i] = i - 2 if i >= 2 else -1
    inp = li.verify_inputs(3, N, V, dtype=li.BF16, has_uncond=True, cfg_scale=1.5, sigma_target=1.0, sigma_draft=0.15,
                           rho=0.95, parents=par, seed=64)
    res = check(inp, host, dev, 0.3, min_tested=3)
    assert res["accept_mean"] > 3


def test_chain_equals_explicit_tree():
    V, k = 1024, 32
    cb = li.codebook_gaussian(V, 8, seed=33)
    host = oracle.build_neighbors(cb, k)[0]
    dev = torch.from_numpy(host).cuda()
    inp = li.verify_inputs(50, 6, V, seed=5, rho=0.9, sigma_draft=0.9)
    a = run_gpu(inp, dev, 0.2)
    b = run_gpu(dataclasses.replace(inp, tree_parents=li.chain_parents(50, 6)), dev, 0.2)
    for f in ("accept_len", "next_token", "accept_path", "status"):
        assert torch.equal(getattr(a, f), getattr(b, f)), f
    # per-node values are defined for the nodes the walk tests: those on the accepted path and the one after it
    tested = torch.arange(6, device="cuda")[None, :] <= a.accept_len[:, None]
    assert torch.equal(a.node_m[tested], b.node_m[tested])
    assert torch.equal(a.node_qa[tested], b.node_qa[tested]) and not torch.isnan(a.node_qa[tested]).any()


# ------------------------------------------------------------------ the named configurations
def test_config_tiny_all_steps():
    host, dev = table_for("tiny")
    tot = 0
    for step in range(64):
        inp = li.config_verify_inputs("tiny", step=step)
        tot += check(inp, host, dev, li.CONFIGS["tiny"]["delta"])["nodes_tested"]
    assert tot >= 64


@pytest.mark.parametrize("rho", [0.0, 0.99])
def test_config_single_image(rho):
    c = li.CONFIGS["single_image"]
    host, dev = table_for("single_image")
    for step in range(3):
        inp = li.config_verify_inputs("single_image", step=step, rho=rho)
        check(inp, host, dev, c["delta"])


@pytest.mark.parametrize("rho", [0.0, 0.99])
def test_config_batch_chain(rho):
    c = li.CONFIGS["batch_chain"]
    host, dev = table_for("batch_chain")
    near = 0
    for step in range(2):
        inp = li.config_verify_inputs("batch_chain", step=step, rho=rho)
        near += check(inp, host, dev, c["delta"], min_tested=32)["near"]
    print("near-threshold sequences:", near)


def test_config_px512_delta_sweep():
    host, dev = table_for("px512_tree")
    inp = li.config_verify_inputs("px512_tree", step=0)      # the configuration's own batch of 8
    lens = []
    for delta in (0.05, 0.1, 0.2, 0.4):
        res = check(inp, host, dev, delta)
        lens.append(res["accept_mean"])
    assert lens == sorted(lens) or max(lens) - min(lens) < 1.0   # acceptance grows with delta (Table 1's trend)


def test_config_stress_shape():
    host, dev = table_for("stress")
    inp = li.config_verify_inputs("stress", step=0, B=16, rho=0.99)
    check(inp, host, dev, li.CONFIGS["stress"]["delta"])


# ------------------------------------------------------------------ edges and faults
def test_no_drafts_and_empty_batch():
    V, k = 512, 8
    cb = li.codebook_gaussian(V, 8, seed=34)
    host = oracle.build_neighbors(cb, k)[0]
    dev = torch.from_numpy(host).cuda()
    inp = li.verify_inputs(9, 0, V, seed=3)              # N = 0: only the bonus draw
    res = compare(inp, host, 0.2, run_gpu(inp, dev, 0.2, trace=False))
    assert_parity(res)
    empty = li.verify_inputs(1, 2, V, seed=3)
    d = to_device(empty)
    out = lt.verify(d["target_logits"][:, :0], d["draft_logits"][:0], 1.0, 1.0, d["draft_tokens"][:0], None, dev,
                    0.2, d["uniforms"][:0])
    assert out.accept_len.numel() == 0


def test_data_faults_are_flagged_not_fatal():
    V, k = 512, 8
    cb = li.codebook_gaussian(V, 8, seed=35)
    host = oracle.build_neighbors(cb, k)[0]
    inp = li.verify_inputs(8, 3, V, dtype=li.F32, has_uncond=False, seed=9, sigma_draft=0.2)
    inp.tree_parents = li.chain_parents(8, 3)
    inp.tree_parents[0, 2] = 2
    inp.draft_tokens[1, 1] = V
    inp.uniforms[2, 0] = 1.0
    inp.target_logits[0, 3, 0, 5] = np.nan
    inp.target_logits[0, 4, 0, :] = -np.inf
    inp.target_logits[0, 5, 0, 7] = -np.inf
    inp.draft_logits[6, 0, 3] = np.inf
    dev = torch.from_numpy(host).cuda()
    gpu = run_gpu(inp, dev, 0.2)
    ora = oracle.verify_inputs(inp, host, 0.2)
    assert np.array_equal(gpu.status.cpu().numpy(), ora.status)
    assert np.array_equal(gpu.accept_len.cpu().numpy(), ora.accept_len)
    assert np.array_equal(gpu.next_token.cpu().numpy(), ora.next_token)
    assert ora.status[0] == lt.ST_BAD_PARENT and ora.status[3] == lt.ST_NONFINITE and ora.status[5] == 0
    # a corrupt neighbour table is reported and carries no mass
    bad = host.copy()
    bad[:, 1] = V + 3
    inp2 = li.verify_inputs(8, 3, V, seed=10)
    gpu = run_gpu(inp2, torch.from_numpy(bad).cuda(), 0.2)
    ora = oracle.verify_inputs(inp2, bad, 0.2)
    assert np.array_equal(gpu.status.cpu().numpy(), ora.status) and np.all(ora.status & lt.ST_BAD_TABLE)
    assert np.array_equal(gpu.accept_len.cpu().numpy(), ora.accept_len)
    assert np.array_equal(gpu.next_token.cpu().numpy(), ora.next_token)


def test_host_argument_errors():
    V, k = 512, 8
    dev = torch.zeros((V, k), dtype=torch.int32, device="cuda")
    inp = li.verify_inputs(2, 2, V, seed=1)
    d = to_device(inp)

    def call(**kw):
        a = dict(target_logits=d["target_logits"], draft_logits=d["draft_logits"], cfg_scale=1.0, T=1.0,
                 draft_tokens=d["draft_tokens"], tree_parents=None, neighbor_idx=dev, delta=0.1,
                 uniforms=d["uniforms"])
        a.update(kw)
        return lt.verify(**a)

    for kw, code in [(dict(T=-1.0), -3), (dict(uniforms=None, T=1.0), None), (dict(delta=-0.1), -3), (dict(delta=float("nan")), -3),
                     (dict(workspace=torch.empty(16, dtype=torch.uint8, device="cuda")), -4)]:
        if code is None:                             # sampling without uniforms: refused by the binding
            with pytest.raises(ValueError):
                call(**kw)
            continue
        with pytest.raises(lt.LanternError) as e:
            call(**kw)
        assert e.value.code == code, kw
    with pytest.raises(lt.LanternError) as e:       # V not a multiple of 8
        lt.verify(d["target_logits"][..., :500].contiguous(), d["draft_logits"][..., :500].contiguous(), 1.0, 1.0,
                  d["draft_tokens"], None, dev[:500].contiguous(), 0.1, d["uniforms"])
    assert e.value.code == -2
    call()                                           # and the unmodified call is fine
    torch.cuda.synchronize()
