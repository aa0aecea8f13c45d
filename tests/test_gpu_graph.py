"""The verification call inside a CUDA graph: it allocates nothing, reads nothing back and never waits for
the stream, so a stream capture records it whole.  A captured call is replayed on inputs rewritten in place
and must match the oracle on every replay (the scratch area is re-initialised by the call itself)."""
import numpy as np
import pytest
import torch

import lantern_inputs as li
import oracle
import paper_2410_03355_b200 as lt
from parity import assert_parity, compare, near_ceiling, to_device
from test_gpu_greedy import check_outputs

pytestmark = pytest.mark.gpu


def _capture(d, inp, table, delta, greedy, top_k):
    B, N = inp.B, inp.N
    i32 = dict(dtype=torch.int32, device="cuda")
    f32 = dict(dtype=torch.float32, device="cuda")
    out = lt.VerifyOutputs(accept_len=torch.empty(B, **i32), next_token=torch.empty(B, **i32),
                           accept_path=torch.empty((B, N), **i32), status=torch.empty(B, **i32),
                           node_qa=torch.empty((B, N), **f32), node_px=torch.empty((B, N), **f32),
                           node_m=torch.empty((B, N), **i32))
    ws = torch.empty(lt.verify_workspace_bytes(B, N, inp.V, table.shape[1], inp.dtype, top_k), dtype=torch.uint8,
                     device="cuda")
    ws.fill_(0xa5)

    def call():
        lt.verify(d["target_logits"], None if greedy else d["draft_logits"], inp.cfg_scale, 0.0 if greedy else inp.T,
                  d["draft_tokens"], d["tree_parents"], table, delta, None if greedy else d["uniforms"], out=out,
                  workspace=ws, stream=torch.cuda.current_stream(), top_k=top_k)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        call()                       # first use outside the capture: kernel attributes are set here
    side.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        call()
    return graph, out, ws


@pytest.mark.parametrize("tree,top_k", [(False, 0), (True, 0), (True, 50)])
def test_replays_of_a_captured_call_follow_their_inputs(tree, top_k):
    B, N, V, k, delta = 48, 9, 1024, 24, 0.25
    host = oracle.build_neighbors(li.codebook_gaussian(V, 8, seed=12), k)[0]
    table = torch.from_numpy(host).cuda()
    gen = dict(dtype=li.BF16, has_uncond=True, cfg_scale=3.0, rho=0.9, sigma_draft=0.6)
    first = li.verify_inputs(B, N, V, seed=101, parents=li.tree_parents(B, N, depth=4, seed=101) if tree else None,
                             **gen)
    d = to_device(first)
    graph, out, ws = _capture(d, first, table, delta, False, top_k)
    near = 0
    for seed in (101, 102, 103):
        inp = li.verify_inputs(B, N, V, seed=seed, parents=li.tree_parents(B, N, depth=4, seed=seed) if tree else None,
                               **gen)
        for name, t in to_device(inp).items():           # same buffers, new contents
            if t is not None:
                d[name].copy_(t)
        out.accept_len.fill_(-9)
        graph.replay()
        torch.cuda.synchronize()
        res = compare(inp, host, delta, out, top_k=top_k)
        assert_parity(res)
        near += res["near"]
        assert lt.last_status(ws) == int(np.bitwise_or.reduce(out.status.cpu().numpy()))
    assert near <= near_ceiling(3 * B)


def test_a_captured_greedy_call():
    B, N, V, k, delta = 40, 6, 1024, 24, 0.3
    host = oracle.build_neighbors(li.codebook_gaussian(V, 8, seed=12), k)[0]
    table = torch.from_numpy(host).cuda()
    gen = dict(dtype=li.BF16, has_uncond=True, cfg_scale=3.0, rho=0.9, sigma_draft=0.6)
    first = li.verify_inputs(B, N, V, seed=7, parents=li.tree_parents(B, N, depth=4, seed=7), **gen)
    d = to_device(first)
    graph, out, _ = _capture(d, first, table, delta, True, 0)
    for seed in (7, 8):
        inp = li.verify_inputs(B, N, V, seed=seed, parents=li.tree_parents(B, N, depth=4, seed=seed), **gen)
        for name, t in to_device(inp).items():
            if t is not None:
                d[name].copy_(t)
        out.node_px.zero_()
        graph.replay()
        torch.cuda.synchronize()
        check_outputs(inp, host, delta, out)
