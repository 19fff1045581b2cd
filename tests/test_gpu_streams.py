"""Stream semantics of the C ABI on the GPU: every call enqueues on the caller's stream and nothing else,
so it can run on a side stream and be captured into a CUDA graph and replayed on new inputs (the way a
serving loop removes launch overhead from the small, latency-bound calls).  Compared with plain calls
of the same library on the same inputs: bit-exact, integers and floats alike."""
import pytest
import torch

from paper_2510_26527_b200 import binding, buildlib, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
KEYS = ("accepted_len", "block_len", "out_len", "out_tokens")


@pytest.fixture(scope="module", autouse=True)
def _lib():
    buildlib.build()
    binding.load_library()
    assert torch.cuda.is_available()


def _chain_inputs(seed, B=24, V=20000):
    spec = synth.scaled(synth.config("cfg5", sigma=0.5), B=B, V=V)
    return synth.make_chain(spec, seed=seed, device=DEV)


def _plain_chain(d):
    out = binding.polyspec_verify_chain(d["models"], d["k"], d["draft_tokens"], d["uniforms"], d["temperature"])
    torch.cuda.synchronize()
    return {k: out[k].clone() for k in KEYS}


def test_chain_on_a_side_stream():
    d = _chain_inputs(51)
    want = _plain_chain(d)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    out = binding.polyspec_verify_chain(d["models"], d["k"], d["draft_tokens"], d["uniforms"], d["temperature"], stream=side)
    side.synchronize()
    for k in KEYS:
        assert torch.equal(out[k], want[k]), k
    assert int(out["device_status"][0]) == 0


def test_chain_call_captured_in_a_graph_and_replayed_on_new_inputs():
    a, b = _chain_inputs(52), _chain_inputs(53)
    want_a, want_b = _plain_chain(a), _plain_chain(b)
    # the call's own static buffers, refilled before every replay
    call = binding.ChainCall([m.clone() for m in a["models"]], a["k"], a["draft_tokens"].clone(), a["uniforms"].clone(), a["temperature"])
    call.launch()                                   # one plain call first: one-time kernel attributes are set outside the capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        call.launch()
    for d, want in ((a, want_a), (b, want_b), (a, want_a)):
        for dst, src in zip(call.models, d["models"]):
            dst.copy_(src)
        call.draft_tokens.copy_(d["draft_tokens"])
        call.uniforms.copy_(d["uniforms"])
        for k in KEYS:
            call.out[k].fill_(-7)
        graph.replay()
        torch.cuda.synchronize()
        for k in KEYS:
            assert torch.equal(call.out[k], want[k]), k
        assert int(call.device_status[0]) == 0


def test_greedy_chain_captured_in_a_graph():
    d = _chain_inputs(54)
    want = binding.polyspec_verify_chain_greedy(d["models"], d["k"], d["draft_tokens"])
    torch.cuda.synchronize()
    rows = [int(m.shape[1]) for m in d["models"][:-1]] + [int(d["k"][-1])]
    B, _, V = d["models"][0].shape
    nbytes = binding.polyspec_verify_chain_greedy_workspace(d["k"], rows, B, V, binding.BF16)
    workspace = torch.empty(nbytes, dtype=torch.uint8, device=DEV)
    out = binding.chain_outputs(len(d["models"]) - 1, B, max(d["k"]), torch.device(DEV))
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        binding.polyspec_verify_chain_greedy(d["models"], d["k"], d["draft_tokens"], workspace=workspace, out=out, device_status=status)
    for k in KEYS:
        out[k].fill_(-7)
    graph.replay()
    torch.cuda.synchronize()
    for k in KEYS:
        assert torch.equal(out[k], want[k]), k


def test_fused_call_captured_in_a_graph_and_replayed_on_new_inputs():
    spec = synth.FusedSpec(B=8, k=4, V=4096, d_p=512, d_q=256)
    a = synth.make_fused(spec, seed=55, device=DEV)
    b = synth.make_fused(spec, seed=56, device=DEV)

    def plain(d):
        out = binding.polyspec_verify_from_hidden(d["hidden_p"], d["W_p"], d["hidden_q"], d["W_q"], d["draft_tokens"], d["uniforms"],
                                                  d["temperature"])
        torch.cuda.synchronize()
        return {k: out[k].clone() for k in ("accepted_len", "next_token")}

    want_a, want_b = plain(a), plain(b)
    call = binding.FusedCall(*[a[n].clone() for n in ("hidden_p", "W_p", "hidden_q", "W_q", "draft_tokens", "uniforms")], a["temperature"])
    call.launch()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        call.launch()
    names = ("hidden_p", "W_p", "hidden_q", "W_q", "draft_tokens", "uniforms")
    for d, want in ((b, want_b), (a, want_a)):
        for dst, name in zip(call.t, names):
            dst.copy_(d[name])
        for k in want:
            call.out[k].fill_(-7)
        graph.replay()
        torch.cuda.synchronize()
        for k in want:
            assert torch.equal(call.out[k], want[k]), k
        assert int(call.device_status[0]) == 0
