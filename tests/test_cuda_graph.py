"""The entry points enqueue on the caller's stream and neither allocate nor synchronize, so a serving loop can capture them
in a CUDA graph: a captured prefill (tensor-core layer kernel) followed by captured decode steps, replayed, gives the
results of the eager calls bit for bit. (The binding's output tensors come from the graph's private memory pool.)"""
import pytest

from paper_2509_18467_b200 import inputs as I

pytestmark = pytest.mark.gpu
NAMES = ["q", "k", "v", "gate", "w_q", "w_k", "W"]


def test_prefill_and_decode_replayed_from_a_graph():
    import torch
    from paper_2509_18467_b200 import api
    s = I.LayerShape(2, 300, 4, 2, 128, 128, dtype="bf16", config_id=91)
    x = I.make(s, NAMES)
    d = {n: api.to_device(v, "bf16") for n, v in x.items()}
    p = api.params(s.B, s.T, s.H, s.H_kv, 128, 128)
    p1 = api.params(s.B, 1, s.H, s.H_kv, 128, 128)
    tok = {n: d[n][:, -1].clone() for n in NAMES[:4]}

    def run():
        r = api.lawcat_layer_fwd(p, *[d[n] for n in NAMES])
        outs = [api.lawcat_decode_step(p1, *[tok[n] for n in NAMES[:4]], d["w_q"], d["w_k"], d["W"], r["S_T"], r["z_T"],
                                       r["cache_q"], r["cache_k"]) for _ in range(3)]
        return r, outs

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):   # warm-up on a side stream (function attributes, tensor maps)
        run()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    eager, eager_outs = run()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        cap, cap_outs = run()
    for t in list(cap.values()) + cap_outs:
        t.zero_()
    g.replay()
    torch.cuda.synchronize()
    for k in eager:
        assert torch.equal(cap[k], eager[k]), k
    for a, b in zip(cap_outs, eager_outs):
        assert torch.equal(a, b)
