"""GPU: calls issued on several streams at once, each with its own scratch, give bit for bit what
the same calls give one after the other on one stream (the schedule `bench.py` uses)."""
import pytest
import torch

from paper_2503_20354_b200 import binding as B
from paper_2503_20354_b200 import workloads as W

pytestmark = pytest.mark.gpu

LAYERS = [
    W.conv("s_3x3", 4, 72, 16, 96, 3),
    W.conv("s_1x1", 4, 136, 14, 64, 1, 1, 0),
    W.conv("s_3x3s2", 3, 40, 28, 48, 3, 2),
    W.linear("s_lin", 300, 256, 384, dist="normal", dt=W.F32),
    W.conv("s_1x1s2", 2, 64, 28, 72, 1, 2, 0),
    W.conv("s_7x7", 2, 3, 64, 32, 7, 2, 3, dist="normal"),
]


def _run(streams):
    n = len(streams) if streams else 1
    xs = [W.activation(l, 20 + i).cuda() for i, l in enumerate(LAYERS)]
    gs = [W.grad_out(l, 20 + i).cuda() for i, l in enumerate(LAYERS)]
    descs = [B.layer_desc(l, B.PATH_TENSOR_CORE) for l in LAYERS]
    stores = [B.CompressedActivation(l.n_act, l.dt, 0.0, "cuda") for l in LAYERS]
    ws_bytes = max(max(s.sizes.workspace_bytes for s in stores),
                   max(B.surgeon_weight_grad_workspace(d) for d in descs), 256)
    ws = [torch.empty(ws_bytes, dtype=torch.uint8, device="cuda") for _ in range(n)]
    dws = [torch.empty(l.dw_shape, dtype=torch.float32, device="cuda") for l in LAYERS]
    torch.cuda.synchronize()
    main = torch.cuda.current_stream()
    for rep in range(3):                                   # several rounds: scratch is reused
        for st in streams:
            st.wait_stream(main)
        for i in range(len(LAYERS)):
            B.surgeon_prune_compact(xs[i], 0.6, out=stores[i], workspace=ws[i % n],
                                    stream=streams[i % n] if streams else None)
        for st in streams:
            main.wait_stream(st)
        for st in streams:
            st.wait_stream(main)
        for j, i in enumerate(reversed(range(len(LAYERS)))):
            B.surgeon_weight_grad(stores[i], descs[i], gs[i], dw=dws[i], workspace=ws[j % n],
                                  stream=streams[j % n] if streams else None)
        for st in streams:
            main.wait_stream(st)
    torch.cuda.synchronize()
    for s in stores:
        assert s.read_header().status == 0
    return [s.to_numpy() for s in stores], [d.cpu() for d in dws]


def test_streams_match_serial():
    stores1, dws1 = _run([])
    stores4, dws4 = _run([torch.cuda.Stream() for _ in range(4)])
    for a, b in zip(stores1, stores4):
        for u, v in zip(a[:3], b[:3]):
            assert (u == v).all()
        assert bytes(a[3]) == bytes(b[3])
    for a, b in zip(dws1, dws4):
        assert torch.equal(a, b)
