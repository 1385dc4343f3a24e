"""The device entry points only launch kernels (no allocation, no synchronisation), so a step can be captured
into a CUDA graph and replayed: the replays must reproduce the bits of the direct calls."""
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from test_gpu_parity import dq  # noqa: E402,F401


def test_a_captured_step_replays_bit_identically(dq):
    B = dq.binding
    n, bucket, W, step = 3_000_000 + 40, 2048, 4, 5
    pd = B.make_params(bucket, 3, 5, 0, 0.0, 0.0)
    pn = B.make_params(bucket, 2, 0, 4, 2.0, 1.0, 32, dq.DQ_FLAG_INPUT_READY | dq.DQ_FLAG_OUTPUT_FREE)
    dev = torch.device("cuda")
    gen = torch.Generator(device="cuda").manual_seed(11)
    grads = [torch.randn(n, device=dev, generator=gen) * 0.01 for _ in range(W)]
    bufs = [B.alloc_message(n, pd if w == 0 else pn, dev) for w in range(W)]
    out = torch.empty(n, device=dev)
    msgs = [dq.Message(pk, sc, 100 + w, w, dq.DQ_KIND_DQSG if w == 0 else dq.DQ_KIND_NDQSG, pd if w == 0 else pn)
            for w, (pk, sc) in enumerate(bufs)]

    def one_step():
        for w in range(W):
            fn = dq.dqsg_encode if w == 0 else dq.ndqsg_encode
            fn(grads[w], 100 + w, w, step, pd if w == 0 else pn, *bufs[w])
        dq.ndqsg_decode_aggregate_side_first(msgs, n, step, out)

    one_step()                                   # also the first call per kernel, which sets function attributes
    torch.cuda.synchronize()
    want_out = out.clone()
    want_msgs = [(pk.clone(), sc.clone()) for pk, sc in bufs]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        one_step()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        one_step()
    for _ in range(3):
        out.zero_()
        for pk, sc in bufs:
            pk.zero_()
            sc.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, want_out)
        for (pk, sc), (wpk, wsc) in zip(bufs, want_msgs):
            assert torch.equal(pk, wpk) and torch.equal(sc, wsc)
    assert dq.device_error_flags() == 0
