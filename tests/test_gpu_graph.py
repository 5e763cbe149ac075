"""The whole linear-layer step (casts + three GEMMs) captured once in a CUDA graph and replayed:
the library makes no host synchronisation, allocation or host-side read of device scalars on the way,
and a replay on new input values gives exactly what eager calls give."""
import pytest
import torch

from paper_2209_05433_b200 import api, synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _step(X, W, dY, buf, fused):
    T, I = X.shape
    O = W.shape[1]
    s = buf["scal"]
    ax, sx, six, aw, sw, siw, ag, sg, sig, ay, adx, adw = [s[i:i + 1] for i in range(12)]
    if fused:
        api.fp8_quantize_current(X, api.E4M3, buf["Xq"], ax, sx, six)
        api.fp8_quantize_current(W, api.E4M3, buf["Wq"], aw, sw, siw)
        api.fp8_quantize_current(dY, api.E5M2, buf["Gq"], ag, sg, sig)
    else:
        for t, q, fmt, a, sc, si in ((X, buf["Xq"], api.E4M3, ax, sx, six), (W, buf["Wq"], api.E4M3, aw, sw, siw),
                                     (dY, buf["Gq"], api.E5M2, ag, sg, sig)):
            api.fp8_amax(t, a)
            api.fp8_scale_from_amax(a, fmt, sc, si)
            api.fp8_quantize(t, fmt, sc, q)
    api.fp8_gemm(buf["Xq"], api.E4M3, api.MAJOR_K, buf["Wq"], api.E4M3, api.MAJOR_MN, buf["Y"], six, siw, ay)
    api.fp8_gemm(buf["Gq"], api.E5M2, api.MAJOR_K, buf["Wq"], api.E4M3, api.MAJOR_K, buf["dX"], sig, siw, adx)
    api.fp8_gemm(buf["Xq"], api.E4M3, api.MAJOR_MN, buf["Gq"], api.E5M2, api.MAJOR_MN, buf["dW"], six, sig, adw)


def _buffers(T, I, O):
    u8, bf = torch.uint8, torch.bfloat16
    return {"Xq": torch.empty(T, I, dtype=u8, device=DEV), "Wq": torch.empty(I, O, dtype=u8, device=DEV),
            "Gq": torch.empty(T, O, dtype=u8, device=DEV), "Y": torch.empty(T, O, dtype=bf, device=DEV),
            "dX": torch.empty(T, I, dtype=bf, device=DEV), "dW": torch.empty(I, O, dtype=bf, device=DEV),
            "scal": torch.zeros(16, dtype=torch.float32, device=DEV)}


@pytest.mark.parametrize("fused", [False, True])
def test_step_replays_from_a_cuda_graph(fused):
    T, I, O = 512, 384, 768
    X = synth.activations(T * I, 3, device=DEV).view(T, I)
    W = synth.weights(I * O, 3, 0.02, device=DEV).view(I, O)
    dY = synth.gradients(T * O, 4, device=DEV).view(T, O)
    graph_buf, eager_buf = _buffers(T, I, O), _buffers(T, I, O)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        api.current_scaling_workspace(X.device)            # the workspace of this stream exists before the capture
        _step(X, W, dY, graph_buf, fused)                   # warm-up outside the capture (first-use set-up)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            _step(X, W, dY, graph_buf, fused)
    torch.cuda.synchronize()
    for trial in range(2):
        # new values in the same input buffers, then replay
        X.copy_(synth.activations(T * I, 30 + trial, device=DEV).view(T, I))
        dY.copy_(synth.gradients(T * O, 40 + trial, device=DEV).view(T, O) * (3.0 + trial))
        g.replay()
        _step(X, W, dY, eager_buf, fused)
        torch.cuda.synchronize()
        assert api.fp8_async_status()[0] == 0
        for k in graph_buf:
            assert torch.equal(graph_buf[k].view(torch.uint8), eager_buf[k].view(torch.uint8)), (k, trial)


def test_rows_beyond_the_core_path_replay_from_a_cuda_graph():
    """quantize + transposed copy, the K-major weight-gradient GEMM on the transposed codes with split
    accumulation, an FP8-output GEMM and a batched GEMM, captured once and replayed on new values"""
    T, I, O = 2304, 256, 384                      # the weight gradient contracts over T = 2304: two chunks of K
    X = synth.activations(T * I, 5, device=DEV).view(T, I)
    dY = synth.gradients(T * O, 6, device=DEV).view(T, O)
    u8, f32 = torch.uint8, torch.float32

    def buffers():
        return {"Xq": torch.empty(T, I, dtype=u8, device=DEV), "XqT": torch.empty(I, T, dtype=u8, device=DEV),
                "Gq": torch.empty(T, O, dtype=u8, device=DEV), "GqT": torch.empty(O, T, dtype=u8, device=DEV),
                "dW": torch.empty(I, O, dtype=f32, device=DEV), "dWq": torch.empty(I, O, dtype=u8, device=DEV),
                "P": torch.empty(3, I, O, dtype=torch.bfloat16, device=DEV), "scal": torch.zeros(8, dtype=f32, device=DEV)}

    sx, sg = torch.tensor([2.0], device=DEV), torch.tensor([4096.0], device=DEV)
    six, sig, sd = torch.tensor([0.5], device=DEV), torch.tensor([1.0 / 4096.0], device=DEV), torch.tensor([8.0], device=DEV)

    def step(b):
        s = b["scal"]
        api.fp8_quantize_transpose(X, api.E4M3, sx, b["Xq"], b["XqT"], s[0:1])
        api.fp8_quantize_transpose(dY, api.E5M2, sg, b["Gq"], b["GqT"], s[1:2])
        api.fp8_gemm(b["XqT"], api.E4M3, api.MAJOR_K, b["GqT"], api.E5M2, api.MAJOR_K, b["dW"], six, sig, s[2:3], acc=api.ACC_SPLIT)
        api.fp8_gemm_fp8out(b["XqT"], api.E4M3, api.MAJOR_K, b["GqT"], api.E5M2, api.MAJOR_K, b["dWq"], api.E4M3, six, sig, sd, s[3:4],
                            acc=api.ACC_SPLIT)
        A3 = b["XqT"].view(I, 3, T // 3).permute(1, 0, 2)          # three K-slices as batch members (pitched views)
        B3 = b["GqT"].view(O, 3, T // 3).permute(1, 0, 2)
        api.fp8_gemm_batched(A3, api.E4M3, api.MAJOR_K, B3, api.E5M2, api.MAJOR_K, b["P"], six, sig, s[4:5])

    gb, eb = buffers(), buffers()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        step(gb)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            step(gb)
    torch.cuda.synchronize()
    for trial in range(2):
        X.copy_(synth.activations(T * I, 50 + trial, device=DEV).view(T, I))
        dY.copy_(synth.gradients(T * O, 60 + trial, device=DEV).view(T, O) * (2.0 + trial))
        g.replay()
        step(eb)
        torch.cuda.synchronize()
        assert api.fp8_async_status()[0] == 0
        for k in gb:
            assert torch.equal(gb[k].view(u8), eb[k].view(u8)), (k, trial)
    # the three K-slices add up to the whole weight-gradient product (bf16 partial results, loose check)
    total = eb["P"].float().sum(0)
    assert torch.allclose(total, eb["dW"], rtol=2e-2, atol=2e-2 * float(eb["dW"].abs().max()))


def test_two_streams_run_independent_steps_concurrently():
    """two steps on two streams at once (separate buffers, separate current-scaling workspaces): each gives
    what it gives alone"""
    T, I, O = 640, 512, 768
    inputs = []
    for k in range(2):
        inputs.append((synth.activations(T * I, 70 + k, device=DEV).view(T, I), synth.weights(I * O, 70 + k, 0.02, device=DEV).view(I, O),
                       synth.gradients(T * O, 80 + k, device=DEV).view(T, O)))
    alone = []
    for X, W, dY in inputs:
        b = _buffers(T, I, O)
        _step(X, W, dY, b, True)
        alone.append(b)
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    together = [_buffers(T, I, O), _buffers(T, I, O)]
    for rep in range(5):
        for k, st in enumerate(streams):
            with torch.cuda.stream(st):
                _step(*inputs[k], together[k], True)
    torch.cuda.synchronize()
    assert api.fp8_async_status()[0] == 0
    for k in range(2):
        for name in alone[k]:
            assert torch.equal(alone[k][name].view(torch.uint8), together[k][name].view(torch.uint8)), (k, name)
