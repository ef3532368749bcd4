"""Alternative code paths behind switches, checked against the default path on the GPU:
the CUDA-core debug kernels, the dense (all experts) search, and replay of a captured CUDA
graph of moe_forward."""
import os

import numpy as np
import pytest
import torch

from paper_2402_14800_b200 import binding, build, synth

pytestmark = pytest.mark.gpu

H, F, E = 128, 448, 8
DEV = "cuda:0"


@pytest.fixture(scope="module")
def weights():
    build.build()
    W = synth.make_layer_weights(H, F, E, seed=0)
    return [t.to(DEV) for t in (W.W_gate, W.W1, W.W3, W.W2)]


def layer_with_env(weights, kept=0xFF, **env):
    """The switches are read when a handle is created."""
    old = {k: os.environ.get(k) for k in env}
    os.environ.update({k: str(v) for k, v in env.items()})
    try:
        return binding.MoeLayer(*weights, kept)
    finally:
        for k, v in old.items():
            if v is None:
                os.environ.pop(k, None)
            else:
                os.environ[k] = v


def rel_l2(a, b):
    """Worst per-token relative L2 distance between two bf16 outputs."""
    a, b = a.double().cpu().numpy(), b.double().cpu().numpy()
    return float((np.linalg.norm(a - b, axis=1) / np.linalg.norm(b, axis=1)).max())


@pytest.mark.parametrize("T", [40, 700])
def test_debug_cuda_core_kernels_agree_with_tensor_core_path(weights, T):
    x = synth.make_tokens(T, H, seed=3).to(DEV)
    ref = binding.MoeLayer(*weights, 0b11011101)
    dbg = layer_with_env(weights, 0b11011101, MOE_DEBUG_SIMT=1)
    y0, y1 = ref.forward(x, 0.4), dbg.forward(x, 0.4)
    torch.cuda.synchronize()
    assert rel_l2(y1, y0) < 5e-3  # different summation orders, same rounding points
    ref.close()
    dbg.close()


@pytest.mark.parametrize("T", [1, 5, 40, 150, 256])
def test_both_small_batch_gemms_at_every_size(weights, T):
    # by default the batch size picks the kernel of a small batch; each one is forced here over
    # the whole range and compared with the CUDA-core kernels
    x = synth.make_tokens(T, H, seed=6).to(DEV)
    dbg = layer_with_env(weights, 0b01111011, MOE_DEBUG_SIMT=1)
    y0 = dbg.forward(x, 0.3)
    for kernel in ("wm", "td"):
        lay = layer_with_env(weights, 0b01111011, MOE_DECODE_KERNEL=kernel)
        y1 = lay.forward(x, 0.3)
        y2 = lay.forward(x, 0.3)
        torch.cuda.synchronize()
        assert rel_l2(y1, y0) < 5e-3
        assert torch.equal(y1, y2)
        assert lay.device_status() == 0
        lay.close()
    dbg.close()


@pytest.mark.parametrize("beta", [0.0, 0.6])
def test_single_token_kernels_agree_with_gemm_path(weights, beta):
    # T = 1 runs matrix-vector kernels by default; MOE_SINGLE_KERNEL=gemm keeps the grouped GEMMs
    gemv = binding.MoeLayer(*weights, 0b11110110)
    gemm = layer_with_env(weights, 0b11110110, MOE_SINGLE_KERNEL="gemm")
    for seed in range(8):
        x = synth.make_tokens(1, H, seed=50 + seed).to(DEV)
        res = synth.make_tokens(1, H, seed=90 + seed).to(DEV) if seed % 2 else None
        y0 = gemm.forward(x, beta, residual=res)
        y1 = gemv.forward(x, beta, residual=res)
        y2 = gemv.forward(x, beta, residual=res)
        torch.cuda.synchronize()
        assert rel_l2(y1, y0) < 5e-3  # different summation orders, same rounding points
        assert torch.equal(y1, y2)
    assert gemv.device_status() == 0 and gemm.device_status() == 0
    gemv.close()
    gemm.close()


@pytest.mark.parametrize("r", [6, 4, 7])
def test_dense_search_equals_pruned_work_search(weights, r):
    x = synth.make_tokens(777, H, seed=4).to(DEV)
    fast = binding.MoeLayer(*weights)
    dense = layer_with_env(weights, MOE_SEARCH_DENSE=1)
    l0, b0 = fast.prune_search(x, r)
    l1, b1 = dense.prune_search(x, r)
    fast.close()
    dense.close()
    np.testing.assert_allclose(l0, l1, rtol=1e-6)
    assert b0 == b1


@pytest.mark.parametrize("T", [1, 16, 600])
def test_forward_replays_from_a_cuda_graph(weights, T):
    layer = binding.MoeLayer(*weights)
    x = synth.make_tokens(T, H, seed=6).to(DEV)
    y = torch.empty_like(x)
    s = torch.cuda.Stream(DEV)
    layer.set_stream(s)
    with torch.cuda.stream(s):
        layer.forward(x, 0.4, y=y)          # first call grows the scratch, outside the capture
        s.synchronize()
        want = y.clone()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            layer.forward(x, 0.4, y=y)
        x2 = synth.make_tokens(T, H, seed=7).to(DEV)
        y.zero_()
        g.replay()
        s.synchronize()
        assert torch.equal(y, want)
        x.copy_(x2)                          # same buffers, new contents
        g.replay()
        s.synchronize()
        fresh = layer.forward(x2, 0.4)
        s.synchronize()
        assert torch.equal(y, fresh)
    layer.close()


@pytest.mark.parametrize("T", [1, 2, 8, 40, 128, 600])
def test_back_to_back_calls_with_changing_inputs_equal_isolated_calls(weights, T):
    # Serving pattern: the same buffers, new contents every step, the calls queued without a
    # synchronisation in between (the kernels of consecutive calls overlap through programmatic
    # dependent launch).  Every step must give what the same input gives in an isolated call.
    n = 12
    layer = binding.MoeLayer(*weights, 0b11110111)
    xs = [synth.make_tokens(T, H, seed=200 + i).to(DEV) for i in range(n)]
    want = []
    for x in xs:
        want.append(layer.forward(x, 0.4).clone())
        torch.cuda.synchronize()
    x_buf = torch.empty_like(xs[0])
    ys = [torch.empty_like(xs[0]) for _ in range(n)]
    for rep in range(3):
        for i in range(n):
            x_buf.copy_(xs[i])
            layer.forward(x_buf, 0.4, y=ys[i])
        torch.cuda.synchronize()
        for i in range(n):
            assert torch.equal(ys[i], want[i]), "step %d of round %d differs from the isolated call" % (i, rep)
    assert layer.device_status() == 0
    layer.close()


STACK_SPECS = [(20, 0xFF, 0.0), (21, 0b10111011, 0.4), (22, 0b00111100, 0.5)]


@pytest.fixture(scope="module")
def stack_layers():
    build.build()
    layers = []
    for seed, kept, _ in STACK_SPECS:
        W = synth.make_layer_weights(H, F, E, seed=seed)
        layers.append(binding.MoeLayer(W.W_gate.to(DEV), W.W1.to(DEV), W.W3.to(DEV), W.W2.to(DEV), kept))
    for l in layers[1:]:
        l.share_scratch(layers[0])
    yield layers
    for l in reversed(layers):
        l.close()


@pytest.mark.parametrize("T", [1, 16, 128, 600])
def test_queued_stack_steps_equal_isolated_calls(stack_layers, T):
    # Three layers out of one set of scratch, every kernel a programmatic dependent of the one
    # before, the state buffer read as the residual and overwritten by the same launch from the
    # second layer on.  Steps are queued without synchronising, once on one refilled input buffer
    # and once on separate inputs with no other kernel between two steps; each must reproduce the
    # isolated call bit for bit.
    n = 8
    betas = [s[2] for s in STACK_SPECS]
    xs = [synth.make_tokens(T, H, seed=400 + i).to(DEV) for i in range(n)]
    want = []
    for x in xs:
        want.append(binding.stack_forward(stack_layers, x, betas, 1e-5).clone())
        torch.cuda.synchronize()
    x_buf = torch.empty_like(xs[0])
    ys = [torch.empty_like(xs[0]) for _ in range(n)]
    for rep in range(6 if T <= 128 else 3):
        for i in range(n):
            if rep % 2 == 0:
                x_buf.copy_(xs[i])
                binding.stack_forward(stack_layers, x_buf, betas, 1e-5, y=ys[i])
            else:
                binding.stack_forward(stack_layers, xs[i], betas, 1e-5, y=ys[i])
        torch.cuda.synchronize()
        for i in range(n):
            assert torch.equal(ys[i], want[i]), "step %d of round %d differs from the isolated call" % (i, rep)
        for y in ys:
            y.zero_()
    assert stack_layers[0].device_status() == 0


@pytest.mark.parametrize("T", [1, 16, 128, 600])
def test_queued_residual_steps_with_y_aliasing_the_residual(weights, T):
    # state <- state + MoE(x) in place (y and residual are the same buffer), queued steps
    n = 8
    layer = binding.MoeLayer(*weights, 0b11110111)
    xs = [synth.make_tokens(T, H, seed=500 + i).to(DEV) for i in range(n)]
    s0 = synth.make_tokens(T, H, seed=599).to(DEV)
    want, state = [], s0.clone()
    for x in xs:
        state = layer.forward(x, 0.4, residual=state).clone()   # separate output buffer, isolated
        torch.cuda.synchronize()
        want.append(state)
    for rep in range(4):
        state = s0.clone()
        snaps = []
        for i in range(n):
            layer.forward(xs[i], 0.4, residual=state, y=state)
            if rep % 2 == 0:
                snaps.append(state.clone())
        torch.cuda.synchronize()
        assert torch.equal(state, want[-1]), "round %d" % rep
        for i, snap in enumerate(snaps):
            assert torch.equal(snap, want[i]), "step %d of round %d" % (i, rep)
    assert layer.device_status() == 0
    layer.close()


@pytest.mark.parametrize("T", [2, 5, 16, 64, 128])
def test_small_batches_repeat_many_queued_steps(weights, T):
    # the small-batch sequences (router, permutation + gather, two GEMMs, combine: five programmatic
    # dependents per step on the same scratch addresses) queued 200 steps deep on alternating inputs
    layer = binding.MoeLayer(*weights, 0b11110111)
    xa, xb = (synth.make_tokens(T, H, seed=s).to(DEV) for s in (610, 611))
    wa, wb = layer.forward(xa, 0.4).clone(), layer.forward(xb, 0.4).clone()
    torch.cuda.synchronize()
    ya, yb = torch.empty_like(xa), torch.empty_like(xa)
    bad = torch.zeros((), dtype=torch.int32, device=DEV)
    for i in range(200):
        if i % 2 == 0:
            layer.forward(xa, 0.4, y=ya)
            bad += (~torch.eq(ya, wa)).any().int()
        else:
            layer.forward(xb, 0.4, y=yb)
            bad += (~torch.eq(yb, wb)).any().int()
    torch.cuda.synchronize()
    assert int(bad.item()) == 0
    assert layer.device_status() == 0
    layer.close()


def test_reserve_makes_later_calls_allocation_free(weights):
    # after moe_reserve(T_max) no forward call with T <= T_max grows the scratch, so a capture
    # needs no warm-up call
    layer = binding.MoeLayer(*weights)
    layer.reserve(700)
    held = layer.scratch_bytes
    assert held > 0
    s = torch.cuda.Stream(DEV)
    layer.set_stream(s)
    with torch.cuda.stream(s):
        x = synth.make_tokens(700, H, seed=6).to(DEV)
        y = torch.empty_like(x)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):       # first forward call of the handle, inside a capture
            layer.forward(x, 0.4, y=y)
        g.replay()
        s.synchronize()
        got = y.clone()
        for T in (1, 2, 40, 256, 257, 700):
            layer.forward(x[:T].contiguous(), 0.4)
        s.synchronize()
        assert layer.scratch_bytes == held
        assert torch.equal(layer.forward(x, 0.4), got)
        s.synchronize()
    with pytest.raises(binding.MoeError):
        layer.reserve(0)
    layer.close()


@pytest.mark.parametrize("T", [1, 40, 700])
def test_plain_stream_order_gives_the_same_bits(weights, T):
    # MOE_NO_PDL=1: every kernel in plain stream order instead of as a programmatic dependent;
    # the overlap of launches must not change a single bit
    x = synth.make_tokens(T, H, seed=8).to(DEV)
    ref = binding.MoeLayer(*weights, 0b11011101)
    want = ref.forward(x, 0.4).clone()
    ref.close()
    plain = layer_with_env(weights, 0b11011101, MOE_NO_PDL=1)
    try:
        got = plain.forward(x, 0.4).clone()
        torch.cuda.synchronize()
        assert plain.device_status() == 0
    finally:
        plain.close()
        layer_with_env(weights, MOE_NO_PDL=0).close()  # the switch is process-wide: back to the default
    assert torch.equal(got, want)
