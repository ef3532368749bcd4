"""The library's error paths on the GPU, driven without faulting, trapping or hanging it.

A bounded wait that runs out: a one-CTA kernel of the library waits, with the grouped GEMMs' own
wait routine and a limit of a millisecond, on a barrier nobody arrives on; it then takes the
GEMMs' abort path (drain, release of tensor memory, status word).  The host must report
MOE_ERR_DEVICE_TIMEOUT once, clean up what an aborted GEMM may leave behind, and the handle must
work afterwards.  Scratch that does not fit: the library's view of free device memory is capped
by a host-side hook, so MOE_ERR_OOM comes back without filling the device."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2402_14800_b200 import binding, build, synth
from tests import parity as P

pytestmark = pytest.mark.gpu

H, F, E = 128, 448, 8
DEV = "cuda:0"
MOE_ERR_OOM, MOE_ERR_DEVICE_TIMEOUT = -4, -5


@pytest.fixture(scope="module")
def tiny():
    build.build()
    W = synth.make_layer_weights(H, F, E, seed=0)
    b = synth.bf16_bits
    host = dict(Wg=b(W.W_gate), W1=b(W.W1), W3=b(W.W3), W2=b(W.W2))
    dev = [t.to(DEV) for t in (W.W_gate, W.W1, W.W3, W.W2)]
    return host, dev


def check_against_oracle(layer, host, T, kept, beta, seed):
    x = synth.make_tokens(T, H, seed=seed)
    xb = synth.bf16_bits(x)
    ora = O.moe_forward(xb, host["Wg"], host["W1"], host["W3"], host["W2"], kept, beta)
    ora["logits"] = O.route(xb, host["Wg"], kept, beta)["logits"]
    stats = binding.RoutingStats(T, E, DEV)
    y = layer.forward(x.to(DEV), beta, stats=stats)
    torch.cuda.synchronize()
    gi, gs = stats.idx.cpu().numpy(), stats.skipped.cpu().numpy()
    P.check_routing(gi, gs, stats.wn.cpu().numpy(), stats.ratio.cpu().numpy(), ora, kept, beta)
    P.check_outputs(synth.bf16_bits(y), ora["y"], (gi == ora["idx"]).all(1) & (gs == ora["skipped"]))


@pytest.mark.parametrize("poison_tail", [0, 1])
def test_an_expired_wait_is_reported_once_and_the_handle_recovers(tiny, poison_tail):
    host, dev = tiny
    lib = binding.load_library()
    layer = binding.MoeLayer(*dev)
    check_against_oracle(layer, host, 40, 0xFF, 0.3, seed=1)   # scratch, K-slice counters in use
    assert layer.device_status() == 0
    assert lib.moe_test_wait_expiry(layer._h, 1000, poison_tail) == 0
    assert layer.device_status() == MOE_ERR_DEVICE_TIMEOUT
    assert "bounded wait" in binding.last_error()
    assert layer.device_status() == 0                          # reported once, then clear
    # the context and the handle are intact: small-batch (K-sliced), large-batch and search paths
    for T in (40, 7, 700):
        check_against_oracle(layer, host, T, 0xFF, 0.3, seed=2 + T)
    x = synth.make_tokens(256, H, seed=0)
    losses, best = layer.prune_search(x.to(DEV), 6)
    P.check_search(losses, best, O.prune_search_allexperts(synth.bf16_bits(x), host["Wg"], host["W1"],
                                                           host["W3"], host["W2"], 6))
    assert layer.device_status() == 0
    layer.close()


def test_an_expired_wait_surfaces_through_the_calls_that_return_to_the_host(tiny):
    host, dev = tiny
    lib = binding.load_library()
    layer = binding.MoeLayer(*dev)
    x = synth.make_tokens(64, H, seed=3)
    xh = x.pin_memory()
    yh = torch.empty_like(xh).pin_memory()
    assert lib.moe_test_wait_expiry(layer._h, 500, 0) == 0
    with pytest.raises(binding.MoeError) as e:
        layer.forward_host(xh, 0.3, yh)                       # reads the status word before returning
    assert e.value.code == MOE_ERR_DEVICE_TIMEOUT
    layer.forward_host(xh, 0.3, yh)
    assert torch.equal(yh, layer.forward(x.to(DEV), 0.3).cpu())
    assert lib.moe_test_wait_expiry(layer._h, 500, 0) == 0
    with pytest.raises(binding.MoeError) as e:
        layer.prune_search(x.to(DEV), 6)
    assert e.value.code == MOE_ERR_DEVICE_TIMEOUT
    assert layer.device_status() == 0
    assert lib.moe_test_wait_expiry(layer._h, 0, 0) == -1 and lib.moe_test_wait_expiry(layer._h, 200000, 0) == -1
    layer.close()


def test_scratch_that_does_not_fit_is_an_error_and_the_handle_stays_usable(tiny):
    host, dev = tiny
    lib = binding.load_library()
    layer = binding.MoeLayer(*dev)
    check_against_oracle(layer, host, 64, 0xFF, 0.3, seed=4)
    try:
        lib.moe_test_set_free_bytes_limit(1 << 20)            # the library sees 1 MiB free
        with pytest.raises(binding.MoeError) as e:
            layer.forward(synth.make_tokens(4096, H, seed=5).to(DEV), 0.3)
        assert e.value.code == MOE_ERR_OOM and "does not fit" in str(e.value)
        with pytest.raises(binding.MoeError) as e:
            layer.reserve(100000)
        assert e.value.code == MOE_ERR_OOM
        with pytest.raises(binding.MoeError) as e:
            binding.MoeLayer(*dev)                            # weights of a new handle do not fit either
        assert "do not fit" in str(e.value)
    finally:
        lib.moe_test_set_free_bytes_limit(-1)
    # buffers that failed to grow are gone; the next calls grow them again
    for T in (64, 4096, 5):
        check_against_oracle(layer, host, T, 0xFF, 0.3, seed=6 + T)
    assert layer.device_status() == 0
    layer.close()
