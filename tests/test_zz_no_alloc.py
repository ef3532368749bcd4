"""The allocation-free beta calibration (moe_calibrate_beta_noalloc) against the regular entry
point.  It exists for callers that cannot allocate device memory while running (their own pool
owns the GPU, or they cannot take cudaMalloc's device-wide synchronisation); its scratch is a
fixed array inside the library.  Two calls in a row share that array, so the second call, on
other tokens and a shorter batch, must not see anything of the first.  Collected last on
purpose: a run that stops at the first failure has then already run every other test."""
import ctypes

import pytest
import torch

from paper_2402_14800_b200 import binding, build, synth

pytestmark = pytest.mark.gpu

H, F, E = 128, 448, 8
DEV = "cuda:0"


def test_noalloc_calibration_matches_the_allocating_entry_point_twice():
    build.build()
    W = synth.make_layer_weights(H, F, E, seed=0)
    Wg = W.W_gate.to(DEV)
    layer = binding.MoeLayer(Wg, W.W1.to(DEV), W.W3.to(DEV), W.W2.to(DEV))
    pruned_rows = torch.tensor([0, 2, 3, 5, 6, 7], device=DEV)
    pruned = binding.MoeLayer(Wg, W.W1.to(DEV), W.W3.to(DEV), W.W2.to(DEV), 0b11101101)
    cases = [(4097, 3, layer, Wg), (1000, 4, pruned, Wg[pruned_rows].contiguous())]
    # the first call on a device is the documented warm-up (it may load this part of the library
    # onto the device); what is promised is that the calls after it take no device memory
    binding.calibrate_beta_noalloc(Wg, synth.make_tokens(64, H, seed=9).to(DEV))
    for T, seed, ref_layer, rows in cases:
        x = synth.make_tokens(T, H, seed=seed).to(DEV)
        want = ref_layer.calibrate_beta(x)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info(DEV)[0]
        got = binding.calibrate_beta_noalloc(rows, x)
        assert torch.cuda.mem_get_info(DEV)[0] >= free_before, "the call took device memory"
        assert abs(got - want) <= 2e-6 * max(1.0, abs(want)), (T, got, want)
    layer.close()
    pruned.close()


def test_noalloc_calibration_rejects_batches_beyond_the_static_scratch():
    build.build()
    lib = binding.load_library()
    x = torch.zeros((8, H), dtype=torch.bfloat16, device=DEV)
    wg = torch.zeros((E, H), dtype=torch.bfloat16, device=DEV)
    out = ctypes.c_float(0)
    rc = lib.moe_calibrate_beta_noalloc(wg.data_ptr(), x.data_ptr(), 16385, H, E, None, ctypes.byref(out))
    assert rc == -1 and "16384" in binding.last_error()
    assert lib.moe_calibrate_beta_noalloc(wg.data_ptr(), x.data_ptr(), 8, H, 1, None, ctypes.byref(out)) == -1
    assert lib.moe_calibrate_beta_noalloc(None, x.data_ptr(), 8, H, E, None, ctypes.byref(out)) == -1
