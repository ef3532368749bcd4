"""GPU parity on the tiny configuration (h=128, f=448, E=8): the CUDA path through the C ABI
against the CPU oracle, element by element on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2402_14800_b200 import binding, build, synth
from tests import parity as P

pytestmark = pytest.mark.gpu

H, F, E = 128, 448, 8
FULL = (1 << E) - 1
DEV = "cuda:0"


@pytest.fixture(scope="module")
def setup():
    build.build()
    W = synth.make_layer_weights(H, F, E, seed=0)
    b = synth.bf16_bits
    host = dict(Wg=b(W.W_gate), W1=b(W.W1), W3=b(W.W3), W2=b(W.W2))
    dev = dict(Wg=W.W_gate.to(DEV), W1=W.W1.to(DEV), W3=W.W3.to(DEV), W2=W.W2.to(DEV))
    return host, dev


def make_layer(dev, kept=FULL):
    return binding.MoeLayer(dev["Wg"], dev["W1"], dev["W3"], dev["W2"], kept)


def run_case(host, dev, T, kept, beta, x_seed=0, residual=False):
    x = synth.make_tokens(T, H, seed=x_seed)
    xb = synth.bf16_bits(x)
    res = synth.make_tokens(T, H, seed=x_seed + 77) if residual else None
    ora = O.moe_forward(xb, host["Wg"], host["W1"], host["W3"], host["W2"], kept, beta,
                        residual=None if res is None else synth.bf16_bits(res))
    ora["logits"] = O.route(xb, host["Wg"], kept, beta)["logits"]
    layer = make_layer(dev, kept)
    stats = binding.RoutingStats(T, E, DEV)
    y = layer.forward(x.to(DEV), beta, stats=stats, residual=None if res is None else res.to(DEV))
    torch.cuda.synchronize()
    assert layer.device_status() == 0
    g_idx = stats.idx.cpu().numpy()
    g_sk = stats.skipped.cpu().numpy()
    g_wn = stats.wn.cpu().numpy()
    g_ratio = stats.ratio.cpu().numpy()
    n_tie, n_close = P.check_routing(g_idx, g_sk, g_wn, g_ratio, ora, kept, beta)
    comparable = (g_idx == ora["idx"]).all(1) & (g_sk == ora["skipped"])
    worst = P.check_outputs(synth.bf16_bits(y), ora["y"], comparable)
    # aggregate counters follow from the per-token record
    cnt = np.zeros((E, 2), np.int64)
    for s in range(2):
        run = np.ones(T, bool) if s == 0 else (g_sk == 0)
        np.add.at(cnt[:, s], g_idx[run, s], 1)
    assert np.array_equal(stats.count.cpu().numpy(), cnt)
    assert int(stats.n_skipped.item()) == int(g_sk.sum())
    assert int(stats.n_experts_touched.item()) == int((cnt.sum(1) > 0).sum())
    layer.close()
    return dict(ties=n_tie, close=n_close, worst=worst, y=y, comparable=comparable, ora=ora)


@pytest.mark.parametrize("T", [256, 1, 7, 64, 130, 255])
def test_forward_small_batches_beta0(setup, T):
    host, dev = setup
    r = run_case(host, dev, T, FULL, 0.0)
    assert r["ties"] <= max(2, T // 20)


@pytest.mark.parametrize("T", [257, 1000, 2048 + 37])
def test_forward_large_batches_beta0(setup, T):
    host, dev = setup
    r = run_case(host, dev, T, FULL, 0.0, x_seed=5)
    assert r["ties"] <= max(2, T // 20)


@pytest.mark.parametrize("T", [256, 1024])
def test_forward_median_beta_skips_half(setup, T):
    host, dev = setup
    x = synth.bf16_bits(synth.make_tokens(T, H, seed=0))
    beta = O.beta_median(O.route(x, host["Wg"], FULL, 0.0)["ratio"])
    r = run_case(host, dev, T, FULL, beta)
    assert abs(int(r["ora"]["skipped"].sum()) - T // 2) <= 1


@pytest.mark.parametrize("kept", [0b11011101, 0b01100110, 0b00000110])
@pytest.mark.parametrize("T", [256, 700])
def test_forward_pruned_with_skipping(setup, kept, T):
    host, dev = setup
    run_case(host, dev, T, kept, 0.45, x_seed=2)


def test_forward_residual_and_beta_above_one(setup):
    host, dev = setup
    r = run_case(host, dev, 256, FULL, 1.5, residual=True)
    assert r["ora"]["skipped"].all()
    run_case(host, dev, 600, FULL, 0.3, residual=True)


@pytest.mark.parametrize("kept", [FULL, 0b01100110, 0b00000110])
@pytest.mark.parametrize("beta", [0.0, 0.45, 1.5])
def test_forward_single_token(setup, kept, beta):
    # T = 1 runs the matrix-vector kernels: one or two experts, with and without the residual,
    # several tokens in turn so that different experts and both skip outcomes occur
    host, dev = setup
    skipped = []
    for seed in range(6):
        r = run_case(host, dev, 1, kept, beta, x_seed=40 + seed, residual=bool(seed % 2))
        skipped.append(bool(r["ora"]["skipped"][0]))
    if beta == 0.0:
        assert not any(skipped)
    if beta > 1.0:
        assert all(skipped)


def test_forward_is_deterministic_and_reuses_scratch(setup):
    host, dev = setup
    layer = make_layer(dev)
    outs = []
    for T in (1000, 32, 1000, 32):
        x = synth.make_tokens(T, H, seed=11).to(DEV)
        outs.append(layer.forward(x, 0.4).clone())
    torch.cuda.synchronize()
    assert torch.equal(outs[0], outs[2]) and torch.equal(outs[1], outs[3])
    assert layer.forward(torch.empty((0, H), dtype=torch.bfloat16, device=DEV)).shape[0] == 0
    layer.close()


def test_forward_host_matches_device_call(setup):
    host, dev = setup
    layer = make_layer(dev)
    x = synth.make_tokens(300, H, seed=4)
    y_dev = layer.forward(x.to(DEV), 0.4)
    xh = x.pin_memory()
    yh = torch.empty_like(xh).pin_memory()
    layer.forward_host(xh, 0.4, yh)
    assert torch.equal(yh, y_dev.cpu())
    layer.close()


def test_weight_bytes_follow_the_kept_experts(setup):
    host, dev = setup
    # the kept experts' three matrices, plus the router rows padded to 16 rows (the operand of the
    # tensor-core router)
    for kept in (FULL, 0b00111111, 0b00001111):
        layer = make_layer(dev, kept)
        assert layer.weight_bytes == bin(kept).count("1") * 3 * H * F * 2 + 16 * H * 2
        layer.close()


def test_argument_errors(setup):
    host, dev = setup
    layer = make_layer(dev, 0b00111111)
    x = synth.make_tokens(8, H, seed=0).to(DEV)
    with pytest.raises(binding.MoeError) as e:
        layer.prune_search(x, 4)
    assert e.value.code == -1 and "all 8 experts" in str(e.value)
    with pytest.raises(binding.MoeError):
        layer.forward(x, -1.0)
    with pytest.raises(binding.MoeError):
        layer.forward(x, 0.0, y=x)
    lib = binding.load_library()
    assert lib.moe_forward(layer._h, x.data_ptr(), (1 << 24) + 1, 0.0, x.data_ptr(), None) == -1
    assert lib.moe_forward(layer._h, x.data_ptr(), -3, 0.0, x.data_ptr(), None) == -1
    layer.close()
    full = make_layer(dev)
    for r in (1, 9):
        with pytest.raises(binding.MoeError):
            full.prune_search(x, r)
    full.close()


@pytest.mark.parametrize("T", [255, 256, 4097])
def test_calibrate_beta(setup, T):
    host, dev = setup
    x = synth.make_tokens(T, H, seed=3)
    ratio = O.route(synth.bf16_bits(x), host["Wg"], FULL, 0.0)["ratio"]
    want = O.beta_median(ratio)
    layer = make_layer(dev)
    got = layer.calibrate_beta(x.to(DEV))
    layer.close()
    assert abs(got - want) <= 2e-6 * max(1.0, abs(want))


@pytest.mark.parametrize("T", [256, 700])
def test_prune_search_multi_equals_one_search_per_size(setup, T):
    # several subset sizes over one evaluation of the experts: same losses, same argmin as a
    # separate search per size, and the oracle's
    host, dev = setup
    x = synth.make_tokens(T, H, seed=5)
    layer = make_layer(dev)
    rs = [6, 4, 7, 8]
    multi = layer.prune_search_multi(x.to(DEV), rs)
    for r, (losses, best) in zip(rs, multi):
        single, best1 = layer.prune_search(x.to(DEV), r)
        assert losses == single and best == best1
    ora = O.prune_search_allexperts(synth.bf16_bits(x), host["Wg"], host["W1"], host["W3"], host["W2"], 4)
    P.check_search(multi[1][0], multi[1][1], ora)
    one = layer.prune_search_multi(x.to(DEV), [5])
    assert one[0] == tuple(layer.prune_search(x.to(DEV), 5))
    with pytest.raises(binding.MoeError):
        layer.prune_search_multi(x.to(DEV), [6, 1])
    with pytest.raises(binding.MoeError):
        layer.prune_search_multi(x.to(DEV), [])
    layer.close()


@pytest.mark.parametrize("r", [6, 4, 8, 2])
def test_prune_search_matches_oracle(setup, r):
    host, dev = setup
    T = 256
    x = synth.make_tokens(T, H, seed=0)
    ora = O.prune_search_allexperts(synth.bf16_bits(x), host["Wg"], host["W1"], host["W3"], host["W2"], r)
    layer = make_layer(dev)
    losses, best = layer.prune_search(x.to(DEV), r)
    losses2, best2 = layer.prune_search(x.to(DEV), r)
    layer.close()
    assert len(losses) == len(ora["losses"])
    assert losses == losses2 and best == best2, "search is not reproducible"
    P.check_search(losses, best, ora)
    if r == 8:
        assert losses == [0.0] and best == FULL


def test_prune_search_ragged_T_and_chunk_additivity(setup):
    host, dev = setup
    x = synth.make_tokens(333, H, seed=8)
    ora = O.prune_search_allexperts(synth.bf16_bits(x), host["Wg"], host["W1"], host["W3"], host["W2"], 6)
    layer = make_layer(dev)
    whole, best = layer.prune_search(x.to(DEV), 6)
    a, _ = layer.prune_search(x[:100].contiguous().to(DEV), 6)
    b, _ = layer.prune_search(x[100:].contiguous().to(DEV), 6)
    layer.close()
    P.check_search(whole, best, ora)
    np.testing.assert_allclose(np.square(a) + np.square(b), np.square(whole), rtol=1e-4)


def test_rmsnorm_and_stack(setup):
    host, dev = setup
    T = 300
    x = synth.make_tokens(T, H, seed=6)
    got = binding.rmsnorm(x.to(DEV), 1e-5)
    want = O.rmsnorm(synth.bf16_bits(x), 1e-5)
    diff = np.abs(synth.bf16_bits(got).astype(np.int32) - want.astype(np.int32))
    assert diff.max() <= 1 and (diff != 0).mean() < 0.01
    # three layers with different seeds, kept sets and betas; the oracle follows the same recurrence
    specs = [(20, FULL, 0.0), (21, 0b10111011, 0.4), (22, 0b00111100, 0.5)]
    b = synth.bf16_bits
    walk = P.StackParity(T, E, DEV)
    layers, cur_o, cur_g = [], b(x), x.to(DEV)
    for seed, kept, beta in specs:
        W = synth.make_layer_weights(H, F, E, seed=seed)
        layers.append(binding.MoeLayer(W.W_gate.to(DEV), W.W1.to(DEV), W.W3.to(DEV), W.W2.to(DEV), kept))
        hw = dict(Wg=b(W.W_gate), W1=b(W.W1), W3=b(W.W3), W2=b(W.W2))
        cur_o, cur_g = walk.layer(layers[-1], hw, kept, beta, cur_o, cur_g)
    y = binding.stack_forward(layers, x.to(DEV), [s[2] for s in specs], 1e-5)
    torch.cuda.synchronize()
    assert torch.equal(y, cur_g), "moe_stack_forward differs from the layer-by-layer calls"
    # every token whose routing agreed with the oracle in all three layers obeys the bound; a
    # re-routed token must have a near-tie in the oracle's own logits
    walk.finish(b(y), cur_o, max_rerouted=T // 20)
    for l in layers:
        l.close()


def test_stack_of_single_tokens(setup):
    # batch-1 decoding through three layers (RMSNorm, single-token kernels with the residual)
    specs = [(20, FULL, 0.0), (21, 0b10111011, 0.4), (22, 0b00111100, 0.5)]
    b = synth.bf16_bits
    Ws = [synth.make_layer_weights(H, F, E, seed=seed) for seed, _, _ in specs]
    hws = [dict(Wg=b(W.W_gate), W1=b(W.W1), W3=b(W.W3), W2=b(W.W2)) for W in Ws]
    layers = [binding.MoeLayer(W.W_gate.to(DEV), W.W1.to(DEV), W.W3.to(DEV), W.W2.to(DEV), kept)
              for W, (_, kept, _) in zip(Ws, specs)]
    rerouted = 0
    for seed in range(8):
        x = synth.make_tokens(1, H, seed=60 + seed)
        walk = P.StackParity(1, E, DEV)
        cur_o, cur_g = b(x), x.to(DEV)
        for layer, hw, (_, kept, beta) in zip(layers, hws, specs):
            cur_o, cur_g = walk.layer(layer, hw, kept, beta, cur_o, cur_g)
        y = binding.stack_forward(layers, x.to(DEV), [s[2] for s in specs], 1e-5)
        torch.cuda.synchronize()
        assert torch.equal(y, cur_g)
        if walk.agree[0]:
            walk.finish(b(y), cur_o, max_rerouted=0)
        else:
            assert not walk.unexplained
            rerouted += 1
    assert rerouted <= 1
    for l in layers:
        assert l.device_status() == 0
        l.close()


@pytest.mark.parametrize("h,f,E,kept,T", [
    (192, 320, 4, 0b1111, 300),     # ragged K and N tiles, few experts
    (192, 320, 4, 0b1011, 40),
    (64, 64, 16, 0xFFFF, 513),      # smallest shapes, 16 experts
    (256, 192, 16, 0xF0F3, 200),    # 10 of 16 experts kept (generic router path)
    (128, 448, 2, 0b11, 129),       # every token uses both experts
    (192, 320, 4, 0b1011, 1),       # single token: matrix-vector kernels, ragged row lengths
    (64, 64, 16, 0xFFFF, 1),
])
def test_forward_other_shapes(h, f, E, kept, T):
    build.build()
    W = synth.make_layer_weights(h, f, E, seed=31)
    b = synth.bf16_bits
    host = dict(Wg=b(W.W_gate), W1=b(W.W1), W3=b(W.W3), W2=b(W.W2))
    x = synth.make_tokens(T, h, seed=32)
    beta = 0.35
    ora = O.moe_forward(b(x), host["Wg"], host["W1"], host["W3"], host["W2"], kept, beta)
    ora["logits"] = O.route(b(x), host["Wg"], kept, beta)["logits"]
    layer = binding.MoeLayer(W.W_gate.to(DEV), W.W1.to(DEV), W.W3.to(DEV), W.W2.to(DEV), kept)
    stats = binding.RoutingStats(T, E, DEV)
    y = layer.forward(x.to(DEV), beta, stats=stats)
    torch.cuda.synchronize()
    assert layer.device_status() == 0
    gi, gs = stats.idx.cpu().numpy(), stats.skipped.cpu().numpy()
    P.check_routing(gi, gs, stats.wn.cpu().numpy(), stats.ratio.cpu().numpy(), ora, kept, beta)
    ok = (gi == ora["idx"]).all(1) & (gs == ora["skipped"])
    P.check_outputs(b(y), ora["y"], ok)
    layer.close()


@pytest.mark.parametrize("E,r", [(4, 2), (4, 3), (16, 14), (16, 15), (6, 3)])
def test_prune_search_other_expert_counts(E, r):
    build.build()
    h, f, T = 128, 192, 150
    W = synth.make_layer_weights(h, f, E, seed=41)
    b = synth.bf16_bits
    x = synth.make_tokens(T, h, seed=42)
    ora = O.prune_search_allexperts(b(x), b(W.W_gate), b(W.W1), b(W.W3), b(W.W2), r)
    layer = binding.MoeLayer(W.W_gate.to(DEV), W.W1.to(DEV), W.W3.to(DEV), W.W2.to(DEV))
    losses, best = layer.prune_search(x.to(DEV), r)
    layer.close()
    P.check_search(losses, best, ora)


def test_coselection_and_frequency_baseline(setup):
    host, dev = setup
    T = 1500
    x = synth.make_tokens(T, H, seed=12)
    want = O.coselection(synth.bf16_bits(x), host["Wg"])
    ties = int(P.near_tie_tokens(O.route(synth.bf16_bits(x), host["Wg"], FULL, 0.0)["logits"], FULL).sum())
    layer = make_layer(dev)
    got = np.array(layer.coselection(x.to(DEV)), np.int64)
    assert got.sum() == T and np.trace(got) == 0
    assert np.abs(got - want).sum() <= 2 * ties
    for r in (6, 4):
        assert layer.frequency_subset(want.tolist(), r) == O.frequency_subset(want, r)
    # the searched subset is never worse than the frequency baseline's or a random subset
    losses, best = layer.prune_search(x.to(DEV), 6)
    subsets = O.enumerate_subsets(E, 6).tolist()
    freq_loss = losses[subsets.index(O.frequency_subset(want, 6))]
    assert min(losses) <= freq_loss and min(losses) <= float(np.mean(losses))
    pruned = make_layer(dev, 0b00111111)
    assert np.array(pruned.coselection(x.to(DEV)))[6:, :].sum() == 0
    pruned.close()
    layer.close()


@pytest.mark.parametrize("r", [6, 4])
def test_progressive_search_matches_oracle(setup, r):
    host, dev = setup
    T = 333
    x = synth.make_tokens(T, H, seed=0)       # states of the unpruned stack
    xp = synth.make_tokens(T, H, seed=5)      # states that went through pruned layers
    layer = make_layer(dev)
    F_ref = layer.forward(x.to(DEV), 0.0).float().contiguous()   # cached unpruned output (bf16 -> fp32)
    ora = O.prune_search_progressive(synth.bf16_bits(xp), host["Wg"], host["W1"], host["W3"], host["W2"],
                                     F_ref.cpu().numpy(), r)
    losses, best = layer.prune_search_progressive(xp.to(DEV), F_ref, r)
    P.check_search(losses, best, ora)
    # identical inputs on both sides: the layer-wise losses up to the bf16 rounding of the cached target
    lw, _ = layer.prune_search(x.to(DEV), r)
    pg, _ = layer.prune_search_progressive(x.to(DEV), F_ref, r)
    fn = float(F_ref.double().norm())
    assert np.abs(np.array(pg) - np.array(lw)).max() <= 2 ** -8 * fn
    layer.close()


@pytest.mark.parametrize("E_,kept,k,T,beta", [
    (16, 0xFFFF, 4, 300, 0.0), (16, 0xFFFF, 4, 300, 0.3), (16, 0xF0F3, 3, 1000, 0.2),
    (8, 0xFF, 2, 256, 0.3), (8, 0xFF, 1, 64, 0.0), (8, 0b10111101, 6, 40, 0.15), (16, 0xFFFF, 8, 33, 0.4),
])
def test_forward_topk_generalised_skipping(E_, kept, k, T, beta):
    build.build()
    h, f = 128, 192
    W = synth.make_layer_weights(h, f, E_, seed=51)
    b = synth.bf16_bits
    x = synth.make_tokens(T, h, seed=52)
    ora = O.moe_forward_topk(b(x), b(W.W_gate), b(W.W1), b(W.W3), b(W.W2), kept, k, beta)
    layer = binding.MoeLayer(W.W_gate.to(DEV), W.W1.to(DEV), W.W3.to(DEV), W.W2.to(DEV), kept)
    y, idx, wn, na = layer.forward_topk(x.to(DEV), k, beta, record=True)
    torch.cuda.synchronize()
    assert layer.device_status() == 0
    idx, wn, na = idx.cpu().numpy(), wn.cpu().numpy(), na.cpu().numpy()
    # near-ties: an adjacent gap below 1e-3 among the k+1 largest kept logits
    keptv = np.array([(kept >> e) & 1 for e in range(E_)], bool)
    srt = -np.sort(-np.where(keptv[None, :], ora["logits"].astype(np.float64), -np.inf), axis=1)
    tie = (np.diff(-srt[:, :min(k + 1, int(keptv.sum()))], axis=1) < P.LOGIT_GAP_TOL).any(1)
    assert tie.mean() < 0.1
    assert np.array_equal(idx[~tie], ora["idx"][~tie])
    same_idx = (idx == ora["idx"]).all(1)
    # the decision i* may differ only where a tail mass sits on the threshold
    sel = np.take_along_axis(ora["logits"].astype(np.float64), ora["idx"].astype(np.int64), 1)
    p = np.exp(sel - sel[:, :1])
    fr = np.stack([p[:, i:].sum(1) for i in range(1, k + 1)], 1) / p.sum(1, keepdims=True)
    close = (np.abs(fr - beta) < P.RATIO_TOL).any(1)
    chk = same_idx & ~close
    assert np.array_equal(na[chk], ora["n_active"][chk])
    # the rule itself, evaluated here in fp64 (App. A.2): i* = the first i whose tail mass is
    # at most beta of the total; the tail beyond k is empty, so i* <= k
    want_na = 1 + np.argmax(fr <= beta, axis=1)
    assert np.array_equal(na[chk], want_na[chk])
    both = same_idx & (na == ora["n_active"])
    np.testing.assert_allclose(wn[both], ora["wn"][both], rtol=2e-5, atol=1e-7)
    P.check_outputs(b(y), ora["y"], both)
    layer.close()


@pytest.mark.parametrize("T,kept", [(256, FULL), (1000, 0b11011101), (5, FULL)])
def test_top2_distance(setup, T, kept):
    host, dev = setup
    x = synth.make_tokens(T, H, seed=13)
    want = O.top2_distance(synth.bf16_bits(x), host["Wg"], host["W1"], host["W3"], host["W2"], kept)
    tie = P.near_tie_tokens(O.route(synth.bf16_bits(x), host["Wg"], kept, 0.0)["logits"], kept)
    layer = make_layer(dev, kept)
    got = layer.top2_distance(x.to(DEV)).cpu().numpy().astype(np.float64)
    layer.close()
    ok = ~tie
    np.testing.assert_allclose(got[ok], want[ok], rtol=5e-3)


@pytest.mark.parametrize("eps", [0.25, 0.03])
def test_prune_search_with_nearly_identical_experts(setup, eps):
    # Experts that differ from one another by a small perturbation of common weights: every
    # subset's loss is then a small difference of large, nearly equal expert outputs, which is
    # where a careless evaluation of the squared errors would lose its digits.  Both the
    # layer-wise and the progressive form must still match the oracle to the usual tolerance.
    W = synth.make_layer_weights(H, F, E, seed=0)
    g = torch.Generator().manual_seed(123)
    def near(Wt):
        base = Wt[0:1].float()
        noise = torch.randn(Wt.shape, generator=g) * synth.WEIGHT_STD
        return (base + eps * noise).to(torch.bfloat16).contiguous()
    W1, W3, W2 = near(W.W1), near(W.W3), near(W.W2)
    b = synth.bf16_bits
    T = 300
    x = synth.make_tokens(T, H, seed=9)
    layer = binding.MoeLayer(W.W_gate.to(DEV), W1.to(DEV), W3.to(DEV), W2.to(DEV))
    for r in (6, 4):
        ora = O.prune_search_allexperts(b(x), b(W.W_gate), b(W1), b(W3), b(W2), r)
        losses, best = layer.prune_search(x.to(DEV), r)
        P.check_search(losses, best, ora)
    xu = synth.make_tokens(T, H, seed=10)
    F_ref = layer.forward(xu.to(DEV), 0.0).float().contiguous()
    ora = O.prune_search_progressive(b(x), b(W.W_gate), b(W1), b(W3), b(W2), F_ref.cpu().numpy(), 6)
    losses, best = layer.prune_search_progressive(x.to(DEV), F_ref, 6)
    P.check_search(losses, best, ora)
    layer.close()


@pytest.mark.parametrize("kept,beta", [(FULL, 0.3), (0b01101101, 0.0)])
def test_forward_many_tokens_on_double_row_items(setup, kept, beta):
    # enough tokens for the large-batch GEMM to run on items of 256 token rows at this small shape
    # (2f = 896 weight rows: the last 256-row weight tile is half empty; ragged expert groups end
    # in half items and partly filled tiles)
    host, dev = setup
    r = run_case(host, dev, 20000, kept, beta, x_seed=21)
    assert r["ties"] <= 20000 // 20


def test_prune_search_many_tokens_on_double_row_items(setup):
    host, dev = setup
    T = 9000   # two chunks of expert evaluations, the first one of 8192 tokens x 6 experts
    x = synth.make_tokens(T, H, seed=22)
    layer = make_layer(dev)
    (l6, b6), (l4, b4) = layer.prune_search_multi(x.to(DEV), [6, 4])
    layer.close()
    xb = synth.bf16_bits(x)
    P.check_search(l6, b6, O.prune_search_allexperts(xb, host["Wg"], host["W1"], host["W3"], host["W2"], 6))
    P.check_search(l4, b4, O.prune_search_allexperts(xb, host["Wg"], host["W1"], host["W3"], host["W2"], 4))


def test_prune_search_multi_in_several_passes():
    # 16 experts: the subsets of sizes 15, 14 and 8 (13006 together) share one enumeration pass, the
    # 11440 of size 7 need a second one; every size must give what a search of its own gives (to
    # rounding: with more than six ranked experts per token the errors are formed pair by pair)
    build.build()
    E_, h, f, T = 16, 128, 192, 150
    W = synth.make_layer_weights(h, f, E_, seed=61)
    x = synth.make_tokens(T, h, seed=62).to(DEV)
    layer = binding.MoeLayer(W.W_gate.to(DEV), W.W1.to(DEV), W.W3.to(DEV), W.W2.to(DEV))
    rs = [15, 14, 8, 7]
    multi = layer.prune_search_multi(x, rs)
    for r, (losses, best) in zip(rs, multi):
        single, best1 = layer.prune_search(x, r)
        assert len(losses) == len(single) == binding.num_subsets(E_, r)
        np.testing.assert_allclose(losses, single, rtol=2e-5, atol=1e-7)
        if best != best1:
            assert abs(min(losses) - single[int(np.argmin(losses))]) <= 1e-4 * min(single)
    b = synth.bf16_bits
    ora = O.prune_search_allexperts(b(x), b(W.W_gate), b(W.W1), b(W.W3), b(W.W2), 14)
    P.check_search(multi[1][0], multi[1][1], ora)
    layer.close()
