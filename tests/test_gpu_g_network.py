"""Weight-operand cache and whole-network calls (Section 3.2 "Freezing Frequency"; Algorithm 1
over every layer): a cached forward / backward must be bit-identical to the uncached one after
any number of optimizer steps, as long as the stepped rows are refreshed; the network calls
must equal the per-layer calls; the freezing-frequency schedule re-selects when it says it does."""
import numpy as np
import pytest
import torch

from oracle import efqat_oracle as O
from paper_2411_11038_b200 import binding as B
from paper_2411_11038_b200 import inputs as I
from paper_2411_11038_b200 import network as NW
from tests import parity_util as U

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    return B.Context(0)


def _case(name, M, K, N, w_bits=8, seed=0, dtype=torch.bfloat16):
    return I.LayerCase(name, M, K, N, act_dtype=dtype, w_bits=w_bits, x_bits=8, seed=seed)


@pytest.mark.parametrize("shape", [
    (640, 768, 2304, 8),      # integer forward (K >= 512): 8-bit codes + row sums in the cache
    (640, 256, 520, 4),       # bf16 forward (short contraction, N % 32 != 0): bf16 codes in the cache
])
def test_cached_calls_bit_identical_over_optimizer_steps(ctx, shape):
    M, K, N, wb = shape
    case = _case("cache", M, K, N, wb, seed=77)
    T = I.make_tensors(case)
    D = {k: v.cuda() for k, v in T.items()}
    s_w = B.init_weight_scales(ctx, D["W"], wb)
    s_x, z_x = B.init_act_qparams(ctx, D["X"], 8, False)
    s_w.mul_(0.9)                          # some weights clip
    mom = torch.zeros_like(D["W"])
    # rates far above the paper's: codes, scales and the importance ranking all move between steps
    sgd = B.make_sgd(1e-5, 0.9, 1e-4, D["W"], mom)
    qopt = B.QParamOptimizer(ctx, s_w, s_x, z_x, lr=1e-4)
    k = max(B.ratio_to_k(0.1, N), 1)
    plan = B.LayerPlan(ctx, M, N, K, torch.bfloat16, wb, 8, False, N, "cuda", with_cache=True)
    ref_plan = B.LayerPlan(ctx, M, N, K, torch.bfloat16, wb, 8, False, N, "cuda")
    plan.cache_update(D["W"], s_w)                      # every row once
    seen = set()
    W_start = D["W"].clone()
    for step in range(4):
        sel, _, _ = B.select_channels(ctx, B.CWPL, [D["W"]], [k])
        idx = sel[0]
        seen.add(tuple(idx.cpu().tolist()))
        out = plan.bwd_cached(D["dY"], D["X"], D["W"], s_w, s_x, z_x, idx, k, want_db=True, sgd=sgd)
        qopt.step(idx, k, out["dS_w_sel"], out["dS_x"], out["dZ_x"])
        plan.cache_update(D["W"], s_w, idx, k)          # only the rows that have just moved
        # forward
        Yc = plan.fwd_cached(D["X"], s_w, s_x, z_x, D["bias"]).clone()
        Yu = ref_plan.fwd(D["X"], D["W"], s_w, s_x, z_x, D["bias"])
        assert torch.equal(Yc, Yu), f"step {step}: cached forward differs"
        # backward without an update, cached against uncached: every output bit for bit
        a = plan.bwd_cached(D["dY"], D["X"], D["W"], s_w, s_x, z_x, idx, k, want_db=True)
        a = {kk: v.clone() for kk, v in a.items()}
        b = ref_plan.bwd(D["dY"], D["X"], D["W"], s_w, s_x, z_x, idx, k, want_db=True)
        for key in ("dX", "dW_sel", "dS_w_sel", "dS_x", "dZ_x", "db"):
            assert torch.equal(a[key], b[key]), f"step {step}: cached backward differs in {key}"
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    assert not torch.equal(W_start, D["W"])
    assert len(seen) > 1, "the selection never changed: the test did not exercise rows leaving the unfrozen set"
    # the state the cache ended in, against the oracle on the final parameters
    Tn = dict(T)
    Tn["W"] = D["W"].cpu()
    U.check_forward_values(case, Tn, Yc, s_w.cpu().numpy(), np.float32(s_x.item()), np.float32(z_x.item()))


def test_stale_row_is_what_the_contract_says(ctx):
    """The cache records no validity: a row changed without a refresh keeps its old codes.  (This is
    the documented contract, checked so that a silent re-quantization cannot hide a missing refresh.)"""
    case = _case("stale", 256, 512, 64, 8, seed=5)
    T = I.make_tensors(case)
    D = {k: v.cuda() for k, v in T.items()}
    s_w = B.init_weight_scales(ctx, D["W"], 8)
    s_x, z_x = B.init_act_qparams(ctx, D["X"], 8, False)
    plan = B.LayerPlan(ctx, 256, 64, 512, torch.bfloat16, 8, 8, False, 64, "cuda", with_cache=True)
    plan.cache_update(D["W"], s_w)
    Y0 = plan.fwd_cached(D["X"], s_w, s_x, z_x, None).clone()
    D["W"][3].mul_(-1.0)
    Y1 = plan.fwd_cached(D["X"], s_w, s_x, z_x, None).clone()
    assert torch.equal(Y0, Y1)
    idx = torch.tensor([3], dtype=torch.int32, device="cuda")
    plan.cache_update(D["W"], s_w, idx, 1)
    Y2 = plan.fwd_cached(D["X"], s_w, s_x, z_x, None).clone()
    assert torch.equal(Y2[:, 3].float(), -Y0[:, 3].float())
    keep = [c for c in range(64) if c != 3]
    assert torch.equal(Y2[:, keep], Y0[:, keep])


def _stack(ctx, shapes, seed0):
    layers = []
    for i, (M, K, N) in enumerate(shapes):
        case = _case(f"net{i}", M, K, N, 4, seed=seed0 + i)
        case.w_std = None
        T = I.make_tensors(case)
        layers.append((case, T))
    return layers


def test_network_calls_equal_layer_calls(ctx):
    shapes = [(384, 512, 512), (384, 512, 1024), (384, 1024, 512), (384, 512, 512)]
    stack = _stack(ctx, shapes, 900)
    states = [NW.LayerState(c, T["W"].cuda(), T["X"].cuda(), T["dY"].cuda(), T["bias"].cuda()) for c, T in stack]
    total = sum(c.N for c, _ in stack)
    net = NW.EfqatNetwork(ctx, states, B.CWPN, B.ratio_to_k(0.1, total), f_samples=1, batch_samples=1,
                          use_cache=True, sgd=None, adam=None, share_outputs=False)
    net.reselect()
    ref = O.select_cwpn([I.as_f64(T["W"]) for _, T in stack], B.ratio_to_k(0.1, total))
    assert net.counts() == [len(r) for r in ref]
    net.forward()
    net.backward()
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    for l, ((case, T), st, plan) in enumerate(zip(stack, states, net.plans)):
        k = net.counts()[l]
        idx = net.net.idx[net.offsets_host[l]:net.offsets_host[l] + k] if k else None
        Y = B.fq_linear_fwd(ctx, st.X, st.W, st.s_w, st.s_x, st.z_x, st.bias, case.w_bits, case.x_bits, False)
        assert torch.equal(Y, plan.Y), f"layer {l}: network forward differs from the layer call"
        out = B.fq_linear_bwd(ctx, st.dY, st.X, st.W, st.s_w, st.s_x, st.z_x, idx, k, case.w_bits, case.x_bits,
                              False, want_db=True)
        assert torch.equal(out["dX"], plan.dX)
        assert torch.equal(out["dW_sel"], plan.dW_sel[:k])
        assert torch.equal(out["dS_w_sel"], plan.dS_w_sel[:k])
        assert torch.equal(out["dS_x"], plan.dS_x) and torch.equal(out["dZ_x"], plan.dZ_x)
        assert torch.equal(out["db"], plan.db)
    # one layer against the oracle end to end (selection from the network-wide ranking)
    case, T = stack[1]
    st = states[1]
    s_w, s_x, z_x = st.s_w.cpu().numpy(), np.float32(st.s_x.item()), np.float32(st.z_x.item())
    D = U.to_dev(T, s_w, s_x, z_x)
    U.check_backward(ctx, case, T, D, s_w, s_x, z_x, ref[1])


def test_training_steps_with_freezing_frequency(ctx):
    """Several whole training steps (fused SGD, Adam on the quantization parameters, cache refresh)
    with re-selection every third step: the cached network ends bit-identical to an uncached twin,
    and the frozen set only changes when the schedule says so."""
    shapes = [(256, 512, 512), (256, 512, 768), (256, 768, 512)]
    stack = _stack(ctx, shapes, 1200)
    total = sum(c.N for c, _ in stack)

    def build(use_cache):
        states = [NW.LayerState(c, T["W"].cuda().clone(), T["X"].cuda(), T["dY"].cuda(), T["bias"].cuda())
                  for c, T in stack]
        return states, NW.EfqatNetwork(ctx, states, B.CWPN, B.ratio_to_k(0.1, total), f_samples=24,
                                       batch_samples=8, use_cache=use_cache, sgd=(2e-5, 0.9, 1e-4),
                                       adam=dict(lr=1e-4), share_outputs=False)

    sa, a = build(True)
    sb, b = build(False)
    sets = []
    for step in range(7):
        a.train_step()
        b.train_step()
        sets.append(tuple(a.net.idx[:a.offsets_host[-1]].cpu().tolist()))
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    assert a.schedule.selections == 3 and b.schedule.selections == 3      # steps 0, 3, 6
    assert sets[0] == sets[1] == sets[2] and sets[3] == sets[4] == sets[5]
    assert sets[0] != sets[3]
    for x, y in zip(sa, sb):
        assert torch.equal(x.W, y.W) and torch.equal(x.s_w, y.s_w)
        assert torch.equal(x.s_x, y.s_x) and torch.equal(x.z_x, y.z_x) and torch.equal(x.mom, y.mom)
    a.forward()
    b.forward()
    for pa, pb in zip(a.plans, b.plans):
        assert torch.equal(pa.Y, pb.Y)


def test_network_calls_on_convolutions_equal_layer_calls(ctx):
    """A small convolutional stack through the network calls (cache on): an input layer on 8 stored
    channels (filter rows as contraction blocks, strip-form grad-input), a 3x3 whose taps share
    boxes per filter column, a stride-2 3x3 and a 1x1: bit-identical to the per-layer calls, and one
    layer against the oracle."""
    def conv_case(name, Bn, H, Wd, Cin, N, R, pad, stride, seed):
        Ho, Wo = (H + 2 * pad - R) // stride + 1, (Wd + 2 * pad - R) // stride + 1
        return I.LayerCase(name, Bn * Ho * Wo, R * R * Cin, N, act_dtype=torch.bfloat16, w_bits=4, x_bits=8, w_std=None,
                           x_abs=True, seed=seed, conv=True, B=Bn, H=H, Wd=Wd, Cin=Cin, R=R, S=R, stride=stride, pad=pad)

    cases = [conv_case("in7x7", 2, 32, 32, 8, 64, 7, 3, 2, 1301), conv_case("c3x3", 2, 16, 24, 64, 64, 3, 1, 1, 1302),
             conv_case("c3x3s2", 2, 16, 24, 64, 128, 3, 1, 2, 1303), conv_case("c1x1", 2, 8, 12, 128, 64, 1, 0, 1, 1304)]
    stack = [(c, I.make_tensors(c)) for c in cases]
    states = [NW.LayerState(c, T["W"].cuda(), T["X"].cuda(), T["dY"].cuda(), T["bias"].cuda()) for c, T in stack]
    total = sum(c.N for c in cases)
    net = NW.EfqatNetwork(ctx, states, B.CWPN, B.ratio_to_k(0.25, total), f_samples=1, batch_samples=1,
                          use_cache=True, sgd=None, adam=None, share_outputs=False)
    net.reselect()
    ref = O.select_cwpn([I.as_f64(T["W"]).reshape(c.N, -1) for c, T in stack], B.ratio_to_k(0.25, total))
    assert net.counts() == [len(r) for r in ref]
    net.forward()
    net.backward()
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    for l, ((case, T), st, plan) in enumerate(zip(stack, states, net.plans)):
        k = net.counts()[l]
        idx = net.net.idx[net.offsets_host[l]:net.offsets_host[l] + k] if k else None
        geom = B.ConvGeom(case.B, case.H, case.Wd, case.Cin, case.R, case.S, case.stride, case.pad)
        Y = B.fq_linear_fwd(ctx, st.X, st.W, st.s_w, st.s_x, st.z_x, st.bias, case.w_bits, case.x_bits, False, conv=geom)
        assert torch.equal(Y, plan.Y), f"layer {l}: network forward differs from the layer call"
        out = B.fq_linear_bwd(ctx, st.dY, st.X, st.W, st.s_w, st.s_x, st.z_x, idx, k, case.w_bits, case.x_bits,
                              False, want_db=True, conv=geom)
        assert torch.equal(out["dX"], plan.dX), f"layer {l}: dX"
        assert torch.equal(out["dW_sel"].reshape(k, case.K), plan.dW_sel[:k].reshape(k, case.K)), f"layer {l}: dW"
        assert torch.equal(out["dS_w_sel"], plan.dS_w_sel[:k])
        assert torch.equal(out["dS_x"], plan.dS_x) and torch.equal(out["dZ_x"], plan.dZ_x)
        assert torch.equal(out["db"], plan.db)
    # the input layer against the oracle (selection from the network-wide ranking)
    case, T = stack[0]
    st = states[0]
    s_w, s_x, z_x = st.s_w.cpu().numpy(), np.float32(st.s_x.item()), np.float32(st.z_x.item())
    X64, W64, dY64, b64 = (I.as_f64(T[kk]) for kk in ("X", "W", "dY", "bias"))
    refY = O.conv_forward(X64, W64, s_w, s_x, z_x, b64, case.w_bits, case.x_bits, case.stride, case.pad)
    U.assert_bf16_class(net.plans[0].Y.float().cpu().numpy(), refY, "input layer Y through the network call")
    ex = O.conv_backward_efqat(dY64, X64, W64, s_w, s_x, z_x, ref[0], case.w_bits, case.x_bits, case.stride, case.pad,
                               operand_model="exact")
    U.assert_bf16_class(net.plans[0].dX.float().cpu().numpy(), ex["dX"], "input layer dX through the network call")
    k0 = net.counts()[0]
    if k0:
        U.assert_bf16_class(net.plans[0].dW_sel[:k0].cpu().numpy().reshape(ex["dW_sel"].shape), ex["dW_sel"],
                            "input layer dW_sel through the network call")


def test_shared_and_alternating_workspaces_give_the_same_bits(ctx):
    """efqat_network_bwd puts a layer's finalize work into the next layer's prepare launch only when
    their workspaces are disjoint: with one shared workspace every layer keeps its own finalize
    launch.  Both ways must produce the same bits, over a stack that mixes the general backward, a
    layer with the one-pass backward (no prepare launch to ride in) and frozen layers."""
    shapes = [(384, 512, 512), (1024, 64, 256), (384, 512, 1024), (1024, 64, 128), (384, 1024, 512)]
    stack = _stack(ctx, shapes, 1500)
    total = sum(c.N for c, _ in stack)
    outs = []
    for alternate in (True, False):
        states = [NW.LayerState(c, T["W"].cuda().clone(), T["X"].cuda(), T["dY"].cuda(), T["bias"].cuda())
                  for c, T in stack]
        net = NW.EfqatNetwork(ctx, states, B.CWPN, B.ratio_to_k(0.2, total), f_samples=1, batch_samples=1,
                              use_cache=True, sgd=(2e-5, 0.9, 1e-4), adam=None, share_outputs=False,
                              alternate_ws=alternate)
        net.reselect()
        n0 = ctx.launch_count() if hasattr(ctx, "launch_count") else None
        net.backward()
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        outs.append((states, net, n0))
    (sa, na, _), (sb, nb, _) = outs
    assert na.counts() == nb.counts()
    for l, (pa, pb) in enumerate(zip(na.plans, nb.plans)):
        k = na.counts()[l]
        assert torch.equal(pa.dX, pb.dX), f"layer {l}: dX"
        assert torch.equal(pa.dW_sel[:k], pb.dW_sel[:k]) and torch.equal(pa.dS_w_sel[:k], pb.dS_w_sel[:k])
        assert torch.equal(pa.dS_x, pb.dS_x) and torch.equal(pa.dZ_x, pb.dZ_x) and torch.equal(pa.db, pb.db)
    for x, y in zip(sa, sb):
        assert torch.equal(x.W, y.W) and torch.equal(x.mom, y.mom)
