"""Per-network selection on the BERT-large-shaped stack (24 blocks x 6 linears = 144 layers,
221 184 channels, 10 % channel budget), bit-exact against the oracle, followed by the
backward of layers with very different per-layer counts (including a frozen one)."""
import numpy as np
import pytest
import torch

from oracle import efqat_oracle as O
from paper_2411_11038_b200 import binding as B
from paper_2411_11038_b200 import inputs as I
from tests import parity_util as U

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    return B.Context(0)


@pytest.fixture(scope="module")
def stack():
    cases = I.config4()
    Ws = []
    for c in cases:
        g = torch.Generator().manual_seed(c.seed)
        Ws.append(torch.randn((c.N, c.K), generator=g) * float(np.sqrt(2.0 / c.K)))
    return cases, Ws


def test_cwpn_over_144_layers_bit_exact(ctx, stack):
    cases, Ws = stack
    total = sum(c.N for c in cases)
    assert total == 221184
    budget = B.ratio_to_k(0.1, total)
    assert budget == 22118
    dW = [w.cuda() for w in Ws]
    got, offsets, imp = B.select_channels(ctx, B.CWPN, dW, [budget], want_importance=True)
    keys = np.concatenate([O.importance_rows(w.numpy()) for w in Ws])
    assert np.array_equal(imp.cpu().numpy(), keys)
    ref = O.select_cwpn([w.numpy() for w in Ws], budget)
    counts = [len(r) for r in ref]
    assert offsets.cpu().tolist() == np.concatenate([[0], np.cumsum(counts)]).tolist()
    for a, b in zip(got, ref):
        assert a.cpu().numpy().tolist() == b.tolist()
    # the fan-in-4096 layers have half the mean |w| of the others: the global ranking freezes them
    assert all(counts[6 * b + 5] == 0 for b in range(24)) and max(counts) > 100
    assert ctx.device_status() == 0
    # layer-wise mode over the same stack
    lw, _, _ = B.select_channels(ctx, B.LWPN, dW, [14])
    ref_l = O.select_lwpn([w.numpy() for w in Ws], 14)
    for a, b in zip(lw, ref_l):
        assert a.cpu().numpy().tolist() == b.tolist()


@pytest.mark.parametrize("li", [0, 5])
def test_backward_with_network_selected_counts(ctx, stack, li):
    cases, Ws = stack
    ref = O.select_cwpn([w.numpy() for w in Ws], 22118)
    case = I.shrink(cases[li], 1152)                  # an eighth of the tokens keeps the oracle in seconds
    T = I.make_tensors(case)
    T["W"] = Ws[li]
    s_w, s_x, z_x = U.oracle_qparams(case, T, (0.8, 0.9, 0.6))
    D = U.to_dev(T, s_w, s_x, z_x)
    idx = ref[li]
    assert (len(idx) == 0) == (li == 5)
    U.check_forward(ctx, case, T, D, s_w, s_x, z_x)
    U.check_backward(ctx, case, T, D, s_w, s_x, z_x, idx)


@pytest.mark.parametrize("li", [0, 4, 5])
def test_network_layer_shapes_at_full_token_count(ctx, stack, li):
    """The three layer shapes of the stack (1024 -> 1024, 1024 -> 4096, 4096 -> 1024) at the full
    M = 24 x 384 = 9216 tokens, W4A8, with the channel counts the network-wide ranking assigns."""
    cases, Ws = stack
    ref = O.select_cwpn([w.numpy() for w in Ws], 22118)
    case = cases[li]
    assert case.M == 9216
    T = I.make_tensors(case)
    T["W"] = Ws[li]
    s_w, s_x, z_x = U.oracle_qparams(case, T, (0.8, 0.9, 0.6))
    D = U.to_dev(T, s_w, s_x, z_x)
    U.check_forward(ctx, case, T, D, s_w, s_x, z_x)
    U.check_backward(ctx, case, T, D, s_w, s_x, z_x, ref[li])
