"""True removal costs (Eq. individual_expert_damage) and retained energy (Eq. energy_retained) on the device
against the oracle's brute-force definitions."""

import numpy as np
import pytest
import torch

from oracle import base_oracle as O
from paper_2609_36222_b200 import binding as B
from paper_2609_36222_b200 import workloads as wl
from paper_2609_36222_b200.layer import bits_to_device

from gpu_harness import device_layer_from_host
from helpers import HostLayer

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

# An energy is a sum of d squared outputs, each carrying the FFN's error (bf16 rounding of the SwiGLU
# activations, fp32 accumulation): a relative error of a few 1e-3 per element that partly averages out.
ENERGY_RTOL = 2e-2


@pytest.mark.parametrize("name,T", [("tiny", 8), ("tiny", 3), ("mid", 32), ("qwen3", 64)])
def test_true_removal_costs_match_brute_force(name, T):
    cfg = wl.CONFIGS[name]
    host = HostLayer(cfg, T=T)
    dl = device_layer_from_host(host, DEV)
    logits = O.router_logits(host.z, host.router_w, host.router_bias)
    _, R, _, _, w = O.route_topk(logits, cfg.K)
    a = O.contributions(host.z, R, w, host.expert_weights)          # a[t,k,:] = w * E_u(z_t)
    ref_energy = (a * a).sum(axis=2) / (w * w)                       # ||E_u(z_t)||^2
    ref_D = O.true_removal_cost(a, R, cfg.E)

    hid = bits_to_device(host.hidden_bits, DEV)
    tc, en, ids, tw = B.base_true_removal_costs(dl.shape, dl.weights, hid, dl.workspace,
                                                router_logits=torch.from_numpy(logits).to(DEV))
    torch.cuda.synchronize()
    np.testing.assert_array_equal(ids.cpu().numpy(), R)
    np.testing.assert_allclose(tw.cpu().numpy(), w, rtol=1e-5)
    np.testing.assert_allclose(en.cpu().numpy(), ref_energy, rtol=ENERGY_RTOL)
    tc = tc.cpu().numpy().astype(np.float64)
    # dense layout: w^2 * energy at the routed pairs, exact zeros elsewhere
    ref_tc = np.zeros((T, cfg.E))
    for t in range(T):
        ref_tc[t, R[t]] = (a[t] * a[t]).sum(axis=1)
    assert ((tc == 0) == (ref_tc == 0)).all()
    np.testing.assert_allclose(tc, ref_tc, rtol=ENERGY_RTOL)

    # aggregated through the staged entry point: the true scores D* and the oracle selection A*
    M = cfg.budgets[0]
    scores, sel, mask = B.base_aggregate_select(torch.from_numpy(tc.astype(np.float32)).to(DEV), M)
    np.testing.assert_allclose(scores.cpu().numpy(), ref_D, rtol=ENERGY_RTOL)

    # retained energy of BASE's own selection, both sides on their own scores
    ref = O.moe_decode_layer(host.z, logits, host.pred_A, host.pred_b, host.expert_weights, cfg.K, M)
    base_mask = torch.from_numpy(ref["mask"].astype(np.uint8)).to(DEV)
    er = B.base_energy_retained(scores, base_mask, M).cpu().numpy()[0]
    assert abs(er - O.energy_retained(ref["mask"], ref_D, M)) <= 2 * ENERGY_RTOL
    # the oracle selection retains everything by definition; an empty mask nothing
    assert B.base_energy_retained(scores, mask, M).cpu().numpy()[0] == pytest.approx(1.0, abs=1e-6)
    assert B.base_energy_retained(scores, torch.zeros_like(mask), M).cpu().numpy()[0] == 0.0


def test_energy_retained_exact_on_small_integers():
    """Integer-valued scores make every sum exact: ties go to the lower id, the budget is clipped to E."""
    scores = torch.tensor([3, 7, 7, 0, 5, 1, 7, 2], dtype=torch.float32, device=DEV)
    mask = torch.tensor([1, 0, 1, 0, 1, 0, 0, 0], dtype=torch.uint8, device=DEV)
    # top-3 of the scores: ids 1, 2, 6 (three sevens) -> 21; the mask holds 3 + 7 + 5 = 15
    assert B.base_energy_retained(scores, mask, 3).cpu().numpy()[0] == np.float32(15) / np.float32(21)
    # top-2: ids 1, 2 (tie on 7 -> lower ids) -> 14
    assert B.base_energy_retained(scores, mask, 2).cpu().numpy()[0] == np.float32(15) / np.float32(14)
    assert B.base_energy_retained(scores, mask, 100).cpu().numpy()[0] == np.float32(15) / np.float32(32)
    zero = torch.zeros(8, dtype=torch.float32, device=DEV)
    assert B.base_energy_retained(zero, mask, 3).cpu().numpy()[0] == 1.0


def test_true_costs_error_codes():
    cfg = wl.CONFIGS["tiny"]
    host = HostLayer(cfg)
    dl = device_layer_from_host(host, DEV)
    hid = bits_to_device(host.hidden_bits, DEV)
    with pytest.raises(B.BaseError, match="workspace"):
        B.base_true_removal_costs(dl.shape, dl.weights, hid, dl.workspace[:1024])
    s = torch.zeros(4, dtype=torch.float32, device=DEV)
    m = torch.zeros(4, dtype=torch.uint8, device=DEV)
    with pytest.raises(B.BaseError, match="invalid"):
        B.base_energy_retained(s, m, 0)


@pytest.mark.parametrize("name,T", [("tiny", 8), ("mid", 32)])
def test_exact_error_decomposition_matches_oracle(name, T):
    """E(A), its individual part and the cross terms (Eq. error_decomposition) for BASE's own selection and for
    two degenerate masks; the individual part must also equal the true scores of the omitted experts."""
    cfg = wl.CONFIGS[name]
    host = HostLayer(cfg, T=T)
    dl = device_layer_from_host(host, DEV)
    logits = O.router_logits(host.z, host.router_w, host.router_bias)
    _, R, _, _, w = O.route_topk(logits, cfg.K)
    a = O.contributions(host.z, R, w, host.expert_weights)
    D = O.true_removal_cost(a, R, cfg.E)
    hid = bits_to_device(host.hidden_bits, DEV)
    lg = torch.from_numpy(logits).to(DEV)
    M = cfg.budgets[0]
    base_mask = O.moe_decode_layer(host.z, logits, host.pred_A, host.pred_b, host.expert_weights, cfg.K, M)["mask"]
    every_other = (np.arange(cfg.E) % 2 == 0).astype(np.uint8)
    for mask in (base_mask.astype(np.uint8), every_other, np.ones(cfg.E, np.uint8), np.zeros(cfg.E, np.uint8)):
        got = B.base_exact_removal_error(dl.shape, dl.weights, hid, torch.from_numpy(mask).to(DEV), dl.workspace,
                                         router_logits=lg).cpu().numpy().astype(np.float64)
        total, indiv, cross = O.exact_error(a, R, mask)
        scale = max(indiv, 1e-30)
        assert abs(got[0] - total) <= ENERGY_RTOL * scale
        assert abs(got[1] - indiv) <= ENERGY_RTOL * scale
        assert abs(got[2] - cross) <= 2 * ENERGY_RTOL * scale
        assert abs(got[1] - D[mask == 0].sum()) <= ENERGY_RTOL * scale          # additive estimate: sum of D*_u
        assert got[0] >= 0 and abs(got[0] - got[1] - got[2]) <= 1e-5 * max(got[0], scale)
        if mask.all():
            assert (got == 0).all()
