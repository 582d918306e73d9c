"""GPU-vs-oracle parity for the block-mean estimate of A' (the contrast scorer, not the paper's) and the
selection from it: scores against the fp64 oracle, the ranking bit-exact on the GPU's own fp32 scores,
the oracle's own ranking within the tolerance band, the case in which the estimate is exact, and the
argument checks."""
import ctypes

import numpy as np
import pytest
import torch

import paper_2509_24014_b200 as sd
from oracle import sparsed_oracle as orc
from paper_2509_24014_b200 import pattern_metrics as pm
from paper_2509_24014_b200 import synthetic as syn
from tests.parity_util import gpu_select, to_f64
from tests.test_gpu_parity_configs import check_row_list

pytestmark = pytest.mark.gpu
DEV = "cuda"
# fp32 means, a 128-term fp32 dot product and exp2f against fp64: relative error of a probability is the
# absolute error of its logit (<= ~2e-6 * |z|, |z| <= ~15 here) plus a few ulp
EST_RTOL, EST_ATOL = 5e-5, 1e-12


def run_estimate(q, k, bs, rho, prefill, scale=0.0):
    B, Hq, L, _ = q.shape
    nb = L // bs
    params = sd.make_params(bs, rho, prefill)
    kp, kg = sd.sparsed_kept_per_row(params, L)
    pat, rp, ci = sd.new_pattern(B, Hq, nb, kp + kg, DEV)
    scores = torch.full((B, Hq, nb, nb), float("nan"), dtype=torch.float32, device=DEV)
    ws = sd.new_workspace(sd.sparsed_workspace_bytes(sd.OP_SELECT_POOLED_QK, sd.make_shape(q, k), params), DEV)
    sd.sparsed_select_pattern_pooled_qk(q, k, params, pat, ws, scores_out=scores, softmax_scale=scale)
    torch.cuda.synchronize()
    assert sd.sparsed_last_device_status(ws) == (0, 0)
    assert pat.nnz == B * Hq * nb * (kp + kg)
    return pat, rp.cpu().numpy(), ci.cpu().numpy(), scores.cpu().numpy()


@pytest.mark.parametrize("B,Hq,Hkv,L,bs,rho,prefill,scale", [
    (1, 2, 2, 1024, 64, 0.3, 0, 0.0),          # the small exhaustive shape
    (2, 4, 2, 128 * 37, 128, 0.2, 128 * 9, 0.0),  # ragged: 37 blocks (not a multiple of the 32-row or 64-column tiles)
    (1, 3, 1, 32 * 70, 32, 0.5, 32 * 20, 0.13),   # 32-token blocks, grouped heads, custom scale
    (1, 2, 2, 64 * 1024, 64, 0.05, 64 * 512, 0.0),  # the largest row the kernel holds (1024 blocks)
])
def test_estimate_matches_oracle(B, Hq, Hkv, L, bs, rho, prefill, scale):
    cfg = syn.AttnConfig("est", B, Hq, Hkv, L, 128, bs, rho, prefill, seed=500 + bs)
    q, k, _ = syn.make_qkv(cfg, DEV)
    pat, rp, ci, est = run_estimate(q, k, bs, rho, prefill, scale)
    nb, pb = L // bs, prefill // bs
    ref = orc.pooled_qk_scores(to_f64(q), to_f64(k), bs, scale=float(np.float32(scale)) if scale else None)
    np.testing.assert_allclose(est, ref, rtol=EST_RTOL, atol=EST_ATOL)
    np.testing.assert_allclose(est.astype(np.float64).sum(-1), 1.0 / bs, rtol=2e-5)
    rp1, ci1 = orc.select_blocks(est, bs, prefill, rho)          # bit-exact on the GPU's own scores
    np.testing.assert_array_equal(rp, rp1)
    np.testing.assert_array_equal(ci, ci1)
    rows = [(b, h, i) for b in range(B) for h in range(Hq) for i in range(nb)]
    rng = np.random.default_rng(L)
    if len(rows) > 600:
        rows = [rows[j] for j in sorted(rng.choice(len(rows), 600, replace=False))]
    for b, h, i in rows:                                          # the oracle's own ranking, with the band
        r = (b * Hq + h) * nb + i
        check_row_list(ci[rp[r]:rp[r + 1]], ref[b, h, i], pb, rho)


def test_estimate_is_exact_for_block_constant_inputs():
    """Every block constant: the estimate equals A', so it must agree with the exact scorer's scores and,
    where the ranking is clear, with its pattern."""
    B, H, nb, bs = 1, 2, 24, 64
    g = torch.Generator(device="cpu").manual_seed(9)
    qb = (torch.randn(B, H, nb, 128, generator=g) * 0.4).to(torch.bfloat16)
    kb = (torch.randn(B, H, nb, 128, generator=g) * 0.4).to(torch.bfloat16)
    q = qb.repeat_interleave(bs, dim=2).contiguous().to(DEV)
    k = kb.repeat_interleave(bs, dim=2).contiguous().to(DEV)
    _, rp_e, ci_e, est = run_estimate(q, k, bs, 0.25, 0)
    pat_x, rp_x, ci_x, exact = gpu_select(q, k, bs, 0.25, 0)
    exact = exact.cpu().numpy()
    np.testing.assert_allclose(est, exact, rtol=1e-4, atol=1e-9)
    recall = pm.pattern_recall(rp_x.cpu().numpy(), ci_x.cpu().numpy(), rp_e, ci_e, nb)
    assert recall.mean() > 0.99


def test_a_strong_token_under_sign_alternating_queries_is_seen_by_the_exact_scorer_only():
    """Why the paper pools probabilities rather than inputs: one key that half of the queries of every
    block attend to strongly (the other half avoid it). Block means cancel the queries' component, so the
    estimate ranks that key's block by noise; the exact A' ranks it first in every row."""
    cfg = syn.AttnConfig("stripe", 1, 1, 1, 4096, 128, 128, 0.1, 0, seed=77, fixed_heads=(("diffuse",),))
    q, k, _ = syn.make_qkv(cfg, DEV)
    u = torch.zeros(128, device=DEV)
    u[:16] = 1.0
    sign = torch.where(torch.arange(4096, device=DEV) % 2 == 0, 1.0, -1.0)[:, None]
    q = (q.float() + 0.75 * sign * u).to(torch.bfloat16)     # +-0.75 * 3 * 16 / sqrt(128) = +-3.2 logits on the key
    k = k.clone()
    k[0, 0, 1777] = (k[0, 0, 1777].float() + 3.0 * u).to(torch.bfloat16)   # token 1777 lies in block 13
    nb = 32
    _, rp_e, ci_e, est = run_estimate(q, k, 128, 0.1, 0)
    pat_x, rp_x, ci_x, exact = gpu_select(q, k, 128, 0.1, 0)
    rp_x, ci_x = rp_x.cpu().numpy(), ci_x.cpu().numpy()
    assert all(13 in ci_x[rp_x[r]:rp_x[r + 1]] for r in range(nb))
    assert (exact[0, 0].cpu().numpy().argmax(axis=1) == 13).all()
    found = sum(13 in ci_e[rp_e[r]:rp_e[r + 1]] for r in range(nb))
    assert found <= nb // 2, found
    # the oracle shows both behaviours too
    qd, kd = to_f64(q), to_f64(k)
    assert (orc.pooled_scores(qd, kd, 128)[0, 0].argmax(axis=1) == 13).all()
    ref_est = orc.pooled_qk_scores(qd, kd, 128)[0, 0]
    np.testing.assert_allclose(est[0, 0], ref_est, rtol=EST_RTOL, atol=EST_ATOL)
    assert np.abs(ref_est[:, 13] * 128 * nb - 1.0).max() < 0.01   # block 13 looks like any other block


def test_argument_checks():
    q = torch.zeros(1, 1, 256, 128, dtype=torch.bfloat16, device=DEV)
    params = sd.make_params(128, 0.5, 0)
    pat, rp, ci = sd.new_pattern(1, 1, 2, 1, DEV)
    ws = sd.new_workspace(sd.sparsed_workspace_bytes(sd.OP_SELECT_POOLED_QK, sd.make_shape(q, q), params), DEV)
    sd.sparsed_select_pattern_pooled_qk(q, q, params, pat, ws)         # zeros: uniform estimate, ties -> lowest index
    torch.cuda.synchronize()
    assert ci.cpu().tolist() == [0, 0] and rp.cpu().tolist() == [0, 1, 2]
    with pytest.raises(sd.SparsedError) as e:
        sd.sparsed_select_pattern_pooled_qk(q, q, params, pat, ws[:256])   # no room for the means
    assert e.value.status == 4
    big = sd.make_shape(q, q)
    big.seq_len = 32 * 1025                                            # 1025 blocks: more than a row holds
    big.q_strides[1] = big.k_strides[1] = big.seq_len * 128
    big.q_strides[0] = big.k_strides[0] = big.seq_len * 128
    p32 = sd.make_params(32, 0.5, 0)
    pat_big, _, _ = sd.new_pattern(1, 1, 1025, 513, DEV)
    with pytest.raises(sd.SparsedError) as e:
        sd.sparsed_select_pattern_pooled_qk(q, q, p32, pat_big, ws, shape=big)
    assert e.value.status == 2
    with pytest.raises(sd.SparsedError) as e:
        sd.sparsed_select_pattern_pooled_qk(q, q, sd.make_params(16, 0.5, 0), pat, ws)
    assert e.value.status == 2
