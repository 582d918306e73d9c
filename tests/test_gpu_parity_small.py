"""GPU-vs-oracle parity through the C ABI at sizes the oracle finishes in seconds."""
import numpy as np
import pytest
import torch

import paper_2509_24014_b200 as sd
from oracle import sparsed_oracle as orc
from paper_2509_24014_b200 import synthetic as syn
from tests.parity_util import check_outputs, gpu_full, gpu_select, gpu_sparse, to_f64

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _small_cfg(L, Hq=2, Hkv=2, bs=128, rho=0.3, p=0, seed=11):
    return syn.AttnConfig("t", 1, Hq, Hkv, L, 128, bs, rho, p, seed=seed)


# ------------------------------------------------------------------ selection logic (bit exact)
@pytest.mark.parametrize("nb,pb,rho,ties", [(16, 0, 0.3, False), (17, 5, 0.3, True), (64, 32, 0.2, False),
                                            (100, 37, 0.15, True), (128, 0, 0.15, False), (512, 0, 0.1, True),
                                            (256, 128, 0.1, False), (1024, 512, 0.05, True), (5, 5, 1.0, True),
                                            (33, 1, 0.5, True)])
def test_select_from_scores_bit_exact(nb, pb, rho, ties):
    bs = 128
    B, H = 1, 3
    s = syn.random_scores(B * H * nb, nb, seed=nb + pb, device=DEV, ties=ties).view(B, H, nb, nb).contiguous()
    if nb >= 16:
        s[0, 1, 3, 7] = float("-0.0"); s[0, 1, 3, 8] = 0.0; s[0, 2, 2, :] = 0.25
    params = sd.make_params(bs, rho, pb * bs)
    kp, kg = sd.sparsed_kept_per_row(params, nb * bs)
    pat, row_ptr, col_idx = sd.new_pattern(B, H, nb, kp + kg, DEV)
    ws = sd.new_workspace(256, DEV)
    sd.sparsed_select_from_scores(s, params, pat, ws)
    torch.cuda.synchronize()
    rp, ci = orc.select_blocks(s.cpu().numpy(), bs, pb * bs, rho)
    assert (kp, kg) == (orc.kept_per_region(pb, rho), orc.kept_per_region(nb - pb, rho))
    assert pat.nnz == len(ci) and pat.num_blocks == nb and pat.block_size == bs
    np.testing.assert_array_equal(row_ptr.cpu().numpy(), rp)
    np.testing.assert_array_equal(col_idx.cpu().numpy()[: len(ci)], ci)
    assert sd.sparsed_pattern_validate(pat, ws)


# ------------------------------------------------------------------ dense attention
@pytest.mark.parametrize("L,Hq,Hkv", [(128, 1, 1), (256, 2, 2), (384, 4, 2), (200, 2, 1), (1000, 2, 2), (72, 1, 1)])
def test_attn_full_matches_oracle(L, Hq, Hkv):
    cfg = _small_cfg(L, Hq, Hkv).with_(fixed_heads=tuple((("band", "64"),) * Hq))
    q, k, v = syn.make_qkv(cfg, DEV)
    o, lse = gpu_full(q, k, v)
    o_ref, lse_ref = orc.attn_full(to_f64(q), to_f64(k), to_f64(v))
    check_outputs(o, o_ref, f"full L={L}")
    np.testing.assert_allclose(to_f64(lse), lse_ref, atol=2e-5, rtol=2e-6)


def test_attn_full_large_logits_rescale_path():
    # logits spread over tens of units: exercises the running-maximum rescale of O
    cfg = _small_cfg(512, 2, 2)
    q, k, v = syn.make_qkv(cfg, DEV)
    q = (q.float() * 40).to(torch.bfloat16)
    # keys ordered so that the row maximum keeps growing along the key axis
    order = torch.argsort((k[0, 0].float() @ q[0, 0, 0].float()))
    k = k[:, :, order].contiguous(); v = v[:, :, order].contiguous()
    o, lse = gpu_full(q, k, v)
    o_ref, lse_ref = orc.attn_full(to_f64(q), to_f64(k), to_f64(v))
    d = np.abs(to_f64(o) - o_ref)
    assert d.max() <= 2e-2 * max(1.0, np.abs(o_ref).max()) and d.mean() <= 2e-3
    np.testing.assert_allclose(to_f64(lse), lse_ref, atol=1e-4, rtol=2e-6)


def test_attn_full_strided_inputs_and_scale():
    # [B, L, H, D] storage viewed as [B, H, L, D] (the layout a fused QKV projection produces)
    B, H, L, D = 2, 2, 256, 128
    g = torch.Generator(device=DEV); g.manual_seed(5)
    raw = torch.randn(3, B, L, H, D, generator=g, device=DEV).to(torch.bfloat16)
    q, k, v = (raw[i].transpose(1, 2) for i in range(3))
    o = torch.empty(B, L, H, D, dtype=torch.bfloat16, device=DEV).transpose(1, 2)
    ws = sd.new_workspace(256, DEV)
    sd.sparsed_attn_full(q, k, v, o, None, ws, softmax_scale=0.05)
    torch.cuda.synchronize()
    o_ref, _ = orc.attn_full(to_f64(q), to_f64(k), to_f64(v), scale=float(np.float32(0.05)))
    check_outputs(o, o_ref, "strided")


# ------------------------------------------------------------------ config 1 end to end
def test_config1_full_select_sparse():
    cfg = syn.CONFIGS["c1"]
    q, k, v = syn.make_qkv(cfg, DEV)
    qd, kd, vd = to_f64(q), to_f64(k), to_f64(v)
    o, lse = gpu_full(q, k, v)
    o_ref, lse_ref = orc.attn_full(qd, kd, vd)
    check_outputs(o, o_ref, "c1 full")
    pat, row_ptr, col_idx, scores = gpu_select(q, k, cfg.block_size, cfg.keep_ratio, cfg.prefill_len, lse=lse)
    a_ref = orc.pooled_scores(qd, kd, cfg.block_size)
    a_gpu = to_f64(scores)
    np.testing.assert_allclose(a_gpu, a_ref, rtol=2e-5, atol=1e-9)
    np.testing.assert_allclose(a_gpu.sum(-1), 1.0 / cfg.block_size, rtol=2e-5)
    # selection logic bit-exact on the GPU's own fp32 scores
    rp, ci = orc.select_blocks(scores.cpu().numpy(), cfg.block_size, cfg.prefill_len, cfg.keep_ratio)
    np.testing.assert_array_equal(row_ptr.cpu().numpy(), rp)
    np.testing.assert_array_equal(col_idx.cpu().numpy(), ci)
    # same pattern without a precomputed LSE (the library makes its own row-statistics pass)
    pat2, row_ptr2, col_idx2, scores2 = gpu_select(q, k, cfg.block_size, cfg.keep_ratio, cfg.prefill_len, lse=None)
    np.testing.assert_allclose(to_f64(scores2), a_ref, rtol=2e-5, atol=1e-9)
    # sparse attention on the GPU's pattern vs the oracle on the same pattern
    o_sp = gpu_sparse(q, k, v, pat)
    o_sp_ref = orc.attn_sparse(qd, kd, vd, rp, ci, cfg.block_size)
    check_outputs(o_sp, o_sp_ref, "c1 sparse")
    # negative controls: zeros and the other head's pattern must fail the same check
    with pytest.raises(AssertionError):
        check_outputs(torch.zeros_like(o_sp), o_sp_ref, "zeros")
    nb, kk = cfg.num_blocks, 5
    swapped = torch.cat([col_idx[nb * kk:], col_idx[: nb * kk]]).contiguous()
    pat_sw = sd.pattern_from_csr(row_ptr, swapped, cfg.block_size, nb, 1, 2)
    with pytest.raises(AssertionError):
        check_outputs(gpu_sparse(q, k, v, pat_sw), o_sp_ref, "swapped pattern")


@pytest.mark.parametrize("bs,L,Hq,Hkv,p", [(128, 512, 2, 2, 256), (64, 448, 4, 2, 128), (128, 1024, 7, 1, 0)])
def test_sparse_all_kept_equals_full_and_user_csr(bs, L, Hq, Hkv, p):
    cfg = _small_cfg(L, Hq, Hkv, bs, 1.0, p)
    q, k, v = syn.make_qkv(cfg, DEV)
    pat, row_ptr, col_idx, _ = gpu_select(q, k, bs, 1.0, p)
    nb = L // bs
    assert torch.equal(col_idx.cpu(), torch.arange(nb, dtype=torch.int32).repeat(Hq * nb))
    o_full, _ = gpu_full(q, k, v)
    o_sp = gpu_sparse(q, k, v, pat)
    o_ref, _ = orc.attn_full(to_f64(q), to_f64(k), to_f64(v))
    check_outputs(o_sp, o_ref, "all kept")
    assert (o_sp.float() - o_full.float()).abs().max().item() <= 2e-2
    # a hand-made ragged CSR: row r keeps (r % 3) + 1 blocks
    lists = [sorted(np.random.default_rng(r).choice(nb, size=(r % 3) + 1, replace=False).tolist())
             for r in range(Hq * nb)]
    rp = np.cumsum([0] + [len(x) for x in lists]).astype(np.int32)
    ci = np.concatenate(lists).astype(np.int32)
    rp_d, ci_d = torch.from_numpy(rp).to(DEV), torch.from_numpy(ci).to(DEV)  # keep alive: the struct holds raw pointers
    pat_u = sd.pattern_from_csr(rp_d, ci_d, bs, nb, 1, Hq)
    ws = sd.new_workspace(256, DEV)
    assert sd.sparsed_pattern_validate(pat_u, ws)
    o_u = gpu_sparse(q, k, v, pat_u)
    check_outputs(o_u, orc.attn_sparse(to_f64(q), to_f64(k), to_f64(v), rp, ci, bs), "user csr")
