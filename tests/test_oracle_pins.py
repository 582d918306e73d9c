"""Pins for the CPU oracle: closed forms, a library routine, brute force and invariants.

None of the expected values below comes from the CUDA path or from the oracle itself:
they are closed forms worked by hand (tests/golden), torch's scaled_dot_product_attention
in fp64, the scalar-loop brute force, or properties that follow from Eq. 1-6.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import brute_force as bf
from oracle import sparsed_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                out.append([float(x) for x in line.split()])
    return out


def _rand(shape, seed, scale=1.0):
    return np.random.default_rng(seed).standard_normal(shape) * scale


def _qkv(B, Hq, Hkv, L, D, seed, qscale=1.0):
    return (_rand((B, Hq, L, D), seed, qscale), _rand((B, Hkv, L, D), seed + 1, qscale),
            _rand((B, Hkv, L, D), seed + 2))


# ------------------------------------------------------------------ Eq. 1 (full attention)
def test_full_two_key_closed_form():
    p0, p1, out, lse = _rows("two_key_softmax.txt")[0]
    q = np.array([[[[1.0]]]])
    k = np.array([[[[0.0], [math.log(3.0)]]]])
    v = np.array([[[[8.0], [4.0]]]])
    o, l = orc.attn_full(q, k, v)
    assert o[0, 0, 0, 0] == pytest.approx(out, abs=1e-14)
    assert l[0, 0, 0] == pytest.approx(lse, abs=1e-14)
    p, _ = orc.softmax_rows(q[0, 0], k[0, 0], slice(0, 1))
    assert p[0] == pytest.approx([p0, p1], abs=1e-15)
    # d = 4 version pins the 1/sqrt(d) factor
    q4 = np.zeros((1, 1, 1, 4)); q4[..., 0] = 2.0
    k4 = np.zeros((1, 1, 2, 4)); k4[0, 0, 1, 0] = math.log(3.0)
    o4, l4 = orc.attn_full(q4, k4, v)
    assert o4[0, 0, 0, 0] == pytest.approx(out, abs=1e-14)
    assert l4[0, 0, 0] == pytest.approx(lse, abs=1e-14)


@pytest.mark.parametrize("Hq,Hkv", [(2, 2), (6, 2)])
def test_full_matches_library_sdpa(Hq, Hkv):
    q, k, v = _qkv(2, Hq, Hkv, 96, 16, 10)
    o, lse = orc.attn_full(q, k, v, block_rows=32)
    g = Hq // Hkv
    tk = torch.from_numpy(k).repeat_interleave(g, dim=1)
    tv = torch.from_numpy(v).repeat_interleave(g, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(torch.from_numpy(q), tk, tv)
    np.testing.assert_allclose(o, ref.numpy(), rtol=1e-12, atol=1e-13)
    s = torch.einsum("bhid,bhjd->bhij", torch.from_numpy(q), tk) / math.sqrt(16)
    np.testing.assert_allclose(lse, torch.logsumexp(s, dim=-1).numpy(), rtol=1e-12, atol=1e-13)


def test_full_matches_brute_force_and_rows_sum_to_one():
    q, k, v = _qkv(1, 1, 1, 24, 5, 20)
    o, _ = orc.attn_full(q, k, v, block_rows=8)
    a = bf.score_matrix(q[0, 0], k[0, 0])
    np.testing.assert_allclose(a.sum(axis=1), 1.0, atol=1e-14)
    np.testing.assert_allclose(o[0, 0], bf.attend(a, v[0, 0]), rtol=1e-12, atol=1e-13)
    p, _ = orc.softmax_rows(q[0, 0], k[0, 0], slice(0, 24))
    np.testing.assert_allclose(p.sum(axis=1), 1.0, atol=1e-14)
    np.testing.assert_allclose(p, a, atol=1e-14)


def test_full_zero_query_gives_mean_of_values_and_dominant_key_gives_its_value():
    q, k, v = _qkv(1, 2, 2, 40, 8, 30)
    o, lse = orc.attn_full(np.zeros_like(q), k, v)
    np.testing.assert_allclose(o[0, 1, 7], v[0, 1].mean(axis=0), atol=1e-14)
    np.testing.assert_allclose(lse, math.log(40), atol=1e-14)
    # one key aligned with the query and huge: output -> that key's value row
    k2 = k.copy(); k2[0, 0, 13] = 200.0 * q[0, 0, 5] / np.linalg.norm(q[0, 0, 5])
    o2, _ = orc.attn_full(q * 50.0, k2, v)
    np.testing.assert_allclose(o2[0, 0, 5], v[0, 0, 13], atol=1e-9)


def test_full_is_not_causal():
    # the last key must influence the first query (bidirectional attention)
    q, k, v = _qkv(1, 1, 1, 16, 4, 40)
    o1, _ = orc.attn_full(q, k, v)
    v2 = v.copy(); v2[0, 0, -1] += 10.0
    o2, _ = orc.attn_full(q, k, v2)
    assert np.abs(o2[0, 0, 0] - o1[0, 0, 0]).max() > 1e-3


# ------------------------------------------------------------------ avgpool(A)
@pytest.mark.parametrize("L,bs,D", [(32, 4, 8), (64, 8, 4), (24, 8, 3)])
def test_pooled_matches_brute_force(L, bs, D):
    q, k, _ = _qkv(1, 2, 1, L, D, 50)
    ap = orc.pooled_scores(q, k, bs)
    for h in range(2):
        ref = bf.avgpool(bf.score_matrix(q[0, h], k[0, 0]), bs)
        np.testing.assert_allclose(ap[0, h], ref, rtol=1e-12, atol=1e-15)


def test_pooled_invariants():
    L, bs, D = 96, 8, 6
    nb = L // bs
    q, k, _ = _qkv(1, 1, 1, L, D, 60, qscale=1.5)
    ap = orc.pooled_scores(q, k, bs)[0, 0]
    # every block-row of A' sums to 1/bs (softmax rows sum to 1, mean over bs*bs cells)
    np.testing.assert_allclose(ap.sum(axis=1), 1.0 / bs, rtol=1e-13)
    # Q = 0 -> uniform attention -> every cell equals 1/L
    a0 = orc.pooled_scores(np.zeros_like(q), k, bs)[0, 0]
    np.testing.assert_allclose(a0, 1.0 / L, rtol=1e-13)
    # permuting keys inside a key block leaves A' unchanged
    perm = np.arange(L); perm[16:24] = perm[16:24][::-1]; perm[40:48] = np.roll(perm[40:48], 3)
    a1 = orc.pooled_scores(q, k[:, :, perm], bs)[0, 0]
    np.testing.assert_allclose(a1, ap, rtol=1e-12, atol=1e-18)
    # permuting whole key blocks permutes the columns of A'
    bperm = np.random.default_rng(1).permutation(nb)
    tperm = (bperm[:, None] * bs + np.arange(bs)[None, :]).reshape(-1)
    a2 = orc.pooled_scores(q, k[:, :, tperm], bs)[0, 0]
    np.testing.assert_allclose(a2, ap[:, bperm], rtol=1e-12, atol=1e-18)
    # pooling is over probabilities, not logits: a planted dominant block gets nearly all mass
    k3 = k.copy(); k3[0, 0, 24:32] += 6.0 * q[0, 0, 0:8].mean(axis=0) / np.linalg.norm(q[0, 0, 0:8].mean(axis=0))
    q3 = q.copy(); q3[0, 0, 0:8] = 8.0 * q[0, 0, 0:8].mean(axis=0)
    a3 = orc.pooled_scores(q3, k3, bs)[0, 0]
    assert a3[0].argmax() == 3 and a3[0, 3] > 0.9 / bs


# ------------------------------------------------------------------ block-mean estimate of A'
def test_pooled_qk_estimate_is_a_library_softmax_at_block_size_one():
    from scipy.special import softmax
    L, D = 20, 6
    q, k, _ = _qkv(2, 4, 2, L, D, 70, qscale=1.3)
    est = orc.pooled_qk_scores(q, k, 1)
    for b in range(2):
        for h in range(4):
            ref = softmax((q[b, h] @ k[b, h // 2].T) / math.sqrt(D), axis=1)
            np.testing.assert_allclose(est[b, h], ref, rtol=1e-12, atol=1e-16)
    # and a custom scale is applied to the logits, not to the probabilities
    est2 = orc.pooled_qk_scores(q, k, 1, scale=0.37)
    np.testing.assert_allclose(est2[1, 3], softmax(0.37 * (q[1, 3] @ k[1, 1].T), axis=1), rtol=1e-12)


def test_pooled_qk_estimate_is_exact_for_block_constant_inputs_and_only_then():
    L, bs, D = 48, 8, 5
    nb = L // bs
    qb, kb, _ = _qkv(1, 2, 1, nb, D, 71, qscale=1.7)
    q = np.repeat(qb, bs, axis=2)
    k = np.repeat(kb, bs, axis=2)
    est = orc.pooled_qk_scores(q, k, bs)
    np.testing.assert_allclose(est, orc.pooled_scores(q, k, bs), rtol=1e-12, atol=1e-18)
    np.testing.assert_allclose(est.sum(axis=-1), 1.0 / bs, rtol=1e-13)
    # one strong key hidden among weak ones of its block: the exact A' sees it, the mean washes it out
    q2, k2, _ = _qkv(1, 1, 1, L, D, 72, qscale=0.05)
    u = np.ones(D) / math.sqrt(D)
    q2[0, 0] += 3.0 * u
    k2[0, 0, 19] += 12.0 * u          # token 19 lies in key block 2
    exact = orc.pooled_scores(q2, k2, bs)[0, 0]
    approx = orc.pooled_qk_scores(q2, k2, bs)[0, 0]
    assert (exact.argmax(axis=1) == 2).all() and (approx.argmax(axis=1) == 2).all()
    assert exact[:, 2].min() > 0.99 / bs and approx[:, 2].max() < 0.7 / bs


# ------------------------------------------------------------------ Eq. 5 / Eq. 6 (selection)
def test_kept_blocks_table():
    for n, rho, kept in _rows("kept_blocks_table.txt"):
        assert orc.kept_per_region(int(n), rho) == int(kept)
    assert orc.kept_per_region(10, 0.3, "floor") == 3
    assert orc.kept_per_region(10, 0.35, "floor") == 3
    assert orc.kept_per_region(10, 0.35, "ceil") == 4


@pytest.mark.parametrize("pb", [0, 3, 6, 12])
def test_select_matches_brute_force(pb):
    rng = np.random.default_rng(70 + pb)
    nb, bs, rho = 12, 4, 0.3
    scores = rng.random((1, 2, nb, nb))
    scores[0, 0, 2, 5] = scores[0, 0, 2, 9] = scores[0, 0, 2, 1]  # ties
    rp, ci = orc.select_blocks(scores, bs, pb * bs, rho)
    kpre, kgen = orc.kept_per_region(pb, rho), orc.kept_per_region(nb - pb, rho)
    for h in range(2):
        rows = bf.select(scores[0, h], pb, kpre, kgen)
        for ib in range(nb):
            r = h * nb + ib
            assert list(ci[rp[r]:rp[r + 1]]) == rows[ib]
    assert rp[-1] == len(ci) == 2 * nb * (kpre + kgen)


def test_select_ties_all_equal_keeps_lowest_indices_per_region():
    nb, bs = 10, 2
    scores = np.full((1, 1, nb, nb), 0.1, dtype=np.float32)
    rp, ci = orc.select_blocks(scores, bs, 4 * bs, 0.5)
    assert list(ci[rp[0]:rp[1]]) == [0, 1, 4, 5, 6]
    # and from real inputs: Q = 0 makes every pooled score equal
    q, k, _ = _qkv(1, 1, 1, 20, 4, 80)
    ap = orc.pooled_scores(np.zeros_like(q), k, bs)
    rp, ci = orc.select_blocks(ap.astype(np.float32), bs, 0, 0.3)
    assert list(ci[rp[3]:rp[4]]) == [0, 1, 2]


def test_select_properties():
    rng = np.random.default_rng(90)
    nb, bs = 16, 4
    scores = rng.random((2, 3, nb, nb)).astype(np.float32)
    scores[1, 2, 7, 11] = 5.0  # planted dominant block must be kept
    rp, ci = orc.select_blocks(scores, bs, 8 * bs, 0.25)
    k_pre = k_gen = 2
    assert np.all(np.diff(rp) == k_pre + k_gen)
    for r in range(len(rp) - 1):
        row = ci[rp[r]:rp[r + 1]]
        assert np.all(np.diff(row) > 0)
        assert np.sum(row < 8) == k_pre
    r = (1 * 3 + 2) * nb + 7
    assert 11 in ci[rp[r]:rp[r + 1]]
    # rho = 1 keeps every block
    rp1, ci1 = orc.select_blocks(scores, bs, 8 * bs, 1.0)
    assert list(ci1[:nb]) == list(range(nb))
    # p = 0 and p = L are the plain (un-isolated) top-k of the whole row
    for p in (0, nb * bs):
        rp2, ci2 = orc.select_blocks(scores, bs, p, 0.25)
        top = np.sort(np.argsort(-scores[0, 0, 0].astype(np.float64), kind="stable")[:4])
        assert list(ci2[rp2[0]:rp2[1]]) == list(top)
    # isolation matters: a row whose best blocks are all prefill still keeps generation blocks
    s3 = np.zeros((1, 1, 1, 8)); s3[0, 0, 0] = [9, 8, 7, 6, 0.4, 0.1, 0.3, 0.2]
    _, ci3 = orc.select_blocks(np.repeat(s3, 8, axis=2), 1, 4, 0.5)
    assert list(ci3[:4]) == [0, 1, 4, 6]


# ------------------------------------------------------------------ Eq. 3 / Eq. 4 (sparse attention)
def _all_kept(B, Hq, nb):
    rows = B * Hq * nb
    return (np.arange(rows + 1, dtype=np.int32) * nb,
            np.tile(np.arange(nb, dtype=np.int32), rows))


def test_sparse_all_blocks_kept_equals_full():
    q, k, v = _qkv(1, 4, 2, 64, 8, 100)
    rp, ci = _all_kept(1, 4, 8)
    o_full, _ = orc.attn_full(q, k, v)
    np.testing.assert_allclose(orc.attn_sparse(q, k, v, rp, ci, 8), o_full, rtol=1e-12, atol=1e-14)


def test_sparse_matches_library_masked_sdpa_and_brute_force():
    B, Hq, Hkv, L, D, bs = 1, 2, 1, 48, 6, 8
    nb = L // bs
    q, k, v = _qkv(B, Hq, Hkv, L, D, 110)
    ap = orc.pooled_scores(q, k, bs)
    rp, ci = orc.select_blocks(ap, bs, 24, 0.34)
    o = orc.attn_sparse(q, k, v, rp, ci, bs)
    mask = torch.zeros(B, Hq, L, L, dtype=torch.bool)
    for h in range(Hq):
        for ib in range(nb):
            r = h * nb + ib
            for jb in ci[rp[r]:rp[r + 1]]:
                mask[0, h, ib * bs:(ib + 1) * bs, jb * bs:(jb + 1) * bs] = True
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(k).expand(B, Hq, L, D), torch.from_numpy(v).expand(B, Hq, L, D),
        attn_mask=mask)
    np.testing.assert_allclose(o, ref.numpy(), rtol=1e-12, atol=1e-13)
    for h in range(Hq):
        rows = [list(ci[rp[h * nb + ib]:rp[h * nb + ib + 1]]) for ib in range(nb)]
        a = bf.score_matrix(q[0, h], k[0, 0], bf.token_mask(rows, bs, L))
        np.testing.assert_allclose(o[0, h], bf.attend(a, v[0, 0]), rtol=1e-12, atol=1e-13)


def test_sparse_single_kept_block_is_attention_over_that_block():
    q, k, v = _qkv(1, 1, 1, 32, 4, 120)
    bs, nb = 8, 4
    rp = np.arange(nb + 1, dtype=np.int32)
    ci = np.array([2, 0, 3, 1], dtype=np.int32)
    o = orc.attn_sparse(q, k, v, rp, ci, bs)
    for ib in range(nb):
        jb = ci[ib]
        sub_o, _ = orc.attn_full(q[:, :, ib * bs:(ib + 1) * bs], k[:, :, jb * bs:(jb + 1) * bs],
                                 v[:, :, jb * bs:(jb + 1) * bs])
        np.testing.assert_allclose(o[0, 0, ib * bs:(ib + 1) * bs], sub_o[0, 0], rtol=1e-12, atol=1e-14)


def test_batch_two_gqa_and_custom_scale_against_library_routines_and_brute_force():
    """Row indexing over (batch, head, query block) and the `scale` argument of the full, pooled and
    masked paths: different data per batch entry, grouped heads, scale 0.37, against torch's SDPA
    (mask and scale given to the library), torch's avg_pool2d of a library softmax, and the scalar
    brute force (which knows only 1/sqrt(d): the scale is folded into the queries first)."""
    B, Hq, Hkv, L, D, bs, scale = 2, 4, 2, 48, 6, 8, 0.37
    nb, g = L // bs, Hq // Hkv
    q, k, v = _qkv(B, Hq, Hkv, L, D, 140, qscale=1.4)
    tq = torch.from_numpy(q)
    tk = torch.from_numpy(k).repeat_interleave(g, dim=1)
    tv = torch.from_numpy(v).repeat_interleave(g, dim=1)
    # Eq. 1 with a custom scale
    o, lse = orc.attn_full(q, k, v, scale=scale, block_rows=8)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, scale=scale)
    np.testing.assert_allclose(o, ref.numpy(), rtol=1e-12, atol=1e-13)
    logits = scale * torch.einsum("bhid,bhjd->bhij", tq, tk)
    np.testing.assert_allclose(lse, torch.logsumexp(logits, dim=-1).numpy(), rtol=1e-12, atol=1e-13)
    # avgpool(A): library softmax + library average pooling, every (batch, head)
    ap = orc.pooled_scores(q, k, bs, scale=scale)
    pooled_ref = torch.nn.functional.avg_pool2d(torch.softmax(logits, dim=-1).reshape(B * Hq, 1, L, L), bs)
    np.testing.assert_allclose(ap.reshape(B * Hq, nb, nb), pooled_ref[:, 0].numpy(), rtol=1e-12, atol=1e-16)
    assert np.abs(ap[0] - ap[1]).max() > 1e-4          # the two batch entries really differ
    # and the brute force, with the scale folded into q (scale * q.k = (q * scale * sqrt(D)).k / sqrt(D))
    qf = q * (scale * math.sqrt(D))
    for b, h in ((0, 1), (1, 0), (1, 3)):
        np.testing.assert_allclose(ap[b, h], bf.avgpool(bf.score_matrix(qf[b, h], k[b, h // g]), bs),
                                   rtol=1e-12, atol=1e-15)
    # Eq. 3 / Eq. 4 with per-(batch, head, block) lists that differ everywhere
    rp, ci = orc.select_blocks(ap, bs, 24, 0.4)
    assert rp[-1] == B * Hq * nb * 4
    o_sp = orc.attn_sparse(q, k, v, rp, ci, bs, scale=scale)
    mask = torch.zeros(B, Hq, L, L, dtype=torch.bool)
    lists = {}
    for b in range(B):
        for h in range(Hq):
            for ib in range(nb):
                r = (b * Hq + h) * nb + ib
                lists[(b, h, ib)] = list(ci[rp[r]:rp[r + 1]])
                for jb in lists[(b, h, ib)]:
                    mask[b, h, ib * bs:(ib + 1) * bs, jb * bs:(jb + 1) * bs] = True
    assert len({tuple(x) for x in lists.values()}) > 4
    ref_sp = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=mask, scale=scale)
    np.testing.assert_allclose(o_sp, ref_sp.numpy(), rtol=1e-12, atol=1e-13)
    for b, h in ((1, 2), (0, 3)):
        rows = [lists[(b, h, ib)] for ib in range(nb)]
        a = bf.score_matrix(qf[b, h], k[b, h // g], bf.token_mask(rows, bs, L))
        np.testing.assert_allclose(o_sp[b, h], bf.attend(a, v[b, h // g]), rtol=1e-12, atol=1e-13)
    # head_sparse_rows / head_pooled_row (the per-row-block forms the sampled GPU tests use) agree
    np.testing.assert_allclose(orc.head_pooled_row(q[1, 2], k[1, 1], 3, bs, scale=scale), ap[1, 2, 3], rtol=1e-13)
    np.testing.assert_allclose(orc.head_sparse_rows(q[1, 2], k[1, 1], v[1, 1], 3, lists[(1, 2, 3)], bs, scale=scale),
                               o_sp[1, 2, 3 * bs:4 * bs], rtol=1e-13)


# ------------------------------------------------------------------ schedule (Algorithm 1)
def test_schedule_table():
    for T, skip, s, n_full, n_sparse in _rows("schedule_table.txt"):
        T, s = int(T), int(s)
        assert orc.switch_step(T, skip) == s
        modes = [orc.schedule_mode(t, T, skip) for t in range(1, T + 1)]
        assert modes.count(orc.FULL) + modes.count(orc.FULL_AND_SELECT) == int(n_full)
        assert modes.count(orc.SPARSE) == int(n_sparse)
        assert modes.count(orc.FULL_AND_SELECT) == 1 and modes[s - 1] == orc.FULL_AND_SELECT
        assert modes == sorted(modes)
    with pytest.raises(ValueError):
        orc.schedule_mode(0, 4, 0.5)
    with pytest.raises(ValueError):
        orc.schedule_mode(5, 4, 0.5)


def test_algorithm_1_composition():
    q, k, v = _qkv(1, 2, 2, 32, 4, 130)
    T, rho, skip, bs = 5, 0.5, 0.4, 8
    pattern = None
    outs = []
    for t in range(1, T + 1):
        o, pattern = orc.sparsed_attention(q, k, v, t, T, rho, skip, bs, 16, pattern)
        outs.append(o)
        assert (pattern is None) == (t < 2)
    full, _ = orc.attn_full(q, k, v)
    np.testing.assert_array_equal(outs[0], full)
    np.testing.assert_array_equal(outs[1], full)  # the switch step still returns full attention
    np.testing.assert_array_equal(outs[2], orc.attn_sparse(q, k, v, pattern[0], pattern[1], bs))
    assert np.abs(outs[2] - full).max() > 1e-6
    with pytest.raises(ValueError):
        orc.sparsed_attention(q, k, v, 4, T, rho, skip, bs, 16, None)
