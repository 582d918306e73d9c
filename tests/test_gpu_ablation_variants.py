"""The component ablation of the paper (Table 2) as modes of the one-call step: without Sparse Reusing
(every sparse step selects its own pattern from that step's tensors), without Isolated Selection (one
top-k over all key blocks), and both; each against the oracle driven the same way."""
import numpy as np
import pytest
import torch

import paper_2509_24014_b200 as sd
from oracle import sparsed_oracle as orc
from paper_2509_24014_b200 import synthetic as syn
from tests.parity_util import check_outputs, to_f64
from tests.test_gpu_parity_configs import check_row_list

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("variant", [sd.VARIANT_NO_REUSE, sd.VARIANT_NO_ISOLATION,
                                     sd.VARIANT_NO_REUSE | sd.VARIANT_NO_ISOLATION, 0])
@pytest.mark.parametrize("bs,L,rho,prefill", [(128, 1536, 0.25, 512), (64, 1024, 0.3, 384), (32, 512, 0.5, 128)])
def test_ablation_variants_follow_the_oracle(variant, bs, L, rho, prefill):
    T, skip, Hq, Hkv = 5, 0.4, 4, 2
    cfg = syn.AttnConfig("abl", 1, Hq, Hkv, L, 128, bs, rho, prefill, seed=300 + bs, total_steps=T, skip=skip,
                         step_noise=0.1, plant_norm=6.0)
    base = syn.make_base(cfg, DEV)
    nb = L // bs
    p_eff = 0 if variant & sd.VARIANT_NO_ISOLATION else prefill
    params = sd.make_params(bs, rho, prefill)
    kp, kg = sd.sparsed_kept_per_row(sd.make_params(bs, rho, p_eff), L)
    pat, rp_t, ci_t = sd.new_pattern(1, Hq, nb, kp + kg, DEV)
    q0, k0, _ = syn.make_qkv(cfg, DEV, step=1, base=base)
    shape = sd.make_shape(q0, k0)
    ws = sd.new_workspace(max(sd.sparsed_workspace_bytes(sd.OP_ATTENTION_STEP, shape, params),
                              sd.sparsed_workspace_bytes(sd.OP_SELECT_PATTERN, shape, params)), DEV)
    s_switch = orc.switch_step(T, skip)
    assert s_switch == 2
    lists_at = {}
    for step in range(1, T + 1):
        q, k, v = syn.make_qkv(cfg, DEV, step=step, base=base)
        o = torch.empty_like(q)
        mode = sd.sparsed_attention_step_variant(q, k, v, o, params, variant, step, T, skip, pat, ws)
        torch.cuda.synchronize()
        assert mode == orc.schedule_mode(step, T, skip)
        qd, kd, vd = to_f64(q), to_f64(k), to_f64(v)
        selects_now = step == s_switch or (step > s_switch and (variant & sd.VARIANT_NO_REUSE))
        if selects_now:
            rp, ci = rp_t.cpu().numpy().copy(), ci_t.cpu().numpy().copy()
            a_ref = orc.pooled_scores(qd, kd, bs)          # this step's tensors
            n_exact = 0
            for h in range(Hq):
                for ib in range(nb):
                    r = h * nb + ib
                    n_exact += check_row_list(ci[rp[r]:rp[r + 1]], a_ref[0, h, ib], p_eff // bs, rho)
            assert n_exact >= 0.5 * Hq * nb
            lists_at[step] = (rp, ci)
        if step <= s_switch:
            check_outputs(o, orc.attn_full(qd, kd, vd)[0], f"step {step} full")
        else:
            rp, ci = lists_at[step] if (variant & sd.VARIANT_NO_REUSE) else lists_at[s_switch]
            np.testing.assert_array_equal(rp_t.cpu().numpy(), rp)   # reuse: the pattern is left untouched
            np.testing.assert_array_equal(ci_t.cpu().numpy(), ci)
            check_outputs(o, orc.attn_sparse(qd, kd, vd, rp, ci, bs), f"step {step} sparse")
    if variant & sd.VARIANT_NO_REUSE:
        # fresh noise each step: re-selected patterns do differ from the switch step's
        assert any(not np.array_equal(lists_at[s][1], lists_at[s_switch][1]) for s in range(s_switch + 1, T + 1))
    assert sd.sparsed_last_device_status(ws) == (0, 0)
    with pytest.raises(sd.SparsedError) as e:
        sd.sparsed_attention_step_variant(q, k, v, o, params, 8, 1, T, skip, pat, ws)
    assert e.value.status == 1
