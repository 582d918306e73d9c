"""Algorithm 1 through the single-call entry point: every step of a short denoising schedule on the GPU
against the oracle's step-by-step composition, on inputs that change from step to step, for every block
size (the switch step selects from the row statistics of its own full-attention pass)."""
import numpy as np
import pytest
import torch

import paper_2509_24014_b200 as sd
from oracle import sparsed_oracle as orc
from paper_2509_24014_b200 import synthetic as syn
from tests.parity_util import check_outputs, to_f64

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("bs,L,rho,prefill,T,skip", [
    (64, 1024, 0.3, 0, 5, 0.4),        # switch at step 2, selection from the full pass's statistics
    (128, 1536, 0.25, 512, 4, 0.5),    # isolated regions, switch at step 2
    (32, 512, 0.5, 128, 4, 0.25),      # 32-token blocks: one statistic per 32 keys
    (64, 768, 0.3, 0, 3, 0.0),         # skip = 0: the first step is the switch step
])
def test_schedule_through_one_entry_point(bs, L, rho, prefill, T, skip):
    cfg = syn.AttnConfig("step", 1, 4, 2, L, 128, bs, rho, prefill, seed=900 + bs, total_steps=T, skip=skip,
                         step_noise=0.05)
    base = syn.make_base(cfg, DEV)
    nb = L // bs
    params = sd.make_params(bs, rho, prefill)
    kp, kg = sd.sparsed_kept_per_row(params, L)
    pat, rp_t, ci_t = sd.new_pattern(1, 4, nb, kp + kg, DEV)
    q0, k0, _ = syn.make_qkv(cfg, DEV, step=1, base=base)
    ws = sd.new_workspace(sd.sparsed_workspace_bytes(sd.OP_ATTENTION_STEP, sd.make_shape(q0, k0), params), DEV)
    s_switch = orc.switch_step(T, skip)
    pattern_ref = None
    modes = []
    for step in range(1, T + 1):
        q, k, v = syn.make_qkv(cfg, DEV, step=step, base=base)
        o = torch.empty_like(q)
        # only the switch step needs the large workspace
        ws_step = ws if step == s_switch else ws[: sd.sparsed_workspace_bytes(sd.OP_ATTN_FULL)]
        mode = sd.sparsed_attention_step(q, k, v, o, params, step, T, skip, pat, ws_step)
        torch.cuda.synchronize()
        modes.append(mode)
        assert mode == orc.schedule_mode(step, T, skip)
        qd, kd, vd = to_f64(q), to_f64(k), to_f64(v)
        if step <= s_switch:
            o_ref = orc.sparsed_attention(qd, kd, vd, step, T, rho, skip, bs, prefill)[0]
            check_outputs(o, o_ref, f"step {step} (full)")
            if step == s_switch:
                # the GPU's pattern: valid, the right counts, and the oracle's wherever the ranking is clear
                rp, ci = rp_t.cpu().numpy(), ci_t.cpu().numpy()
                a_ref = orc.pooled_scores(qd, kd, bs)
                rp64, ci64 = orc.select_blocks(a_ref, bs, prefill, rho)
                np.testing.assert_array_equal(rp, rp64)
                same = sum(list(ci[rp[r]:rp[r + 1]]) == list(ci64[rp64[r]:rp64[r + 1]]) for r in range(4 * nb))
                assert same >= 0.5 * 4 * nb, same
                pattern_ref = (rp, ci)
        else:
            o_ref, _ = orc.sparsed_attention(qd, kd, vd, step, T, rho, skip, bs, prefill, pattern=pattern_ref)
            check_outputs(o, o_ref, f"step {step} (sparse)")
    assert modes == [sd.MODE_FULL] * (s_switch - 1) + [sd.MODE_FULL_AND_SELECT] + [sd.MODE_SPARSE] * (T - s_switch)
    assert sd.sparsed_last_device_status(ws) == (0, 0)


def test_schedule_at_config2_size_sampled():
    """The LLaDA-shaped 8k layer (32 heads, 4096 prompt + 4096 generation tokens) through the one-call
    entry point, with fresh noise each step: step 1 full, step 2 full + selection from that pass's row
    statistics, steps 3-4 sparse on the kept pattern. The oracle follows on sampled (head, query block)
    rows, including the two blocks next to the prompt boundary."""
    from tests.test_gpu_parity_configs import check_row_list
    cfg = syn.CONFIGS["c2"].with_(total_steps=4, skip=0.5, step_noise=0.05)
    T, skip, bs, nb, pb = 4, 0.5, cfg.block_size, cfg.num_blocks, cfg.prefill_len // cfg.block_size
    base = syn.make_base(cfg, DEV)
    params = sd.make_params(bs, cfg.keep_ratio, cfg.prefill_len)
    kp, kg = sd.sparsed_kept_per_row(params, cfg.seq_len)
    assert (kp, kg) == (7, 7)
    pat, rp_t, ci_t = sd.new_pattern(1, cfg.heads_q, nb, kp + kg, DEV)
    q0, k0, _ = syn.make_qkv(cfg, DEV, step=1, base=base)
    ws = sd.new_workspace(sd.sparsed_workspace_bytes(sd.OP_ATTENTION_STEP, sd.make_shape(q0, k0), params), DEV)
    heads, blocks = (0, 13, 31), (0, pb - 1, pb, nb - 1)
    rp = ci = None
    for step in range(1, T + 1):
        q, k, v = syn.make_qkv(cfg, DEV, step=step, base=base)
        o = torch.empty_like(q)
        mode = sd.sparsed_attention_step(q, k, v, o, params, step, T, skip, pat, ws)
        torch.cuda.synchronize()
        assert mode == orc.schedule_mode(step, T, skip)
        if step == 2:
            rp, ci = rp_t.cpu().numpy(), ci_t.cpu().numpy()
            assert pat.nnz == 32 * nb * 14 and sd.sparsed_pattern_validate(pat, sd.new_workspace(256, DEV))
        for h in heads:
            qh, kh, vh = to_f64(q[0, h]), to_f64(k[0, h]), to_f64(v[0, h])
            for ib in blocks:
                rows = slice(ib * bs, (ib + 1) * bs)
                r = h * nb + ib
                if mode != sd.MODE_SPARSE:
                    check_outputs(o[0, h, rows], orc.head_full_rows(qh, kh, vh, rows)[0], f"step {step} full h{h} ib{ib}")
                    if mode == sd.MODE_FULL_AND_SELECT:
                        check_row_list(ci[rp[r]:rp[r + 1]], orc.head_pooled_row(qh, kh, ib, bs), pb, cfg.keep_ratio)
                else:
                    ref = orc.head_sparse_rows(qh, kh, vh, ib, ci[rp[r]:rp[r + 1]], bs)
                    check_outputs(o[0, h, rows], ref, f"step {step} sparse h{h} ib{ib}")
    assert sd.sparsed_last_device_status(ws) == (0, 0)


def test_step_argument_checks():
    cfg = syn.AttnConfig("step", 1, 1, 1, 256, 128, 128, 0.5, 0, seed=1)
    q, k, v = syn.make_qkv(cfg, DEV)
    o = torch.empty_like(q)
    params = sd.make_params(128, 0.5, 0)
    pat, _, _ = sd.new_pattern(1, 1, 2, 1, DEV)
    ws = sd.new_workspace(sd.sparsed_workspace_bytes(sd.OP_ATTENTION_STEP, sd.make_shape(q, k), params), DEV)
    for bad_step, T, skip in ((0, 4, 0.5), (5, 4, 0.5), (1, 4, 1.5)):
        with pytest.raises(sd.SparsedError) as e:
            sd.sparsed_attention_step(q, k, v, o, params, bad_step, T, skip, pat, ws)
        assert e.value.status == 1
    with pytest.raises(sd.SparsedError) as e:     # the switch step with a status-only workspace
        sd.sparsed_attention_step(q, k, v, o, params, 2, 4, 0.5, pat, ws[:256])
    assert e.value.status == 4
    assert sd.sparsed_attention_step(q, k, v, o, params, 2, 4, 0.5, pat, ws) == sd.MODE_FULL_AND_SELECT
    assert sd.sparsed_attention_step(q, k, v, o, params, 3, 4, 0.5, pat, ws[:256]) == sd.MODE_SPARSE
    torch.cuda.synchronize()
    assert sd.sparsed_last_device_status(ws) == (0, 0)
