"""One layer's heads split over ranks (whole grouped-query groups per rank): the shards run one after
the other on this GPU, each through the ordinary one-call step on head-offset views, and the
results must be bitwise what the unsharded call gives: outputs of every step, and the selected
pattern once the shard patterns are merged back into the single-device row order."""
import numpy as np
import pytest
import torch

import paper_2509_24014_b200 as sd
from paper_2509_24014_b200 import replicas
from paper_2509_24014_b200 import synthetic as syn

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("B,Hq,Hkv,L,bs,rho,p,world", [(1, 8, 4, 2048, 128, 0.25, 1024, 2), (2, 12, 4, 768, 64, 0.3, 0, 4),
                                                     (1, 4, 4, 512, 32, 0.5, 128, 2)])
def test_head_shards_equal_the_unsharded_layer_bitwise(B, Hq, Hkv, L, bs, rho, p, world):
    T, skip = 4, 0.5
    cfg = syn.AttnConfig("shard", B, Hq, Hkv, L, 128, bs, rho, p, seed=77, total_steps=T, skip=skip, step_noise=0.05)
    base = syn.make_base(cfg, DEV)
    params = sd.make_params(bs, rho, p)
    nb = L // bs
    kp, kg = sd.sparsed_kept_per_row(params, L)
    pat, rp_t, ci_t = sd.new_pattern(B, Hq, nb, kp + kg, DEV)
    shards = [replicas.plan_head_shard(B, Hq, Hkv, L, params, world, r, DEV) for r in range(world)]
    assert sorted(h for s in shards for h in s.heads) == list(range(Hq))
    q0, k0, _ = syn.make_qkv(cfg, DEV, step=1, base=base)
    ws = sd.new_workspace(sd.sparsed_workspace_bytes(sd.OP_ATTENTION_STEP, sd.make_shape(q0, k0), params), DEV)
    for step in range(1, T + 1):
        q, k, v = syn.make_qkv(cfg, DEV, step=step, base=base)
        o_ref = torch.empty_like(q)
        mode = sd.sparsed_attention_step(q, k, v, o_ref, params, step, T, skip, pat, ws)
        o = torch.full_like(q, float("nan"))
        for s in shards:
            assert replicas.head_shard_step(s, q, k, v, o, step, T, skip) == mode
        torch.cuda.synchronize()
        assert torch.equal(o, o_ref), f"step {step}"
        if mode == sd.MODE_FULL_AND_SELECT:
            parts = [(list(s.heads), s.row_ptr.cpu().numpy(), s.col_idx.cpu().numpy()) for s in shards]
            assert all(part[1][0] == 0 for part in parts)
            rp, ci = replicas.merge_shard_patterns(parts, B, Hq, nb)
            np.testing.assert_array_equal(rp, rp_t.cpu().numpy())
            np.testing.assert_array_equal(ci, ci_t.cpu().numpy()[: int(pat.nnz)])
    for s in shards:
        assert sd.sparsed_last_device_status(s.ws) == (0, 0)
    assert sd.sparsed_last_device_status(ws) == (0, 0)
