"""The seeded input generator: determinism, shapes, and that the planted structure is what
the oracle's selection finds (band head -> diagonal block, sink head -> block 0)."""
import numpy as np
import torch

from oracle import sparsed_oracle as orc
from paper_2509_24014_b200 import synthetic as syn


def test_configs_and_determinism():
    cfg = syn.CONFIGS["c1"]
    q1, k1, v1 = syn.make_qkv(cfg)
    q2, k2, v2 = syn.make_qkv(cfg)
    assert q1.dtype == torch.bfloat16 and q1.shape == (1, 2, 1024, 128) and k1.shape == v1.shape
    assert torch.equal(q1, q2) and torch.equal(k1, k2) and torch.equal(v1, v2)
    q3, _, _ = syn.make_qkv(cfg.with_(seed=1))
    assert not torch.equal(q1, q3)
    kinds = syn.head_kinds(syn.CONFIGS["c2"])
    assert len(kinds) == 32 and {k[0] for k in kinds} <= {"band", "sink", "stripes", "diffuse"}
    assert kinds == syn.head_kinds(syn.CONFIGS["c2"])


def test_gqa_and_step_noise_shapes():
    cfg = syn.CONFIGS["c3"].with_(seq_len=512)
    q, k, v = syn.make_qkv(cfg)
    assert q.shape == (1, 28, 512, 128) and k.shape == (1, 4, 512, 128)
    cfg4 = syn.CONFIGS["c4"].with_(seq_len=256, heads_q=2, heads_kv=2)
    base = syn.make_base(cfg4)
    a = syn.make_qkv(cfg4, step=3, base=base)
    b = syn.make_qkv(cfg4, step=3, base=base)
    c = syn.make_qkv(cfg4, step=4, base=base)
    assert torch.equal(a[0], b[0]) and not torch.equal(a[0], c[0])
    noise = (a[2].float() - base[2]).std().item()
    assert 0.04 < noise < 0.06


def test_planted_structure_is_selected_by_the_oracle():
    cfg = syn.CONFIGS["c1"]
    q, k, v = (t.to(torch.float64).numpy() for t in syn.make_qkv(cfg))
    ap = orc.pooled_scores(q, k, cfg.block_size)
    rp, ci = orc.select_blocks(ap, cfg.block_size, cfg.prefill_len, cfg.keep_ratio)
    nb = cfg.num_blocks
    assert np.all(np.diff(rp) == 5)
    for ib in range(nb):
        assert ib in ci[rp[ib]:rp[ib + 1]]            # band head keeps its diagonal block
        assert 0 in ci[rp[nb + ib]:rp[nb + ib + 1]]    # sink head keeps key block 0
