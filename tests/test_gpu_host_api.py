"""The host-buffer entry (chunks of heads on several streams) gives bitwise the result of the resident call."""
import pytest
import torch

import paper_2509_24014_b200 as sd
from paper_2509_24014_b200 import synthetic as syn
from paper_2509_24014_b200.host_api import HostSparseAttention
from tests.parity_util import gpu_select, gpu_sparse

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("Hq,Hkv,chunk", [(8, 8, 3), (12, 4, 1), (4, 4, 8)])
def test_host_sparse_attention_matches_resident(Hq, Hkv, chunk):
    cfg = syn.AttnConfig("h", 1, Hq, Hkv, 1024, 128, 128, 0.4, 512, seed=71)
    q, k, v = syn.make_qkv(cfg, DEV)
    pat, row_ptr, col_idx, _ = gpu_select(q, k, 128, 0.4, 512)
    o_ref = gpu_sparse(q, k, v, pat)
    hq, hk, hv = (t.cpu().pin_memory() for t in (q, k, v))
    ho = torch.zeros(q.shape, dtype=torch.bfloat16).pin_memory()
    plan = HostSparseAttention(hq, hk, row_ptr, col_idx, 128, DEV, kv_heads_per_chunk=chunk, n_streams=2)
    for _ in range(2):
        plan.run(hq, hk, hv, ho)
        torch.cuda.synchronize()
        assert torch.equal(ho, o_ref.cpu())
    assert all(st == (0, 0) for st in plan.device_status())
