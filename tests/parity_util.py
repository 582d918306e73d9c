"""Shared helpers for the GPU parity tests (no method arithmetic here)."""
import numpy as np
import torch

import paper_2509_24014_b200 as sd


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Exact widening of a bf16/fp32 tensor to a float64 numpy array on the host."""
    return t.detach().to("cpu").to(torch.float64).numpy()


def gpu_full(q, k, v, want_lse=True):
    o = torch.empty_like(q)
    lse = torch.empty(q.shape[:3], dtype=torch.float32, device=q.device) if want_lse else None
    ws = sd.new_workspace(sd.sparsed_workspace_bytes(sd.OP_ATTN_FULL), q.device)
    sd.sparsed_attn_full(q, k, v, o, lse, ws)
    torch.cuda.synchronize()
    assert sd.sparsed_last_device_status(ws) == (0, 0)
    return o, lse


def gpu_select(q, k, block_size, keep_ratio, prefill_len, lse=None, want_scores=True):
    B, Hq, L, _ = q.shape
    nb = L // block_size
    params = sd.make_params(block_size, keep_ratio, prefill_len)
    kp, kg = sd.sparsed_kept_per_row(params, L)
    pat, row_ptr, col_idx = sd.new_pattern(B, Hq, nb, kp + kg, q.device)
    scores = torch.full((B, Hq, nb, nb), float("nan"), dtype=torch.float32, device=q.device) if want_scores else None
    ws = sd.new_workspace(sd.sparsed_workspace_bytes(sd.OP_SELECT_PATTERN, sd.make_shape(q, k), params), q.device)
    sd.sparsed_select_pattern(q, k, params, pat, ws, lse=lse, scores_out=scores)
    torch.cuda.synchronize()
    assert sd.sparsed_last_device_status(ws) == (0, 0)
    return pat, row_ptr, col_idx, scores


def gpu_sparse(q, k, v, pat):
    o = torch.empty_like(q)
    ws = sd.new_workspace(sd.sparsed_workspace_bytes(sd.OP_ATTN_SPARSE), q.device)
    sd.sparsed_attn_sparse(q, k, v, o, pat, ws)
    torch.cuda.synchronize()
    assert sd.sparsed_last_device_status(ws) == (0, 0)
    return o


def check_outputs(o_gpu: torch.Tensor, o_ref: np.ndarray, what=""):
    """The acceptance bar for bf16 attention outputs: max-abs 2e-2 and mean-abs 2e-3 (the
    stated contract), plus a relative Frobenius bound so that an all-zero output of a
    near-uniform attention (|O| ~ 1e-2) cannot pass."""
    d = np.abs(to_f64(o_gpu) - o_ref)
    assert np.isfinite(d).all(), what
    assert d.max() <= 2e-2, f"{what}: max abs {d.max()}"
    assert d.mean() <= 2e-3, f"{what}: mean abs {d.mean()}"
    rel = np.linalg.norm(d) / max(np.linalg.norm(o_ref), 1e-30)
    assert rel <= 1e-2, f"{what}: relative Frobenius error {rel}"
    return d.max(), d.mean(), rel
