"""Helpers shared by the GPU parity tests: move a seeded workload to the device, run the C-ABI
stages through the Python binding, and bring results back as numpy arrays."""
import numpy as np
import torch

import oracle as O


def bf16_tensor_from_bits(bits: np.ndarray, device="cuda") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device).view(torch.bfloat16)


def bits_from_bf16_tensor(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def u32(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint32)


def make_step(w, with_x=True, alias_expert_out=True):
    """Layout + RouteStep buffers with the workload's inputs uploaded."""
    import paper_2609_36959_b200 as cb
    from paper_2609_36959_b200.router import RouteStep

    layout = cb.Layout(w.N, w.Q, w.S, w.E, w.slot_expert.tolist(), w.primary_slot.tolist())
    step = RouteStep(layout, w.T, w.K, w.H, alias_expert_out=alias_expert_out)
    step.topk_ids.copy_(torch.from_numpy(w.topk_ids))
    step.gate_w.copy_(torch.from_numpy(w.gate_w))
    step.src_rank.copy_(torch.from_numpy(w.src_rank))
    if with_x and w.T > 0:
        step.x.copy_(bf16_tensor_from_bits(w.hidden_rows(), "cpu"))
    return layout, step


def oracle_assign(w, seed, naive=False):
    return O.assign(w.N, w.Q, w.S, w.E, w.slot_expert, w.primary_slot, w.topk_ids, w.src_rank, seed, naive=naive)


def assert_combine_close(y_gpu_bits: np.ndarray, y_oracle: np.ndarray):
    """|gpu - oracle| <= 1e-2 + 1e-2 |oracle| element-wise (oracle: fp32 accumulation, unrounded)."""
    from workloads import f32_from_bf16_bits

    y = f32_from_bf16_bits(y_gpu_bits).astype(np.float64)
    ref = y_oracle.astype(np.float64)
    err = np.abs(y - ref)
    tol = 1e-2 + 1e-2 * np.abs(ref)
    worst = float((err - tol).max()) if err.size else -1.0
    assert worst <= 0.0, f"combine outside tolerance by {worst}; max abs err {err.max()}"
