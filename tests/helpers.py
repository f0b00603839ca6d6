"""Shared helpers of the GPU parity tests: run the CUDA library and the CPU oracle on
the same seeded inputs and compare the routing tables element by element."""
import numpy as np
import torch

import paper_2402_12399_b200 as rr
from oracle import rr_oracle as orc

INT_TABLES = ["topk_expert", "route_slot", "slot_token", "slot_rank", "drop_count", "ir_expert", "ir_pos",
              "ir_offset", "ir_token", "expert_count", "n_routed", "row_offset", "row_token", "token_rows"]


def gpu_route(logits_np, k, C, G, mode):
    a = torch.from_numpy(np.ascontiguousarray(logits_np)).cuda()
    t = rr.route(a, k, C, G, mode)
    rr.check(t._workspace)
    return t


def assert_tables_equal(t_gpu, t_cpu, where=""):
    """Integer tables bit-exact; combine weights within 1e-5 relative."""
    for name in INT_TABLES:
        g = getattr(t_gpu, name).cpu().numpy()
        c = getattr(t_cpu, name)
        assert g.shape == c.shape, (where, name, g.shape, c.shape)
        if not np.array_equal(g, c):
            bad = np.argwhere(g != c)
            raise AssertionError(f"{where}: table {name} differs at {len(bad)} places, first {bad[0]}: "
                                 f"gpu {g[tuple(bad[0])]} cpu {c[tuple(bad[0])]}")
    w = t_gpu.combine_w.cpu().numpy().astype(np.float64)
    np.testing.assert_allclose(w, t_cpu.combine_w, rtol=1e-5, atol=1e-7, err_msg=f"{where}: combine_w")
    rw = t_gpu.row_weight.cpu().numpy().astype(np.float64)
    np.testing.assert_allclose(rw, t_cpu.row_weight, rtol=1e-5, atol=1e-7, err_msg=f"{where}: row_weight")


def route_both(logits_np, k, C, G, mode, where=""):
    tg = gpu_route(logits_np, k, C, G, mode)
    tc = orc.route(logits_np, k, C, G, mode)
    assert_tables_equal(tg, tc, where)
    return tg, tc


def to_torch(x_np, dtype):
    """Host array from synth (float32, or uint16 bf16 bit patterns) -> CUDA tensor."""
    if dtype == "bf16":
        return torch.from_numpy(x_np.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(x_np).cuda()
