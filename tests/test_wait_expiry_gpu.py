"""A bounded device-side wait that really runs out: the kernel must set the status bit, unwind (drain its
copies, free its TMEM) and return, and the next call on the same plan must be correct again.

No invalid access is involved: through the test hook psattn_plan_debug_waits the first TMA barrier of the
kernel expects 16 bytes more than are ever sent, so it never completes, and the wait limit is cut from 1 s
to 20 microseconds.  Covered: the long-row-list / dense attention kernel and the fused forward kernel."""
import time

import numpy as np
import pytest
import torch

import parity
from oracle import psattn_oracle as orc
from paper_2106_09236_b200 import binding as ps
from paper_2106_09236_b200 import workloads as wl

pytestmark = pytest.mark.gpu

WAIT_EXPIRED = 4


def _inputs(B, H, T, seed):
    c = 5.0
    wk = wl.Workload("adhoc", 0, B, H, T, 64, "bf16", c, 0.1, 3.0)
    inp = wl.make_inputs(wk, orc.count(c, T), seed=seed)
    dev = {k: torch.from_numpy(inp[k]).to("cuda", torch.bfloat16) for k in ("Q", "K", "V")}
    dev["lengths"] = torch.from_numpy(inp["lengths"]).cuda()
    dev["sample_idx"] = torch.from_numpy(inp["sample_idx"]).cuda()
    return inp, dev, c


def test_dense_attention_kernel_gives_up_and_recovers():
    B, H, T = 1, 2, 384
    inp, dev, c = _inputs(B, H, T, 71)
    plan = ps.Plan(B, H, T, dtype=torch.bfloat16, c=c, idx_cols=inp["sample_idx"].shape[-1])
    O = torch.zeros((B, H, T, 64), dtype=torch.bfloat16, device="cuda")
    plan.psattn_plan_debug_waits(20_000, 16)
    t0 = time.perf_counter()
    plan.psattn_dense_forward(dev["Q"], dev["K"], dev["V"], dev["lengths"], O)
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 5.0, "the kernel must return once its waits have run out"
    assert plan.psattn_read_status() & WAIT_EXPIRED
    # back to normal: same plan, same buffers
    plan.psattn_plan_debug_waits(0, 0)
    plan.psattn_dense_forward(dev["Q"], dev["K"], dev["V"], dev["lengths"], O)
    torch.cuda.synchronize()
    assert plan.psattn_read_status() == 0
    ref = orc.dense(inp["Q"], inp["K"], inp["V"], inp["lengths"], nthreads=4)
    assert np.abs(O.float().cpu().numpy() - ref).max() <= parity.O_ATOL["bf16"]
    plan.close()


def test_fused_forward_kernel_gives_up_and_recovers():
    B, H, T = 2, 2, 200
    inp, dev, c = _inputs(B, H, T, 72)
    plan = ps.Plan(B, H, T, dtype=torch.bfloat16, c=c, idx_cols=inp["sample_idx"].shape[-1], path=ps.PSATTN_PATH_FUSED)
    plan.psattn_plan_debug_waits(20_000, 16)
    O = torch.full((B, H, T, 64), 3.0, dtype=torch.bfloat16, device="cuda")
    M = torch.full((B, H, T), 3.0, dtype=torch.float32, device="cuda")
    t0 = time.perf_counter()
    _, sel = plan.psattn_forward(dev["Q"], dev["K"], dev["V"], dev["lengths"], dev["sample_idx"], O, None, M)
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 5.0
    assert plan.psattn_read_status() & WAIT_EXPIRED
    # what the kernel leaves behind when the keys never arrive: a zero measure and zero rows
    assert float(M.abs().max()) == 0.0
    assert float(O.float().abs().max()) == 0.0
    plan.psattn_plan_debug_waits(0, 0)
    O2, sel2 = plan.psattn_forward(dev["Q"], dev["K"], dev["V"], dev["lengths"], dev["sample_idx"], None, None, M)
    torch.cuda.synchronize()
    assert plan.psattn_read_status() == 0
    parity.check_forward(O2.float().cpu().numpy(), sel2.cpu().numpy(), M.cpu().numpy(), inp, inp["lengths"], "bf16", c)
    plan.close()
