"""The entry point that allocates nothing (ff_high_attention_noalloc): a host that cannot call
cudaMalloc -- all device memory already belongs to its pool, or an allocation's device-wide
synchronisation is not acceptable -- still gets the high-band operator.  Called through the C ABI
and compared with what the plan-based ff_forward produces for the same band tokens, twice in a row
(the kernel's scratch is one array shared by all calls and keeps the previous call's contents).
Collected last on purpose, so that a run that stops at the first failure has run everything else."""
import numpy as np
import pytest

from paper_2604_22808_b200 import configs as C
from paper_2604_22808_b200 import inputs as I

import harness as Hn

pytestmark = pytest.mark.gpu


def test_no_alloc_entry_point_matches_plan_path_twice():
    import torch
    from paper_2604_22808_b200 import binding as B
    cfg = C.R64K
    Q, K, V = Hn.host_inputs(cfg)
    plan = B.Plan(cfg, None)
    q, k, v = (Hn.to_device(x, cfg) for x in (Q, K, V))
    out = torch.empty_like(q)
    alloc = torch.full((cfg.batch * cfg.heads,), B.FF_BAND_HIGH, dtype=torch.uint8, device="cuda")
    plan.forward(q, k, v, out, alloc=alloc)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    spec = plan.tap(B.TAP_SPEC_HIGH)                 # [3][BH][N_high][128]: Q~, K~, V~ of the high band
    expect = plan.tap(B.TAP_Y_HIGH).float().cpu().numpy()
    qh, kh, vh = (spec[t].clone() for t in range(3))
    before = torch.cuda.memory_allocated()
    for call in range(2):
        y = torch.full_like(qh, float("nan"))
        reserved = torch.cuda.memory_reserved()
        B.ff_high_attention_noalloc(qh, kh, vh, y, cfg.R, sync=True)
        assert torch.cuda.memory_reserved() == reserved
        got = y.float().cpu().numpy()
        Hn.assert_close(got, expect, "bf16", f"no-alloc call {call}")
    assert torch.cuda.memory_allocated() >= before
    plan.destroy()


def test_no_alloc_entry_point_rejects_bad_arguments():
    import torch
    from paper_2604_22808_b200 import binding as B
    lib = B.library()
    t = torch.zeros((2, 256, 128), dtype=torch.bfloat16, device="cuda")
    p = t.data_ptr()
    assert lib.ff_high_attention_noalloc(None, p, p, p, 2, 256, 4, 1, None) == 1
    assert lib.ff_high_attention_noalloc(p + 2, p, p, p, 2, 256, 4, 1, None) == 1
    assert lib.ff_high_attention_noalloc(p, p, p, p, 0, 256, 4, 1, None) == 1
    assert lib.ff_high_attention_noalloc(p, p, p, p, 2000, 256, 4, 1, None) == 2
    assert lib.ff_high_attention_noalloc(p, p, p, p, 2, 2 ** 31, 4, 1, None) == 2
    assert b"1024 heads" in lib.ff_last_error(None)
