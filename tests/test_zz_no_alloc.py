"""The entry point that allocates nothing (ff_high_attention_noalloc): a host that cannot call
cudaMalloc -- all device memory already belongs to its pool, or an allocation's device-wide
synchronisation is not acceptable -- still gets the high-band operator.  Called through the C ABI
and compared with what the plan-based ff_forward produces for the same band tokens, and with the
fp64 oracle's window attention on the same tokens, twice in a row (the kernel's scratch is one array
shared by all calls and keeps the previous call's contents); the device's free memory, as the
driver reports it, must not move across a call.
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
    # the oracle's operator on the same band tokens, on sampled query rows of every head
    from oracle import freqformer_oracle as O
    n_high = qh.shape[1]
    ref_rows = []
    for h in range(qh.shape[0]):
        rows = I.sample_rows(cfg, 990 + h, n_high, 512)
        Qo, Ko, Vo = (x[h].float().cpu().numpy().astype(np.float64) for x in (qh, kh, vh))
        ref_rows.append((rows, O.high_operator(Qo, Ko, Vo, cfg.R, rows=rows)[0]))
    y = torch.full_like(qh, float("nan"))
    for call in range(2):
        y.fill_(float("nan"))
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]          # cudaMemGetInfo: sees any allocation, whoever makes it
        B.ff_high_attention_noalloc(qh, kh, vh, y, cfg.R, sync=True)
        if call == 1:                                       # (the first call may load the kernel's module)
            assert torch.cuda.mem_get_info()[0] == free_before
        got = y.float().cpu().numpy()
        Hn.assert_close(got, expect, "bf16", f"no-alloc call {call} against the plan path")
        for h, (rows, ref) in enumerate(ref_rows):
            Hn.assert_close(got[h][rows], ref, "bf16", f"no-alloc call {call} against the oracle, head {h}")
    plan.destroy()


@pytest.mark.parametrize("heads,n,radius", [(1, 1, 3), (2, 100, 7), (3, 129, 0), (2, 300, 10 ** 6), (1024, 5, 2)])
def test_no_alloc_small_shapes_match_the_oracle(heads, n, radius):
    """Bands shorter than one 128-row tile, a single token, a tile plus one row, a window of one
    key (R = 0: y = v), a window wider than the band (dense), and the largest head count."""
    import torch
    from oracle import freqformer_oracle as O
    from paper_2604_22808_b200 import binding as B
    g = np.random.Generator(np.random.Philox(key=[7, heads * 1000003 + n]))
    host = [I.round_to_bf16(g.standard_normal((heads, n, 128), dtype=np.float32)) for _ in range(3)]
    q, k, v = (torch.from_numpy(x).to("cuda", torch.bfloat16) for x in host)
    y = torch.full_like(q, float("nan"))
    B.ff_high_attention_noalloc(q, k, v, y, radius, sync=True)
    got = y.float().cpu().numpy()
    for h in sorted(set([0, heads // 2, heads - 1])):
        ref, _ = O.high_operator(*(x[h].astype(np.float64) for x in host), radius)
        Hn.assert_close(got[h], ref, "bf16", f"heads {heads} n {n} R {radius}, head {h}")


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
    # host tensors and tensors on different devices are refused by the binding before any launch
    with pytest.raises(B.FFError):
        B.ff_high_attention_noalloc(t.cpu(), t, t, t, 4)
