"""feplb_dispatch_noalloc -- the dispatch for callers that cannot allocate device memory (a
server whose pool owns all of it, a loop that cannot take cudaMalloc's synchronisation) -- must
give exactly what feplb_dispatch gives.  Called through the C ABI, twice in a row on different
inputs, because its built-in scratch is shared between calls and keeps the previous contents.
Collected last (file name) so that a run stopping at the first failure has run everything else."""
import numpy as np
import pytest

from paper_2604_19654_b200 import build as B
from paper_2604_19654_b200 import feplb as F
from paper_2604_19654_b200 import workloads as W


@pytest.mark.gpu
def test_noalloc_dispatch_matches_dispatch_twice_in_a_row():
    import torch
    B.build()
    w = W.get_workload("cfg2").with_(T=1500)         # 9000 slots: 9 CTAs and a ragged tail
    for A in (1, 128):
        cfg = F.config_from_workload(w, row_align=A)
        ctx, ref = F.Context(cfg), F.Buffers(cfg)
        got = F.Buffers(cfg)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        for call, mb in enumerate((0, 5)):           # second call: other routing, same scratch
            x, ids, _ = W.gen_microbatch(w, mb)
            d_x, d_ids = F.bf16_tensor(x), torch.from_numpy(ids).cuda()
            ctx.route_hist(d_ids, ref.counts, ref.rank_load)
            ref.x_perm.fill_(1.0)
            got.x_perm.fill_(1.0)
            ctx.dispatch(d_x, d_ids, ref.counts, ref.x_perm, ref.slot_to_row, ref.row_to_token)
            ctx.check_status()
            F.dispatch_noalloc(cfg, d_x, d_ids, ref.counts, got.x_perm, got.slot_to_row, got.row_to_token, status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            assert torch.equal(got.slot_to_row, ref.slot_to_row), (A, call)
            assert torch.equal(got.row_to_token, ref.row_to_token), (A, call)
            assert torch.equal(got.x_perm.view(torch.int16), ref.x_perm.view(torch.int16)), (A, call)
        ctx.close()


def test_noalloc_dispatch_rejects_sizes_beyond_its_scratch():
    B.build()
    cfg = F.make_config(T=1 << 20, K=8, E=128, R=8, d=128, f=64)        # 8192 CTAs x 128 experts > limit
    with pytest.raises(F.FeplbError) as ei:
        F.dispatch_noalloc(cfg, 16, 16, 16, 16, 16, 16, stream=0)
    assert ei.value.code == F.E_NOMEM


def test_noalloc_limit_is_declared():
    src = open(F.LIB_PATH.replace("paper_2604_19654_b200/libfeplb.so", "include/feplb.h")).read()
    assert "FEPLB_NOALLOC_MAX_HIST_INTS 524288" in src
