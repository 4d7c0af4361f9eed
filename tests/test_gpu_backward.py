"""GPU parity of the backward pass against the oracle's gradients (fp64 chain rule of the forward
definition, itself pinned by finite differences).  bf16 operands, fp32 accumulation, several bf16
intermediates (a, b, H, dY, dA, dB): tolerance |gpu - ref| <= 2e-2 * max|ref| + 2e-2 * |ref|."""
import numpy as np
import pytest

from oracle import feplb_oracle as O
from paper_2604_19654_b200 import build as B
from paper_2604_19654_b200 import feplb as F
from paper_2604_19654_b200 import workloads as W

from gpu_utils import DeviceCase

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    B.build()


def _close(got, ref, what, tol=2e-2):
    bound = tol * np.abs(ref).max() + tol * np.abs(ref)
    err = np.abs(got - ref)
    assert np.all(err <= bound), (f"{what}: {int((err > bound).sum())} of {err.size} out of tolerance, max err "
                                  f"{err.max():.3e}, max|ref| {np.abs(ref).max():.3e}, at {np.argwhere(err > bound)[0].tolist()}")
    return float(err.max() / (np.abs(ref).max() + 1e-300))


def test_transpose_weights_bit_exact():
    import torch
    w = W.get_workload("cfg1").with_(E=4, d=256, f=192)
    case = DeviceCase(w)
    w1t, w3t = torch.zeros(w.E, w.d, w.f, dtype=torch.bfloat16, device="cuda"), torch.zeros(w.E, w.d, w.f, dtype=torch.bfloat16, device="cuda")
    w2t = torch.zeros(w.E, w.f, w.d, dtype=torch.bfloat16, device="cuda")
    case.ctx.transpose_weights(case.d_w1, case.d_w3, case.d_w2, w1t, w3t, w2t)
    torch.cuda.synchronize()
    assert np.array_equal(F.bf16_bits(w1t), case.w1.transpose(0, 2, 1))
    assert np.array_equal(F.bf16_bits(w3t), case.w3.transpose(0, 2, 1))
    assert np.array_equal(F.bf16_bits(w2t), case.w2.transpose(0, 2, 1))
    case.close()


def test_pack_weights_from_input_major_layout():
    """feplb_pack_weights: [E,d,f] / [E,f,d] (x W as the operator is usually written) -> the library's layout."""
    import torch
    w = W.get_workload("cfg1").with_(E=4, d=384, f=192)
    case = DeviceCase(w)
    w1_in = F.bf16_tensor(np.ascontiguousarray(case.w1.transpose(0, 2, 1)))     # [E, d, f]
    w3_in = F.bf16_tensor(np.ascontiguousarray(case.w3.transpose(0, 2, 1)))
    w2_in = F.bf16_tensor(np.ascontiguousarray(case.w2.transpose(0, 2, 1)))     # [E, f, d]
    w1, w3, w2 = torch.zeros_like(case.d_w1), torch.zeros_like(case.d_w3), torch.zeros_like(case.d_w2)
    case.ctx.pack_weights(w1_in, w3_in, w2_in, w1, w3, w2)
    torch.cuda.synchronize()
    assert np.array_equal(F.bf16_bits(w1), case.w1) and np.array_equal(F.bf16_bits(w3), case.w3)
    assert np.array_equal(F.bf16_bits(w2), case.w2)
    case.close()


def _run_backward(w, mb=0, scale=1.0, pair=-1, **cfg_kw):
    import torch
    case = DeviceCase(w, mb=mb, row_align=128, **cfg_kw)
    bwd = F.BackwardBuffers(case.cfg)
    ctx = case.ctx
    ctx.set_gemm_form(F.FORM_AUTO, pair)
    ctx.set_preact_buffer(bwd.ab)
    ctx.moe_forward(case.d_x, case.d_ids, case.d_gates, case.d_w1, case.d_w3, case.d_w2, case.buf)
    w1t = torch.zeros(w.E, w.d, w.f, dtype=torch.bfloat16, device="cuda")
    w3t = torch.zeros_like(w1t)
    w2t = torch.zeros(w.E, w.f, w.d, dtype=torch.bfloat16, device="cuda")
    ctx.transpose_weights(case.d_w1, case.d_w3, case.d_w2, w1t, w3t, w2t)
    rng = np.random.default_rng(77 + mb)
    d_out = W.f32_to_bf16_bits((rng.standard_normal((w.T, w.d)) * scale).astype(np.float32))
    dw1 = torch.full((w.E, w.f, w.d), 5.0, dtype=torch.float32, device="cuda")     # must be overwritten
    dw3 = torch.full((w.E, w.f, w.d), 5.0, dtype=torch.float32, device="cuda")
    dw2 = torch.full((w.E, w.d, w.f), 5.0, dtype=torch.float32, device="cuda")
    ctx.moe_backward(F.bf16_tensor(d_out), case.d_gates, w1t, w3t, w2t, case.buf, bwd, dw1, dw3, dw2)
    ctx.check_status()
    ref = O.moe_layer_backward(case.x, case.ids, case.gates, case.w1, case.w3, case.w2, W.bf16_bits_to_f64(d_out), w.E)
    return case, bwd, (dw1, dw3, dw2), ref, (w1t, w3t, w2t), d_out


@pytest.mark.parametrize("pair", [0, 3])
@pytest.mark.parametrize("name,T", [("cfg1", 256), ("cfg2", 384), ("cfg4", 512)])
def test_backward_parity(name, T, pair):
    """``pair``: both forms of the backward GEMMs (single CTA per 128-row tile; clusters of two CTAs on
    256-row tiles), forced with feplb_set_gemm_form."""
    import torch
    w = W.get_workload(name).with_(T=T)
    if name != "cfg1":
        w = w.with_(E=16, R=4)                       # fewer experts: the fp64 reference stays cheap
    case, bwd, (dw1, dw3, dw2), ref, wt, d_out = _run_backward(w, pair=pair)
    rdx, rdg, rdw1, rdw3, rdw2 = ref
    _close(W.bf16_bits_to_f64(F.bf16_bits(bwd.d_x))[: w.T], rdx, "dx")
    _close(bwd.d_gates.cpu().numpy().astype(np.float64)[: w.T], rdg, "dgates")
    _close(dw2.cpu().numpy().astype(np.float64), rdw2, "dw2")
    _close(dw1.cpu().numpy().astype(np.float64), rdw1, "dw1")
    _close(dw3.cpu().numpy().astype(np.float64), rdw3, "dw3")
    # experts that received no rows: exact zeros (the 5.0 fill is gone)
    counts = np.bincount(case.ids.ravel(), minlength=w.E)
    for e in np.flatnonzero(counts == 0):
        assert not dw1[e].any() and not dw2[e].any()
    # accumulate: a second backward with accumulate doubles the weight gradients
    snap = dw2.clone()
    case.ctx.moe_backward(F.bf16_tensor(d_out), case.d_gates, *wt, case.buf, bwd, dw1, dw3, dw2, accumulate=True)
    case.ctx.check_status()
    assert torch.allclose(dw2, 2 * snap, rtol=1e-6, atol=1e-12)
    # without weight gradients only the activation path runs (and needs no transposed scratch)
    case.ctx.moe_backward(F.bf16_tensor(d_out), case.d_gates, *wt, case.buf, bwd)
    case.ctx.check_status()
    _close(W.bf16_bits_to_f64(F.bf16_bits(bwd.d_x))[: w.T], rdx, "dx (no wgrad)")
    case.close()


@pytest.mark.parametrize("seed", range(8))
def test_backward_random_shapes(seed):
    """Seeded random small layers (odd token counts, 1-4 ranks, ragged tiles, experts without rows),
    both GEMM forms."""
    rng = np.random.default_rng(9100 + seed)
    R = int(rng.choice([1, 2, 4]))
    L = int(rng.choice([1, 2, 3, 6]))
    E = R * L
    w = W.get_workload("cfg2").with_(
        name=f"randb{seed}", T=int(rng.integers(1, 500)), E=E, R=R, K=int(rng.integers(1, min(E, 6) + 1)),
        d=int(rng.choice([128, 256, 384])), f=int(rng.choice([64, 192, 256])), dyn=int(rng.integers(0, L + 1)),
        max_num_dyn=2, tau=8, routing="dirichlet", alpha=float(rng.choice([0.1, 0.5])))
    case, bwd, (dw1, dw3, dw2), ref, wt, d_out = _run_backward(w, mb=seed, pair=int(rng.choice([0, 3])))
    rdx, rdg, rdw1, rdw3, rdw2 = ref
    _close(W.bf16_bits_to_f64(F.bf16_bits(bwd.d_x))[: w.T], rdx, "dx")
    _close(bwd.d_gates.cpu().numpy().astype(np.float64)[: w.T], rdg, "dgates")
    _close(dw2.cpu().numpy().astype(np.float64), rdw2, "dw2")
    _close(dw1.cpu().numpy().astype(np.float64), rdw1, "dw1")
    _close(dw3.cpu().numpy().astype(np.float64), rdw3, "dw3")
    case.close()


def test_backward_at_the_maximum_expert_count():
    """E = 1024: expert and group tables at the library's limit, most experts with few rows or none."""
    w = W.get_workload("cfg2").with_(name="maxEb", T=700, E=1024, R=16, K=4, d=128, f=64, dyn=8, max_num_dyn=4, tau=1, alpha=0.3)
    case, bwd, (dw1, dw3, dw2), ref, wt, d_out = _run_backward(w)
    rdx, rdg, rdw1, rdw3, rdw2 = ref
    _close(W.bf16_bits_to_f64(F.bf16_bits(bwd.d_x))[: w.T], rdx, "dx")
    _close(bwd.d_gates.cpu().numpy().astype(np.float64)[: w.T], rdg, "dgates")
    _close(dw2.cpu().numpy().astype(np.float64), rdw2, "dw2")
    _close(dw1.cpu().numpy().astype(np.float64), rdw1, "dw1")
    _close(dw3.cpu().numpy().astype(np.float64), rdw3, "dw3")
    case.close()


@pytest.mark.parametrize("pair", [0, 3])
def test_backward_of_an_empty_batch(pair):
    """T = 0 with padded segments: every expert has zero rows.  The weight gradients are zeros when
    overwriting and untouched when accumulating; nothing traps."""
    import torch
    w = W.get_workload("cfg1").with_(T=0)
    cfg = F.config_from_workload(w, row_align=128)
    ctx, buf, bwd = F.Context(cfg), F.Buffers(cfg), F.BackwardBuffers(cfg)
    ctx.set_gemm_form(F.FORM_AUTO, pair)
    ctx.set_preact_buffer(bwd.ab)
    z = torch.zeros(1, w.d, dtype=torch.bfloat16, device="cuda")
    zi = torch.zeros(1, w.K, dtype=torch.int32, device="cuda")
    zg = torch.zeros(1, w.K, device="cuda")
    w1 = torch.ones(w.E, w.f, w.d, dtype=torch.bfloat16, device="cuda")
    w2 = torch.ones(w.E, w.d, w.f, dtype=torch.bfloat16, device="cuda")
    ctx.moe_forward(z, zi, zg, w1, w1, w2, buf)
    dw1 = torch.full((w.E, w.f, w.d), 3.0, device="cuda")
    dw3 = torch.full((w.E, w.f, w.d), 3.0, device="cuda")
    dw2 = torch.full((w.E, w.d, w.f), 3.0, device="cuda")
    w1t = torch.ones(w.E, w.d, w.f, dtype=torch.bfloat16, device="cuda")
    w2t = torch.ones(w.E, w.f, w.d, dtype=torch.bfloat16, device="cuda")
    ctx.moe_backward(z, zg, w1t, w1t, w2t, buf, bwd, dw1, dw3, dw2, accumulate=True)
    ctx.check_status()
    assert float(dw1.min()) == 3.0 and float(dw2.max()) == 3.0
    ctx.moe_backward(z, zg, w1t, w1t, w2t, buf, bwd, dw1, dw3, dw2)
    ctx.check_status()
    assert not dw1.any() and not dw3.any() and not dw2.any()
    ctx.close()


def test_combine_bwd_bit_exact_rows_and_gate_gradients():
    import torch
    w = W.get_workload("cfg2").with_(T=300, E=16, R=4)
    case = DeviceCase(w, row_align=128)
    bwd = F.BackwardBuffers(case.cfg)
    case.ctx.moe_forward(case.d_x, case.d_ids, case.d_gates, case.d_w1, case.d_w3, case.d_w2, case.buf)
    rng = np.random.default_rng(5)
    d_out = W.f32_to_bf16_bits(rng.standard_normal((w.T, w.d)).astype(np.float32))
    case.ctx.combine_bwd(F.bf16_tensor(d_out), case.buf.y_perm, case.buf.slot_to_row, case.d_gates, bwd.d_y_perm, bwd.d_gates)
    case.ctx.check_status()
    s2r = case.buf.slot_to_row.cpu().numpy()
    dy = F.bf16_bits(bwd.d_y_perm)
    y = W.bf16_bits_to_f64(F.bf16_bits(case.buf.y_perm))
    do32 = W.bf16_bits_to_f32(d_out)
    for t in (0, 17, w.T - 1):
        for k in range(w.K):
            exp = W.f32_to_bf16_bits((case.gates[t, k] * do32[t]).astype(np.float32))     # one fp32 product, one rounding
            assert np.array_equal(dy[s2r[t, k]], exp)
    ref_dg = np.einsum("td,tkd->tk", W.bf16_bits_to_f64(d_out), y[s2r])
    got = bwd.d_gates.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - ref_dg) <= 1e-5 * np.abs(ref_dg).max() + 1e-4 * np.abs(ref_dg))
    case.close()


def test_weight_gradients_need_padded_segments():
    w = W.get_workload("cfg1")
    case = DeviceCase(w)                               # row_align = 1
    bwd = F.BackwardBuffers(case.cfg)
    import torch
    z = torch.zeros(w.E, w.d, w.f, dtype=torch.bfloat16, device="cuda")
    z2 = torch.zeros(w.E, w.f, w.d, dtype=torch.bfloat16, device="cuda")
    g = torch.zeros(w.E, w.f, w.d, dtype=torch.float32, device="cuda")
    g2 = torch.zeros(w.E, w.d, w.f, dtype=torch.float32, device="cuda")
    case.ctx.moe_forward(case.d_x, case.d_ids, case.d_gates, case.d_w1, case.d_w3, case.d_w2, case.buf)
    with pytest.raises(F.FeplbError) as ei:
        case.ctx.moe_backward(case.d_x, case.d_gates, z, z, z2, case.buf, bwd, g, g, g2)
    assert ei.value.code == F.E_INVALID
    case.close()
