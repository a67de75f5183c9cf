"""The fused output stage of the token mixer, y = SRMSNorm(o) (.) u (Eq. 3 with Eq. 8), through the C ABI against the
fp64 oracle: la_fwd_gated (epilogue inside the full-width walk kernel at d = 128, row kernel behind the walk
otherwise) and la_gate_bwd, alone and chained into la_bwd."""
import numpy as np
import pytest
import torch

from la_check import TOL_BF16, assert_close
from oracle import la_oracle as orc
from paper_2307_14995_b200 import binding as la, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def draw_gate(shape, seed, dtype=torch.bfloat16):
    gen = torch.Generator("cpu")
    gen.manual_seed(seed)
    # the gate of the token mixer is a linear projection passed through no activation (Eq. 3): normal draws
    return inputs.draw(shape, gen, "normal", dtype)


def run_gated(q, k, v, u, lam, out_dtype=torch.float32, want_o=True, want_rstd=True, seg_len=0, kv_in=None,
              path=la.LA_PATH_AUTO, misalign=False):
    B, H, N, d = q.shape
    qg, kg, vg, ug = (x.to(DEV) for x in (q, k, v, u))
    shape = la.make_shape(B, H, N, d, d, q.dtype, out_dtype, seg_len, path)
    n = B * H * N * d
    pad = 4 if misalign else 0   # elements: 16 bytes for fp32, 8 for bf16 -> use 8 elements for bf16
    if misalign and out_dtype == torch.bfloat16:
        pad = 8
    ybuf = torch.full((n + pad,), float("nan"), dtype=out_dtype, device=DEV)
    y = ybuf[pad:pad + n].view(B, H, N, d)
    o = torch.full((B, H, N, d), float("nan"), dtype=out_dtype, device=DEV) if want_o else None
    rstd = torch.full((B, H, N), float("nan"), dtype=torch.float32, device=DEV) if want_rstd else None
    kv_out = torch.empty((B, H, d, d), dtype=torch.float32, device=DEV)
    ws = la.alloc_workspace(la.LA_OP_FWD, shape, DEV)
    la.la_fwd_gated(shape, qg, kg, vg, ug, lam, y, o, rstd, None if kv_in is None else kv_in.to(DEV), kv_out, ws)
    torch.cuda.synchronize()
    la.device_status()
    return y, o, rstd, kv_out


def check_gated(q, k, v, u, lam, got, tol, kv_in=None):
    y, o, rstd, kv_out = got
    ref_o, ref_kv = orc.fwd_rec(q, k, v, lam.double().numpy(), kv_in=None if kv_in is None else kv_in.double().numpy(),
                                want_state=True)
    ref_y, ref_rstd = orc.norm_gate_fwd(ref_o, u, want_rstd=True)
    assert_close(y, ref_y, tol, "y")
    assert_close(kv_out, ref_kv, tol, "kv_out")
    if o is not None:
        assert_close(o, ref_o, tol, "o")
    if rstd is not None:
        r = rstd.double().cpu().numpy()
        assert np.all(np.isfinite(r)) and np.max(np.abs(r - ref_rstd) / ref_rstd) <= 1e-3


@pytest.mark.parametrize("name", ["385m", "1b"])
def test_gated_forward_workloads(name):
    w = inputs.make_workload(name)
    u = draw_gate(tuple(w["v"].shape), seed=77)
    got = run_gated(w["q"], w["k"], w["v"], u, w["lam"])
    check_gated(w["q"], w["k"], w["v"], u, w["lam"], got, TOL_BF16)


def test_gated_forward_7b_long_full_size():
    """The 7B-like launch configuration: epilogue fused into the full-width walk, o not written at all; every head's
    y against the oracle (recurrence, then norm and gate), eight heads at a time."""
    w = inputs.device_randn_like_workload("7b_long", DEV, seed=2)
    q, k, v, lam = w["q"], w["k"], w["v"], w["lam"]
    B, H, N, d = q.shape
    gen = torch.Generator(DEV)
    gen.manual_seed(5)
    u = torch.randn((B, H, N, d), generator=gen, device=DEV).to(torch.bfloat16)
    shape = la.make_shape(B, H, N, d, d, torch.bfloat16, torch.float32)
    y = torch.empty((B, H, N, d), dtype=torch.float32, device=DEV)
    ws = la.alloc_workspace(la.LA_OP_FWD, shape, DEV)
    l0 = la.launch_count()
    la.la_fwd_gated(shape, q, k, v, u, lam, y, None, None, None, None, ws)
    torch.cuda.synchronize()
    la.device_status()
    assert la.launch_count() - l0 == 3          # pre-pass, scan, walk: no separate norm pass
    for h0 in range(0, H, 8):
        heads = list(range(h0, h0 + 8))
        qs, ks, vs, us = (x[:, heads].cpu() for x in (q, k, v, u))
        ref_o = orc.fwd_rec(qs, ks, vs, lam[heads].double().numpy())
        ref_y = orc.norm_gate_fwd(ref_o, us)
        assert_close(y[:, heads], ref_y, TOL_BF16, "y heads %d..%d" % (h0, h0 + 7))
        del ref_o, ref_y


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("N", [1, 127, 300, 1000])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_gated_forward_ragged_states_and_options(N, d, out_dtype):
    B, H = 2, 3
    q, k, v, _ = inputs.make_qkvdo(B, H, N, d, d, seed=100 + N, with_do=False)
    u = draw_gate((B, H, N, d), seed=N)
    lam = torch.tensor([1.0, 0.97, 0.3])
    kv_in = inputs.make_state(B, H, d, d, seed=8)
    ref_o, ref_kv = orc.fwd_rec(q, k, v, lam.double().numpy(), kv_in=kv_in.double().numpy(), want_state=True)
    ref_y = orc.norm_gate_fwd(ref_o, u)
    for seg_len, want_o, misalign in ((0, True, False), (128, False, False), (256, True, True)):
        y, o, rstd, kv_out = run_gated(q, k, v, u, lam, out_dtype=out_dtype, want_o=want_o, want_rstd=want_o,
                                       seg_len=seg_len, kv_in=kv_in, misalign=misalign)
        if out_dtype == torch.float32:
            assert_close(y, ref_y, TOL_BF16, "y")
            if o is not None:
                assert_close(o, ref_o, TOL_BF16, "o")
        else:
            # bf16 outputs add their own rounding (see the bf16-output test of the plain forward pass): one rounding
            # where the epilogue is fused (d = 128, aligned), two where the attention output passes through a bf16
            # tensor on its way to the row kernel
            fused = d == 128 and not misalign
            for g, r in ((y, ref_y),) + (((o, ref_o),) if o is not None else ()):
                gn = g.double().cpu().numpy().reshape(B * H, -1)
                rn = r.reshape(B * H, -1)
                rms = np.sqrt(np.mean(rn * rn, axis=1, keepdims=True))
                assert np.all(np.abs(gn - rn) <= TOL_BF16 * rms + (2.0 ** -8 if fused else 2.0 ** -7) * np.abs(rn))
        assert_close(kv_out, ref_kv, TOL_BF16, "kv_out")


def test_gated_forward_fp32_path():
    w = inputs.make_workload("pr1_ref")
    u = draw_gate(tuple(w["v"].shape), seed=3, dtype=torch.float32)
    got = run_gated(w["q"], w["k"], w["v"], u, w["lam"])
    check_gated(w["q"], w["k"], w["v"], u, w["lam"], got, 1e-4)


def test_zero_rows_give_zero():
    """A row whose attention output is exactly zero (here: v = 0) has no direction: y = 0, no NaN."""
    B, H, N, d = 1, 2, 200, 128
    q, k, v, _ = inputs.make_qkvdo(B, H, N, d, d, seed=4, with_do=False)
    v = torch.zeros_like(v)
    u = draw_gate((B, H, N, d), seed=4)
    y, o, rstd, _ = run_gated(q, k, v, u, torch.tensor([1.0, 0.5]))
    assert torch.all(y == 0) and torch.all(o == 0) and torch.all(rstd == 0)


@pytest.mark.parametrize("shape_", [(2, 3, 333, 64), (1, 4, 1000, 128), (1, 1, 5, 128)])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_gate_backward_kernel(shape_, out_dtype):
    B, H, N, e = shape_
    gen = torch.Generator("cpu")
    gen.manual_seed(N)
    o = (inputs.draw((B, H, N, e), gen, "normal", torch.float32) * 7.0).to(out_dtype)
    u = inputs.draw((B, H, N, e), gen, "normal", torch.bfloat16)
    dy = inputs.draw((B, H, N, e), gen, "normal", torch.bfloat16)
    sh = la.make_shape(B, H, N, e, e, torch.bfloat16, out_dtype)
    d_o = torch.empty((B, H, N, e), dtype=torch.bfloat16, device=DEV)
    d_u = torch.empty((B, H, N, e), dtype=out_dtype, device=DEV)
    la.la_gate_bwd(sh, o.to(DEV), u.to(DEV), dy.to(DEV), d_o, d_u)
    torch.cuda.synchronize()
    ref_do, ref_du = orc.norm_gate_bwd(o.double().numpy(), u, dy)
    # d_o is written in bf16 (it feeds la_bwd): its rounding is part of the result
    for g, r in ((d_o, ref_do), (d_u, ref_du)):
        gn = g.double().cpu().numpy().reshape(B * H, -1)
        rn = r.reshape(B * H, -1)
        rms = np.sqrt(np.mean(rn * rn, axis=1, keepdims=True))
        bound = 1e-5 * rms + (2.0 ** -8 * np.abs(rn) if g.dtype == torch.bfloat16 else 0.0)
        assert np.all(np.abs(gn - rn) <= bound)


def test_gated_forward_then_backward_chain():
    """la_fwd_gated -> la_gate_bwd -> la_bwd gives the gradients of <y, dy> with respect to q, k, v and u."""
    B, H, N, d = 1, 3, 700, 128
    q, k, v, _ = inputs.make_qkvdo(B, H, N, d, d, seed=61, with_do=False)
    u = draw_gate((B, H, N, d), seed=62)
    dy = draw_gate((B, H, N, d), seed=63)
    lam = torch.tensor([1.0, 0.98, 0.6])
    qg, kg, vg, ug, dyg = (x.to(DEV) for x in (q, k, v, u, dy))
    shape = la.make_shape(B, H, N, d, d, torch.bfloat16, torch.float32, 256)
    y, o = (torch.empty((B, H, N, d), dtype=torch.float32, device=DEV) for _ in range(2))
    ws_f = la.alloc_workspace(la.LA_OP_FWD, shape, DEV)
    ws_b = la.alloc_workspace(la.LA_OP_BWD, shape, DEV)
    la.la_fwd_gated(shape, qg, kg, vg, ug, lam, y, o, None, None, None, ws_f)
    d_o = torch.empty((B, H, N, d), dtype=torch.bfloat16, device=DEV)
    d_u, dq, dk, dv = (torch.empty((B, H, N, d), dtype=torch.float32, device=DEV) for _ in range(4))
    la.la_gate_bwd(shape, o, ug, dyg, d_o, d_u)
    la.la_bwd(shape, qg, kg, vg, d_o, lam, dq, dk, dv, None, None, None, ws_b, fwd_workspace=ws_f)
    torch.cuda.synchronize()
    la.device_status()
    lam64 = lam.double().numpy()
    ref_o = orc.fwd_rec(q, k, v, lam64)
    ref_do, ref_du = orc.norm_gate_bwd(ref_o, u, dy)
    assert_close(d_u, ref_du, TOL_BF16, "du")
    # d_o leaves la_gate_bwd in bf16 (it is an input tensor of la_bwd): checked with its own rounding allowed, and
    # la_bwd is then compared with the oracle run on those same bf16 values (same input bits on both sides)
    dn = d_o.double().cpu().numpy().reshape(B * H, -1)
    rn = ref_do.reshape(B * H, -1)
    rms = np.sqrt(np.mean(rn * rn, axis=1, keepdims=True))
    assert np.all(np.abs(dn - rn) <= TOL_BF16 * rms + 2.0 ** -8 * np.abs(rn))
    ref_dq, ref_dk, ref_dv = orc.bwd_rec(q, k, v, d_o.cpu(), lam64)
    for n, g, r in (("dq", dq, ref_dq), ("dk", dk, ref_dk), ("dv", dv, ref_dv)):
        assert_close(g, r, TOL_BF16, n)


@pytest.mark.parametrize("d", [64, 128])
def test_gated_forward_token_major_layout(d):
    """[B,N,H,d] tensors (q, k, v, u as a fused projection leaves them; y, o and rstd [B,N,H] in the same order)."""
    B, H, N = 2, 3, 650
    q, k, v, _ = inputs.make_qkvdo(B, H, N, d, d, seed=81, with_do=False)
    u = draw_gate((B, H, N, d), seed=82)
    lam = torch.tensor([1.0, 0.97, 0.3])
    ref_o = orc.fwd_rec(q, k, v, lam.double().numpy())
    ref_y, ref_rstd = orc.norm_gate_fwd(ref_o, u, want_rstd=True)
    tm = lambda x: x.permute(0, 2, 1, 3).contiguous().to(DEV)
    shape = la.make_shape(B, H, N, d, d, torch.bfloat16, torch.float32, 256, layout=la.LA_LAYOUT_BNHD)
    y, o = (torch.full((B, N, H, d), float("nan"), dtype=torch.float32, device=DEV) for _ in range(2))
    rstd = torch.full((B, N, H), float("nan"), dtype=torch.float32, device=DEV)
    ws = la.alloc_workspace(la.LA_OP_FWD, shape, DEV)
    la.la_fwd_gated(shape, tm(q), tm(k), tm(v), tm(u), lam, y, o, rstd, None, None, ws)
    torch.cuda.synchronize()
    la.device_status()
    assert_close(y.permute(0, 2, 1, 3), ref_y, TOL_BF16, "y")
    assert_close(o.permute(0, 2, 1, 3), ref_o, TOL_BF16, "o")
    r = rstd.permute(0, 2, 1).double().cpu().numpy()
    assert np.max(np.abs(r - ref_rstd) / ref_rstd) <= 1e-3
