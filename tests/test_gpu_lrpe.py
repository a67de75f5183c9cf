"""LRPE-d (Eq. 1) through the C ABI against the fp64 oracle's relative-position definition.

Outputs and the gradients of q, k, v, bf16 inputs: the position features are rounded to bf16 before they reach
the tensor cores (they are the operator's inputs, in the input dtype), which the oracle's exact features are not,
so every product term carries a relative error of up to 2^-9 twice; on top of the operator's own bound this gives
    |err| <= 2e-2 * RMS(ref[b,h]) + 2^-8 * |ref|
per element (the same form as the bf16-output mode of the plain operator; the second term matters for fast-decaying
heads, where one term dominates an element that is many RMS large).  fp32 inputs: 1e-4 * RMS.  The gradient of the angles is a position-weighted sum whose q and k parts cancel down to
the relative-position result, so its error scales with the absolute positions: with features and feature gradients
carrying a relative error of about 2^-8 (bf16 features on the tensor cores), independent from token to token,
    |err_i|  <~  2^-8 * sqrt( sum_{b,t} t^2 [ (qc gs)^2 + (qs gc)^2 + (kc hs)^2 + (ks hc)^2 ]_i )
where gc, gs (hc, hs) are the exact gradients of the two feature halves of q (k).  The tests bound the error by
4 times that figure, computed in fp64 from the oracle's side, and separately make sure the bound is small against
the result where the sequence is short (so that a wrong sign or index cannot hide in it)."""
import numpy as np
import pytest
import torch

from la_check import TOL_BF16, TOL_F32, assert_close
from oracle import la_oracle as orc
from paper_2307_14995_b200 import binding as la, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def features64(x, theta, pos0=0):
    x = np.asarray(x.double().numpy() if hasattr(x, "double") else x, np.float64)
    N = x.shape[2]
    ang = theta[None, :, None, :] * (pos0 + np.arange(N, dtype=np.float64))[None, None, :, None]
    return x * np.cos(ang), x * np.sin(ang)


def theta_bound(q, k, v, do, lam64, th64, pos0=0):
    """The error scale of d_theta described in the module docstring, [H, d], from fp64 quantities only."""
    qc, qs = features64(q, th64, pos0)
    kc, ks = features64(k, th64, pos0)
    qf = np.concatenate([qc, qs], -1)
    kf = np.concatenate([kc, ks], -1)
    N = qf.shape[2]
    t = np.arange(N)
    mask = np.tril(np.power(lam64[:, None, None], (t[:, None] - t[None, :]).clip(min=0)[None]))
    dA = np.einsum("bhtj,bhsj->bhts", do.double().numpy(), v.double().numpy()) * mask[None]
    gq = np.einsum("bhts,bhsi->bhti", dA, kf)          # gradients of the doubled features
    gk = np.einsum("bhts,bhti->bhsi", dA, qf)
    d = qc.shape[-1]
    pos = (pos0 + t)[None, None, :, None].astype(np.float64)
    sq = (pos * qc * gq[..., d:]) ** 2 + (pos * qs * gq[..., :d]) ** 2 + \
         (pos * kc * gk[..., d:]) ** 2 + (pos * ks * gk[..., :d]) ** 2
    return 2.0 ** -8 * np.sqrt(sq.sum(axis=(0, 2)))


def run_gpu(q, k, v, do, lam, theta, *, out_dtype=torch.float32, layout=None, pos0=0, kv_in=None, gko=None,
            want_state=False, seg_len=0):
    layout = la.LA_LAYOUT_BHND if layout is None else layout
    B, H, N, d = q.shape
    tm = (lambda x: x.permute(0, 2, 1, 3).contiguous()) if layout == la.LA_LAYOUT_BNHD else (lambda x: x)
    back = (lambda x: x.permute(0, 2, 1, 3)) if layout == la.LA_LAYOUT_BNHD else (lambda x: x)
    qg, kg, vg, dog = (tm(x).to(DEV) for x in (q, k, v, do))
    thg = theta.to(DEV)
    shape = la.make_shape(B, H, N, d, d, q.dtype, out_dtype, seg_len, layout=layout)
    new = lambda: torch.full(qg.shape, float("nan"), dtype=out_dtype, device=DEV)
    o, dq, dk, dv = new(), new(), new(), new()
    dth = torch.full((H, d), float("nan"), dtype=torch.float32, device=DEV)
    kv_out = torch.empty((2, B, H, d, d), dtype=torch.float32, device=DEV) if want_state else None
    gin = torch.empty((2, B, H, d, d), dtype=torch.float32, device=DEV) if want_state else None
    wf = torch.empty(la.lrpe_workspace_bytes(la.LA_OP_FWD, shape), dtype=torch.uint8, device=DEV)
    wb = torch.empty(la.lrpe_workspace_bytes(la.LA_OP_BWD, shape), dtype=torch.uint8, device=DEV)
    kin = None if kv_in is None else kv_in.to(DEV)
    gk = None if gko is None else gko.to(DEV)
    la.la_lrpe_fwd(shape, qg, kg, vg, thg, lam, o, pos0, kin, kv_out, wf)
    la.la_lrpe_bwd(shape, qg, kg, vg, dog, thg, lam, dq, dk, dv, dth, pos0, kin, gk, gin, wb)
    torch.cuda.synchronize()
    la.device_status()
    return back(o), back(dq), back(dk), back(dv), dth, kv_out, gin


def close_with_feature_rounding(got, ref, what, rel=2.0 ** -8):
    g = got.double().cpu().numpy()
    rms = np.sqrt(np.mean(ref * ref, axis=(2, 3), keepdims=True))
    excess = np.abs(g - ref) - (TOL_BF16 * rms + rel * np.abs(ref))
    assert np.all(np.isfinite(g)) and excess.max() <= 0, "%s: %.3e above the bound (RMS %.3e)" % (
        what, excess.max(), rms.max())


def check_theta(dth, ref, bound, what=""):
    err = np.abs(dth.double().cpu().numpy() - ref)
    ratio = err / np.maximum(bound, 1e-300)
    assert np.all(np.isfinite(err)) and ratio.max() <= 4.0, "%s d_theta: |err| / scale = %.2f" % (what, ratio.max())
    return ratio.max()


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("layout", ["BHND", "BNHD"])
def test_lrpe_forward_backward(d, layout):
    B, H, N = 2, 3, 333
    q, k, v, do = inputs.make_qkvdo(B, H, N, d, d, seed=21)
    lam = torch.tensor([1.0, 0.97, 0.5])
    theta = inputs.make_theta(H, d, seed=5)
    lam64, th64 = lam.double().numpy(), theta.double().numpy()
    o, dq, dk, dv, dth, _, _ = run_gpu(q, k, v, do, lam, theta, layout=getattr(la, "LA_LAYOUT_" + layout))
    close_with_feature_rounding(o, orc.lrpe_fwd_quad(q, k, v, lam64, th64), "o")
    rq, rk, rv, rth = orc.lrpe_bwd_quad(q, k, v, do, lam64, th64)
    close_with_feature_rounding(dq, rq, "dq")
    close_with_feature_rounding(dk, rk, "dk")
    close_with_feature_rounding(dv, rv, "dv")
    check_theta(dth, rth, theta_bound(q, k, v, do, lam64, th64))


def test_lrpe_long_sequence_in_segments():
    """Several segments (pre-pass, scan, walk) inside both runs of the operator, positions past 1000."""
    B, H, N, d = 1, 2, 1100, 128
    q, k, v, do = inputs.make_qkvdo(B, H, N, d, d, seed=27)
    lam = torch.tensor([1.0, 0.9])
    theta = inputs.make_theta(H, d, seed=10)
    lam64, th64 = lam.double().numpy(), theta.double().numpy()
    o, dq, dk, dv, dth, _, _ = run_gpu(q, k, v, do, lam, theta, seg_len=256)
    close_with_feature_rounding(o, orc.lrpe_fwd_quad(q, k, v, lam64, th64), "o")
    rq, rk, rv, rth = orc.lrpe_bwd_quad(q, k, v, do, lam64, th64)
    close_with_feature_rounding(dq, rq, "dq")
    close_with_feature_rounding(dk, rk, "dk")
    close_with_feature_rounding(dv, rv, "dv")
    check_theta(dth, rth, theta_bound(q, k, v, do, lam64, th64))


def test_lrpe_angle_gradient_has_teeth_on_a_short_sequence():
    """Short sequence, no decay in head 0: the error scale is far below the gradient itself, so a wrong sign,
    a swapped half or a shifted position in d_theta cannot pass."""
    B, H, N, d = 2, 2, 48, 64
    q, k, v, do = inputs.make_qkvdo(B, H, N, d, d, seed=22)
    lam = torch.tensor([1.0, 0.9])
    theta = inputs.make_theta(H, d, seed=6) * 0.2
    lam64, th64 = lam.double().numpy(), theta.double().numpy()
    *_, dth, _, _ = run_gpu(q, k, v, do, lam, theta)
    ref = orc.lrpe_bwd_quad(q, k, v, do, lam64, th64)[3]
    bound = theta_bound(q, k, v, do, lam64, th64)
    rms = np.sqrt(np.mean(ref * ref, axis=1))
    assert np.all(4.0 * np.median(bound, axis=1) < 0.25 * rms), (bound.max(), rms)
    check_theta(dth, ref, bound)
    err = np.abs(dth.double().cpu().numpy() - ref).max(axis=1)
    assert np.all(err < 0.25 * rms)


def test_lrpe_zero_angles_equal_the_plain_operator_bitwise():
    """theta = 0: the sin half is exactly zero and the cos half is the input, so the result must equal la_fwd's."""
    B, H, N, d = 1, 2, 300, 128
    q, k, v, do = inputs.make_qkvdo(B, H, N, d, d, seed=23)
    lam = torch.tensor([1.0, 0.8])
    theta = torch.zeros((H, d))
    o, dq, dk, dv, dth, _, _ = run_gpu(q, k, v, do, lam, theta)
    o2 = la.fwd(q.to(DEV), k.to(DEV), v.to(DEV), lam)
    dq2, dk2, dv2 = la.bwd(q.to(DEV), k.to(DEV), v.to(DEV), do.to(DEV), lam)
    for a, b in ((o, o2), (dq, dq2), (dk, dk2), (dv, dv2)):
        assert torch.equal(a, b)


def test_lrpe_fp32_inputs():
    B, H, N, d = 1, 2, 200, 64
    q, k, v, do = inputs.make_qkvdo(B, H, N, d, d, dtype=torch.float32, seed=24)
    q, k = q / 8, k / 8
    lam = torch.tensor([0.99, 0.7])
    theta = inputs.make_theta(H, d, seed=7)
    lam64, th64 = lam.double().numpy(), theta.double().numpy()
    o, dq, dk, dv, dth, _, _ = run_gpu(q, k, v, do, lam, theta)
    assert_close(o, orc.lrpe_fwd_quad(q, k, v, lam64, th64), TOL_F32, "o")
    rq, rk, rv, rth = orc.lrpe_bwd_quad(q, k, v, do, lam64, th64)
    for g, r, n in ((dq, rq, "dq"), (dk, rk, "dk"), (dv, rv, "dv")):
        assert_close(g, r, TOL_F32, n)
    scale = np.sqrt(np.mean(rth * rth, axis=1, keepdims=True))
    assert np.max(np.abs(dth.double().cpu().numpy() - rth) / scale) < 1e-3   # fp32 products times positions <= 200


def test_lrpe_bf16_outputs():
    B, H, N, d = 1, 2, 260, 128
    q, k, v, do = inputs.make_qkvdo(B, H, N, d, d, seed=25)
    lam = torch.tensor([1.0, 0.6])
    theta = inputs.make_theta(H, d, seed=8)
    lam64, th64 = lam.double().numpy(), theta.double().numpy()
    o, dq, dk, dv, dth, _, _ = run_gpu(q, k, v, do, lam, theta, out_dtype=torch.bfloat16)
    refs = (orc.lrpe_fwd_quad(q, k, v, lam64, th64),) + orc.lrpe_bwd_quad(q, k, v, do, lam64, th64)
    for g, r, n in zip((o, dq, dk, dv), refs[:4], ("o", "dq", "dk", "dv")):
        close_with_feature_rounding(g, r, n, rel=2.0 ** -7)      # feature rounding and the output's own rounding
    check_theta(dth, refs[4], theta_bound(q, k, v, do, lam64, th64))


def test_lrpe_chunks_with_states_and_position_offset():
    """Two chunks of one sequence: the second starts at pos0 = N1 from the first's state; results against the
    oracle on the whole sequence, and the state gradients chained backwards."""
    B, H, N, d = 1, 2, 400, 128
    N1 = 150
    q, k, v, do = inputs.make_qkvdo(B, H, N, d, d, seed=26)
    lam = torch.tensor([0.995, 0.8])
    theta = inputs.make_theta(H, d, seed=9)
    lam64, th64 = lam.double().numpy(), theta.double().numpy()
    cut = lambda x, a, b: x[:, :, a:b].contiguous()
    first = [cut(x, 0, N1) for x in (q, k, v, do)]
    second = [cut(x, N1, N) for x in (q, k, v, do)]
    # forward chain for the states, then backward in reverse order
    o1, _, _, _, _, kv1, _ = run_gpu(*first, lam, theta, want_state=True)
    o2, dq2, dk2, dv2, dth2, _, gin2 = run_gpu(*second, lam, theta, pos0=N1, kv_in=kv1, want_state=True)
    _, dq1, dk1, dv1, dth1, _, _ = run_gpu(*first, lam, theta, gko=gin2, want_state=True)
    ref_o = orc.lrpe_fwd_quad(q, k, v, lam64, th64)
    rq, rk, rv, rth = orc.lrpe_bwd_quad(q, k, v, do, lam64, th64)
    close_with_feature_rounding(torch.cat([o1, o2], 2), ref_o, "o")
    close_with_feature_rounding(torch.cat([dq1, dq2], 2), rq, "dq")
    close_with_feature_rounding(torch.cat([dk1, dk2], 2), rk, "dk")
    close_with_feature_rounding(torch.cat([dv1, dv2], 2), rv, "dv")
    # the angle gradient of the whole sequence is the sum over the chunks, plus what flows through the handed-over
    # state -- which the chain above already carries in the first chunk's feature gradients
    check_theta(dth1 + dth2, rth, theta_bound(q, k, v, do, lam64, th64), "chunks")


def test_lrpe_rejects_bad_arguments():
    shape = la.make_shape(1, 2, 64, 128, 128, torch.bfloat16, torch.float32, 0)
    x = torch.zeros((1, 2, 64, 128), dtype=torch.bfloat16, device=DEV)
    o = torch.zeros((1, 2, 64, 128), dtype=torch.float32, device=DEV)
    th = torch.zeros((2, 128), device=DEV)
    ws = torch.empty(la.lrpe_workspace_bytes(la.LA_OP_FWD, shape), dtype=torch.uint8, device=DEV)
    lam = torch.tensor([1.0, 0.5])
    with pytest.raises(la.LaError):
        la.la_lrpe_fwd(shape, x, x, x, th, lam, o, 0, None, None, ws[:1024])          # workspace too small
    with pytest.raises(la.LaError):
        la.la_lrpe_fwd(shape, x, x, x, th, lam, o, -1, None, None, ws)                # negative position
    with pytest.raises(la.LaError):
        la.la_lrpe_fwd(shape, x, x, x, th, torch.tensor([1.0, 1.5]), o, 0, None, None, ws)   # lambda out of range
