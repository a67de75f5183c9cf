"""Pins for the CPU oracle: each routine is checked against something other than
itself -- a hand-worked example, closed forms, numpy library routines for the
no-decay case, a literal brute-force loop, finite differences, and the other
form of the same function.  No GPU involved."""
import json
import os

import numpy as np
import pytest
import torch

from oracle import la_oracle as orc
from paper_2307_14995_b200 import inputs

HERE = os.path.dirname(os.path.abspath(__file__))


def rand_inputs(B, H, N, d, e, seed=0, dtype=torch.float32):
    q, k, v, do = inputs.make_qkvdo(B, H, N, d, e, dtype=dtype, seed=seed)
    return q, k, v, do


def brute_forward(q, k, v, lam):
    """The defining sum o_t = sum_{s<=t} lambda^(t-s) (q_t . k_s) v_s as literal Python loops."""
    q, k, v = (np.asarray(x, dtype=np.float64) for x in (q, k, v))
    B, H, N, d = q.shape
    e = v.shape[-1]
    o = np.zeros((B, H, N, e))
    for b in range(B):
        for h in range(H):
            for t in range(N):
                for s in range(t + 1):
                    dot = 0.0
                    for i in range(d):
                        dot += q[b, h, t, i] * k[b, h, s, i]
                    w = float(lam[h]) ** (t - s)
                    for j in range(e):
                        o[b, h, t, j] += w * dot * v[b, h, s, j]
    return o


def relerr(a, b):
    a, b = np.asarray(a, np.float64), np.asarray(b, np.float64)
    rms = np.sqrt(np.mean(b * b)) + 1e-300
    return np.max(np.abs(a - b)) / rms


# --- hand-worked example ------------------------------------------------------
def test_hand_worked_example():
    g = json.load(open(os.path.join(HERE, "golden", "hand_example.json")))
    sh = (1, 1, 3, 1)
    q, k, v, do = (np.array(g[n], np.float32).reshape(sh) for n in ("q", "k", "v", "dO"))
    lam = np.array([g["lambda"]])
    o, kv = orc.fwd_rec(q, k, v, lam, want_state=True)
    assert np.array_equal(o.ravel(), np.array(g["o"]))
    assert kv.ravel()[0] == g["kv_out"]
    assert np.array_equal(orc.fwd_quad(q, k, v, lam).ravel(), np.array(g["o"]))
    for fn in (lambda: orc.bwd_rec(q, k, v, do, lam), lambda: orc.bwd_quad(q, k, v, do, lam)):
        dq, dk, dv = fn()
        assert np.array_equal(dq.ravel(), np.array(g["dq"]))
        assert np.array_equal(dk.ravel(), np.array(g["dk"]))
        assert np.array_equal(dv.ravel(), np.array(g["dv"]))
    *_, gin = orc.bwd_rec(q, k, v, do, lam, want_state_grad=True)
    assert gin.ravel()[0] == g["grad_kv_in"]
    for kind in ("o", "dq", "dk", "dv"):
        r = orc.rows(kind, q, k, v, do, lam, [0, 0, 0], [0, 1, 2])
        assert np.array_equal(r.ravel(), np.array(g[kind]))


# --- brute force on tiny inputs ----------------------------------------------
@pytest.mark.parametrize("N,d,e", [(1, 1, 1), (5, 2, 3), (8, 3, 2)])
def test_brute_force_tiny(N, d, e):
    q, k, v, _ = rand_inputs(2, 2, N, d, e, seed=3)
    lam = np.array([0.7, 1.0])
    ref = brute_forward(q, k, v, lam)
    assert relerr(orc.fwd_rec(q, k, v, lam), ref) < 1e-14
    assert relerr(orc.fwd_quad(q, k, v, lam), ref) < 1e-14


# --- closed forms ---------------------------------------------------------------
@pytest.mark.parametrize("lam", [float(np.exp(-2.0)), 0.5, 1.0])
def test_closed_form_geometric(lam):
    """q_t = k_t = e_1, v_t = 1: o_t[j] = (1 - lam^(t+1)) / (1 - lam), or t+1 for lam = 1;
    with dO = 1: dv_s[j] = (1 - lam^(N-s)) / (1 - lam)."""
    N, d, e = 40, 3, 2
    q = np.zeros((1, 1, N, d), np.float32)
    q[..., 0] = 1.0
    k = q.copy()
    v = np.ones((1, 1, N, e), np.float32)
    do = np.ones((1, 1, N, e), np.float32)
    t = np.arange(N)
    want_o = (t + 1.0) if lam == 1.0 else (1 - lam ** (t + 1)) / (1 - lam)
    want_dv = (N - t).astype(float) if lam == 1.0 else (1 - lam ** (N - t)) / (1 - lam)
    L = np.array([lam])
    for o in (orc.fwd_rec(q, k, v, L), orc.fwd_quad(q, k, v, L)):
        assert np.allclose(o[0, 0, :, 0], want_o, rtol=1e-13, atol=0)
        assert np.allclose(o[0, 0, :, 1], want_o, rtol=1e-13, atol=0)
    for dq, dk, dv in (orc.bwd_rec(q, k, v, do, L), orc.bwd_quad(q, k, v, do, L)):
        assert np.allclose(dv[0, 0, :, 0], want_dv, rtol=1e-13, atol=0)
        # dq_t = kv_t do_t = (sum_j kv[0,j]) e_1, and kv[0,j] = o_t[j]
        assert np.allclose(dq[0, 0, :, 0], e * want_o, rtol=1e-13, atol=0)
        assert np.all(dq[0, 0, :, 1:] == 0)
        # dk_s = R_s v_s with R_s[0,j] = dv_s[j]
        assert np.allclose(dk[0, 0, :, 0], e * want_dv, rtol=1e-13, atol=0)
    if lam == float(np.exp(-2.0)):
        long_q = np.zeros((1, 1, 400, 1), np.float32) + 1.0
        o = orc.fwd_rec(long_q, long_q, long_q, L)
        assert abs(o[0, 0, -1, 0] - 1.1565176427496657) < 1e-15


def test_no_decay_is_prefix_sum():
    """lambda = 1: O = tril(Q K^T) V, i.e. prefix sums of k_s v_s^T (numpy cumsum / tril)."""
    q, k, v, do = rand_inputs(1, 2, 33, 4, 5, seed=5)
    lam = np.array([1.0, 1.0])
    qn, kn, vn, don = (x.double().numpy() for x in (q, k, v, do))
    kv_prefix = np.cumsum(np.einsum("bhsi,bhsj->bhsij", kn, vn), axis=2)
    want = np.einsum("bhti,bhtij->bhtj", qn, kv_prefix)
    assert relerr(orc.fwd_rec(q, k, v, lam), want) < 1e-14
    assert relerr(orc.fwd_quad(q, k, v, lam), want) < 1e-14
    A = np.tril(np.einsum("bhti,bhsi->bhts", qn, kn))
    dA = np.tril(np.einsum("bhtj,bhsj->bhts", don, vn))
    want_g = (np.einsum("bhts,bhsi->bhti", dA, kn), np.einsum("bhts,bhti->bhsi", dA, qn),
              np.einsum("bhts,bhtj->bhsj", A, don))
    for got in (orc.bwd_rec(q, k, v, do, lam), orc.bwd_quad(q, k, v, do, lam)):
        for g, w in zip(got, want_g):
            assert relerr(g, w) < 1e-14
    # the state handed out is the last prefix sum, rows = key feature, columns = value feature
    # (d = 4 and e = 5 differ, so a transposed convention cannot pass)
    _, kv_out = orc.fwd_rec(q, k, v, lam, want_state=True)
    assert kv_out.shape == (1, 2, 4, 5)
    assert relerr(kv_out, kv_prefix[:, :, -1]) < 1e-14


@pytest.mark.parametrize("lam_val", [0.9, 0.35])
def test_state_orientation_and_decay_by_explicit_sum(lam_val):
    """kv_out[i, j] = sum_s lambda^(N-1-s) k_s[i] v_s[j], written as a plain numpy loop over s; with a
    state handed in, it enters as lambda^N kv_in, and grad_kv_in = lambda^N grad_kv_out +
    sum_t lambda^(t+1) q_t do_t^T in the same orientation (d != e throughout)."""
    B, H, N, d, e = 1, 2, 21, 3, 5
    q, k, v, do = rand_inputs(B, H, N, d, e, seed=51)
    lam = np.array([lam_val, 1.0])
    qn, kn, vn, don = (x.double().numpy() for x in (q, k, v, do))
    rng = np.random.default_rng(3)
    kv_in = rng.standard_normal((B, H, d, e))
    gko = rng.standard_normal((B, H, d, e))
    want_kv = np.zeros((B, H, d, e))
    want_gin = np.zeros((B, H, d, e))
    for h in range(H):
        for s in range(N):
            want_kv[0, h] += lam[h] ** (N - 1 - s) * np.outer(kn[0, h, s], vn[0, h, s])
            want_gin[0, h] += lam[h] ** (s + 1) * np.outer(qn[0, h, s], don[0, h, s])
    _, kv0 = orc.fwd_rec(q, k, v, lam, want_state=True)
    assert relerr(kv0, want_kv) < 1e-14
    decay_n = (lam ** N)[None, :, None, None]
    o1, kv1 = orc.fwd_rec(q, k, v, lam, kv_in=kv_in, want_state=True)
    assert relerr(kv1, want_kv + decay_n * kv_in) < 1e-14
    # o_t with a state handed in gains lambda^(t+1) kv_in^T q_t
    t = np.arange(N)
    extra = np.einsum("bhti,bhij->bhtj", qn, kv_in) * (lam[None, :, None] ** (t[None, None, :] + 1))[..., None]
    assert relerr(o1 - orc.fwd_rec(q, k, v, lam), extra) < 1e-13
    *_, gin = orc.bwd_rec(q, k, v, do, lam, kv_in=kv_in, grad_kv_out=gko, want_state_grad=True)
    assert relerr(gin, want_gin + decay_n * gko) < 1e-14


def test_fast_decay_limit_is_diagonal():
    """lambda -> 0: o_t = (q_t.k_t) v_t, dq_t = (do_t.v_t) k_t, dk_t = (do_t.v_t) q_t, dv_t = (q_t.k_t) do_t."""
    q, k, v, do = rand_inputs(1, 1, 17, 4, 3, seed=7)
    lam = np.array([1e-30])
    qn, kn, vn, don = (x.double().numpy() for x in (q, k, v, do))
    qk = np.sum(qn * kn, -1, keepdims=True)
    dov = np.sum(don * vn, -1, keepdims=True)
    for o in (orc.fwd_rec(q, k, v, lam), orc.fwd_quad(q, k, v, lam)):
        assert np.all(np.isfinite(o)) and relerr(o, qk * vn) < 1e-14
    for dq, dk, dv in (orc.bwd_rec(q, k, v, do, lam), orc.bwd_quad(q, k, v, do, lam)):
        assert relerr(dq, dov * kn) < 1e-14
        assert relerr(dk, dov * qn) < 1e-14
        assert relerr(dv, qk * don) < 1e-14


# --- the two forms against each other -----------------------------------------
@pytest.mark.parametrize("shape", [(1, 2, 96, 8, 6), (2, 3, 257, 16, 16), (1, 1, 1, 4, 4)])
def test_recurrence_equals_quadratic(shape):
    B, H, N, d, e = shape
    q, k, v, do = rand_inputs(B, H, N, d, e, seed=11)
    lam = inputs.decay_rates(H, 0.5).double().numpy()
    assert relerr(orc.fwd_rec(q, k, v, lam), orc.fwd_quad(q, k, v, lam)) < 1e-12
    for a, b in zip(orc.bwd_rec(q, k, v, do, lam), orc.bwd_quad(q, k, v, do, lam)):
        assert relerr(a, b) < 1e-12


def test_recurrence_equals_quadratic_pr1_workload():
    w = inputs.make_workload("pr1_ref")
    lam = w["lam"].double().numpy()
    assert np.allclose(lam, [1.0, np.exp(-2.0)], rtol=1e-7)
    assert relerr(orc.fwd_rec(w["q"], w["k"], w["v"], lam), orc.fwd_quad(w["q"], w["k"], w["v"], lam)) < 1e-12
    for a, b in zip(orc.bwd_rec(w["q"], w["k"], w["v"], w["do"], lam),
                    orc.bwd_quad(w["q"], w["k"], w["v"], w["do"], lam)):
        assert relerr(a, b) < 1e-12


def test_sampled_rows_equal_full_forms():
    B, H, N, d, e = 2, 2, 70, 8, 5
    q, k, v, do = rand_inputs(B, H, N, d, e, seed=13)
    lam = np.array([0.9, 0.3])
    o = orc.fwd_rec(q, k, v, lam)
    dq, dk, dv = orc.bwd_rec(q, k, v, do, lam)
    bh = np.array([0, 1, 2, 3, 3, 0])
    t = np.array([0, 69, 31, 32, 1, 68])
    for kind, full in (("o", o), ("dq", dq), ("dk", dk), ("dv", dv)):
        got = orc.rows(kind, q, k, v, do, lam, bh, t)
        want = full.reshape(B * H, N, -1)[bh, t]
        assert relerr(got, want) < 1e-12


# --- gradients: finite differences, Euler identities, role swaps -------------------
def test_finite_differences_including_state_gradients():
    B, H, N, d, e = 1, 2, 12, 3, 4
    q, k, v, do = rand_inputs(B, H, N, d, e, seed=17)
    lam = np.array([0.8, 1.0])
    rng = np.random.default_rng(0)
    kv_in = rng.standard_normal((B, H, d, e))
    gko = rng.standard_normal((B, H, d, e))
    qn, kn, vn, don = (x.double().numpy().copy() for x in (q, k, v, do))

    def loss(qq, kk, vv, s_in):
        o, s_out = orc.fwd_rec(qq, kk, vv, lam, kv_in=s_in, want_state=True)
        return float(np.sum(o * don) + np.sum(s_out * gko))

    dq, dk, dv, gin = orc.bwd_rec(q, k, v, do, lam, kv_in=kv_in, grad_kv_out=gko, want_state_grad=True)
    # inputs are fp32 containers: use perturbations that are exact in fp32 (power of two)
    h = 2.0 ** -10
    for name, arr, grad in (("q", qn, dq), ("k", kn, dk), ("v", vn, dv)):
        for _ in range(6):
            idx = tuple(rng.integers(0, s) for s in arr.shape)
            base = float(np.float32(arr[idx]))
            args = {"q": qn, "k": kn, "v": vn}
            plus, minus = arr.copy(), arr.copy()
            plus[idx], minus[idx] = base + h, base - h
            lp = loss(*[plus if n == name else args[n] for n in ("q", "k", "v")], kv_in)
            lm = loss(*[minus if n == name else args[n] for n in ("q", "k", "v")], kv_in)
            fd = (lp - lm) / (2 * h)  # the loss is linear in each single entry: exact up to rounding
            assert abs(fd - grad[idx]) <= 1e-9 * max(1.0, abs(grad[idx])), (name, idx, fd, grad[idx])
    for _ in range(6):
        idx = tuple(rng.integers(0, s) for s in kv_in.shape)
        plus, minus = kv_in.copy(), kv_in.copy()
        plus[idx] += 1e-3
        minus[idx] -= 1e-3
        fd = (loss(qn, kn, vn, plus) - loss(qn, kn, vn, minus)) / 2e-3
        assert abs(fd - gin[idx]) <= 1e-9 * max(1.0, abs(gin[idx]))


def test_euler_identities():
    """O is linear in each of q, k, v, so <Q,dQ> = <K,dK> = <V,dV> = <O,dO> per head."""
    B, H, N, d, e = 1, 3, 50, 6, 7
    q, k, v, do = rand_inputs(B, H, N, d, e, seed=19)
    lam = np.array([1.0, 0.95, 0.2])
    o = orc.fwd_rec(q, k, v, lam)
    dq, dk, dv = orc.bwd_rec(q, k, v, do, lam)
    qn, kn, vn, don = (x.double().numpy() for x in (q, k, v, do))
    ref = np.sum(o * don, axis=(2, 3))
    for a, b in ((qn, dq), (kn, dk), (vn, dv)):
        assert np.allclose(np.sum(a * b, axis=(2, 3)), ref, rtol=1e-12)


def test_role_swap_identities():
    """dQ = LA(q:=dO, k:=V, v:=K); dK, dV are the same operator run on the reversed sequence."""
    B, H, N, d, e = 1, 2, 40, 5, 5
    q, k, v, do = rand_inputs(B, H, N, d, e, seed=23)
    lam = np.array([0.9, 0.6])
    dq, dk, dv = orc.bwd_rec(q, k, v, do, lam)
    assert relerr(orc.fwd_rec(do, v, k, lam), dq) < 1e-13
    flip = lambda x: torch.flip(x, dims=[2])
    assert relerr(orc.fwd_rec(flip(v), flip(do), flip(q), lam)[:, :, ::-1], dk) < 1e-13
    assert relerr(orc.fwd_rec(flip(k), flip(q), flip(do), lam)[:, :, ::-1], dv) < 1e-13


def test_linearity_scaling():
    q, k, v, _ = rand_inputs(1, 1, 20, 4, 4, seed=29)
    lam = np.array([0.75])
    base = orc.fwd_rec(q, k, v, lam)
    assert relerr(orc.fwd_rec(2 * q, 4 * k, 0.5 * v, lam), 4 * base) < 1e-15


# --- random tiny shapes: both forms of the oracle against the literal loops -----------
from hypothesis import given, settings, strategies as st  # noqa: E402


@settings(max_examples=25, deadline=None)
@given(N=st.integers(1, 9), d=st.integers(1, 4), e=st.integers(1, 4), H=st.integers(1, 2),
       lam0=st.sampled_from([1.0, 0.97, 0.5, 0.05, 1e-30]), seed=st.integers(0, 10_000))
def test_random_tiny_shapes_against_brute_force(N, d, e, H, lam0, seed):
    """Any N >= 1 and d != e: recurrence == quadratic form == literal loops (forward), and the two
    backward forms agree with each other and satisfy the Euler identities."""
    q, k, v, do = rand_inputs(1, H, N, d, e, seed=seed)
    lam = np.array([lam0, 0.8][:H])
    want = brute_forward(q.numpy(), k.numpy(), v.numpy(), lam)
    o_rec, o_quad = orc.fwd_rec(q, k, v, lam), orc.fwd_quad(q, k, v, lam)
    scale = np.sqrt(np.mean(want * want)) + 1e-30
    assert np.max(np.abs(o_rec - want)) <= 1e-13 * scale + 1e-300
    assert np.max(np.abs(o_quad - want)) <= 1e-13 * scale + 1e-300
    g_rec, g_quad = orc.bwd_rec(q, k, v, do, lam), orc.bwd_quad(q, k, v, do, lam)
    for a, b in zip(g_rec, g_quad):
        assert np.max(np.abs(a - b)) <= 1e-12 * (np.sqrt(np.mean(b * b)) + 1e-30) + 1e-300
    qn, kn, vn, don = (x.double().numpy() for x in (q, k, v, do))
    ref = np.sum(want * don, axis=(2, 3))
    for a, b in ((qn, g_rec[0]), (kn, g_rec[1]), (vn, g_rec[2])):
        assert np.allclose(np.sum(a * b, axis=(2, 3)), ref, rtol=1e-10, atol=1e-12 * (np.abs(ref).max() + 1e-30))


# --- state hand-over, decode, causality ---------------------------------------------
@pytest.mark.parametrize("split", [1, 13, 32, 49])
def test_chaining_equals_one_call(split):
    B, H, N, d, e = 1, 2, 50, 4, 6
    q, k, v, _ = rand_inputs(B, H, N, d, e, seed=31)
    lam = np.array([0.85, 1.0])
    full, kv_full = orc.fwd_rec(q, k, v, lam, want_state=True)
    o1, kv1 = orc.fwd_rec(q[:, :, :split], k[:, :, :split], v[:, :, :split], lam, want_state=True)
    o2, kv2 = orc.fwd_rec(q[:, :, split:], k[:, :, split:], v[:, :, split:], lam, kv_in=kv1, want_state=True)
    assert relerr(np.concatenate([o1, o2], axis=2), full) < 1e-14
    assert relerr(kv2, kv_full) < 1e-14


def test_decode_steps_equal_parallel_form():
    B, H, P, S, d, e = 2, 2, 9, 5, 4, 3
    q, k, v, _ = rand_inputs(B, H, P + S, d, e, seed=37)
    lam = np.array([0.9, 0.5])
    full = orc.fwd_quad(q, k, v, lam)
    _, kv = orc.fwd_rec(q[:, :, :P], k[:, :, :P], v[:, :, :P], lam, want_state=True)
    for s in range(S):
        t = P + s
        o = orc.decode_step(q[:, :, t], k[:, :, t], v[:, :, t], lam, kv)
        assert relerr(o, full[:, :, t]) < 1e-13


def test_causality_bitwise():
    B, H, N, d, e = 1, 1, 30, 4, 4
    q, k, v, do = rand_inputs(B, H, N, d, e, seed=41)
    lam = np.array([0.9])
    t0 = 17
    q2, k2, v2, do2 = (x.clone() for x in (q, k, v, do))
    q2[:, :, t0] += 1
    k2[:, :, t0] -= 2
    v2[:, :, t0] *= 3
    o, o2 = orc.fwd_rec(q, k, v, lam), orc.fwd_rec(q2, k2, v2, lam)
    assert np.array_equal(o[:, :, :t0], o2[:, :, :t0]) and not np.array_equal(o[:, :, t0:], o2[:, :, t0:])
    dq, _, _ = orc.bwd_rec(q, k, v, do, lam)
    dqb, _, _ = orc.bwd_rec(q2, k2, v2, do, lam)
    assert np.array_equal(dq[:, :, :t0], dqb[:, :, :t0])
    do2[:, :, t0] += 1
    _, dk, dv = orc.bwd_rec(q, k, v, do, lam)
    _, dkb, dvb = orc.bwd_rec(q2, k, v, do2, lam)
    assert np.array_equal(dk[:, :, t0 + 1:], dkb[:, :, t0 + 1:])
    assert np.array_equal(dv[:, :, t0 + 1:], dvb[:, :, t0 + 1:])


# --- the prescaled recurrence: equal while it is safe, broken when it is not ----------
def test_origin_inference_agrees_then_overflows():
    q, k, v, _ = rand_inputs(1, 1, 64, 4, 4, seed=43)
    lam = np.array([0.9])
    assert relerr(orc.fwd_origin(q, k, v, lam), orc.fwd_rec(q, k, v, lam)) < 1e-10
    # lambda = e^-2: lambda^-t overflows fp64 once 2 t > ~709
    q, k, v, _ = rand_inputs(1, 1, 500, 4, 4, seed=43)
    lam = np.array([np.exp(-2.0)])
    with np.errstate(all="ignore"):
        bad = orc.fwd_origin(q, k, v, lam)
    good = orc.fwd_rec(q, k, v, lam)
    assert np.all(np.isfinite(good))
    assert not np.all(np.isfinite(bad[:, :, 400:]))


# --- input generator facts ------------------------------------------------------------
def test_decay_schedule_values():
    lam = inputs.decay_rates(2, 0.5).double().numpy()
    assert np.allclose(lam, [1.0, np.exp(-2.0)], rtol=1e-7)
    lam = inputs.decay_rates(32, 0.9).double().numpy()
    assert lam[0] == 1.0 and np.allclose(lam[-1], np.exp(-0.025 * 31), rtol=1e-7)
    lam = inputs.decay_rates(16, 0.25).double().numpy()
    assert np.allclose(lam[-1], np.exp(-0.375 * 15), rtol=1e-6)


def test_generator_is_seeded_and_bf16_exact():
    a = inputs.make_qkvdo(1, 2, 16, 8, 8, seed=0)
    b = inputs.make_qkvdo(1, 2, 16, 8, 8, seed=0)
    for x, y in zip(a, b):
        assert torch.equal(x, y) and x.dtype == torch.bfloat16
    # SiLU moments of the draw
    q = inputs.make_qkvdo(1, 4, 4096, 64, 64, seed=0, dtype=torch.float32)[0]
    assert abs(q.mean().item() - 0.20662) < 2e-3
    assert abs((q * q).mean().item() - 0.35578) < 4e-3


# --- SimpleRMSNorm followed by the gate (Eq. 3 with Eq. 8) ---------------------------------
def test_norm_gate_hand_worked_example():
    g = json.load(open(os.path.join(HERE, "golden", "norm_gate_example.json")))
    o = np.array(g["o"]).reshape(1, 2)
    u = np.array(g["u"], np.float32).reshape(1, 2)
    dy = np.array(g["dy"], np.float32).reshape(1, 2)
    y, rstd = orc.norm_gate_fwd(o, u, want_rstd=True)
    assert np.allclose(y.ravel(), g["y"], rtol=1e-15) and abs(rstd[0] - g["rstd"]) < 1e-16
    d_o, d_u = orc.norm_gate_bwd(o, u, dy)
    assert np.allclose(d_o.ravel(), g["do"], rtol=1e-14) and np.allclose(d_u.ravel(), g["du"], rtol=1e-15)


def test_norm_gate_invariants_and_finite_differences():
    rng = np.random.default_rng(7)
    rows, e = 6, 5
    o = rng.standard_normal((rows, e)) * np.array([1e-3, 1, 10, 1e3, 1, 1])[:, None]
    u = rng.standard_normal((rows, e)).astype(np.float32)
    dy = rng.standard_normal((rows, e)).astype(np.float32)
    y = orc.norm_gate_fwd(o, u)
    # the normalised row has root-mean-square 1, whatever the scale of o
    assert np.allclose(np.sqrt(np.mean((y / u) ** 2, axis=1)), 1.0, rtol=1e-13)
    # scale invariance of the norm: y(a o) = y(o); do(a o) = do(o) / a; do is orthogonal to o
    d_o, d_u = orc.norm_gate_bwd(o, u, dy)
    assert np.allclose(orc.norm_gate_fwd(7.5 * o, u), y, rtol=1e-13)
    assert np.allclose(orc.norm_gate_bwd(7.5 * o, u, dy)[0], d_o / 7.5, rtol=1e-12)
    assert np.all(np.abs(np.sum(o * d_o, axis=1)) <= 1e-12 * np.linalg.norm(o, axis=1) * np.linalg.norm(d_o, axis=1))
    # central differences of L = <y, dy> in o and in u
    L = lambda oo, uu: float(np.sum(orc.norm_gate_fwd(oo, uu) * dy))
    for (r, j) in [(0, 1), (2, 4), (3, 0), (5, 2)]:
        h = 1e-6 * max(1.0, abs(o[r, j]))
        op, om = o.copy(), o.copy()
        op[r, j] += h
        om[r, j] -= h
        fd = (L(op, u) - L(om, u)) / (2 * h)
        assert abs(fd - d_o[r, j]) <= 1e-6 * max(abs(fd), np.abs(d_o[r]).max())
        # L is linear in u: the derivative is dy * n, exactly the forward value divided by u
        assert abs(d_u[r, j] - dy[r, j] * y[r, j] / u[r, j]) <= 1e-12 * abs(d_u[r, j]) + 1e-300
    # a zero row is given y = 0 and zero gradients (Eq. 8 has no epsilon)
    z = np.zeros((1, e))
    assert np.all(orc.norm_gate_fwd(z, u[:1]) == 0) and np.all(orc.norm_gate_bwd(z, u[:1], dy[:1])[0] == 0)


# --- LRPE-d (Eq. 1): decay and rotation of the relative position ---------------------------------------------
def lrpe_features(x, theta, pos0=0):
    """[x cos(theta t), x sin(theta t)] along the feature axis: the split of Eq. 1's rotation into a factor that
    depends on the query position only and one that depends on the key position only."""
    x = np.asarray(x, np.float64)
    N = x.shape[2]
    ang = np.asarray(theta, np.float64)[None, :, None, :] * (pos0 + np.arange(N, dtype=np.float64))[None, None, :, None]
    return np.concatenate([x * np.cos(ang), x * np.sin(ang)], axis=-1)


def test_lrpe_hand_worked_two_tokens():
    g = json.load(open(os.path.join(HERE, "golden", "lrpe_example.json")))
    sh = (1, 1, 2, 2)
    q, k, v, do = (np.array(g[n], np.float32).reshape(sh) for n in ("q", "k", "v", "dO"))
    lam, th = np.array([g["lambda"]]), np.array([g["theta"]])
    o = orc.lrpe_fwd_quad(q, k, v, lam, th)
    np.testing.assert_allclose(o.ravel(), np.array(g["o"]), rtol=0, atol=1e-14)
    dq, dk, dv, dth = orc.lrpe_bwd_quad(q, k, v, do, lam, th)
    for got, name in ((dq, "dq"), (dk, "dk"), (dv, "dv"), (dth, "dtheta")):
        np.testing.assert_allclose(got.ravel(), np.array(g[name]), rtol=0, atol=1e-14, err_msg=name)


def test_lrpe_zero_angle_is_the_plain_operator():
    q, k, v, do = rand_inputs(2, 3, 40, 8, 6, seed=5)
    lam = np.array([1.0, 0.9, 0.4])
    th = np.zeros((3, 8))
    np.testing.assert_allclose(orc.lrpe_fwd_quad(q, k, v, lam, th), orc.fwd_quad(q, k, v, lam), rtol=0, atol=1e-13)
    got = orc.lrpe_bwd_quad(q, k, v, do, lam, th)
    ref = orc.bwd_quad(q, k, v, do, lam)
    for a, b in zip(got[:3], ref):
        np.testing.assert_allclose(a, b, rtol=0, atol=1e-12)
    assert np.all(got[3] == 0.0)        # sin(0) = 0: no first-order dependence on theta at theta = 0


def test_lrpe_is_the_real_part_of_the_complex_form():
    """Eq. 1 as printed: a_ts = q_t^T k_s lambda^(t-s) exp(i theta (t-s)), evaluated with complex numbers."""
    B, H, N, d, e = 1, 2, 33, 6, 5
    q, k, v, _ = rand_inputs(B, H, N, d, e, seed=6)
    q, k, v = (np.asarray(x, np.float64) for x in (q, k, v))
    lam = np.array([0.97, 0.6])
    th = inputs.make_theta(H, d, seed=3).double().numpy() * 50.0       # angles large enough to wrap within 33 tokens
    t = np.arange(N)
    rot = np.exp(1j * th[None, :, None, :] * t[None, None, :, None])    # [1,H,N,d]
    scores = np.einsum("bhti,bhsi->bhts", q * rot, np.conj(k * rot))
    mask = np.tril(np.power(lam[:, None, None], (t[:, None] - t[None, :]).clip(min=0)[None]))
    o_ref = np.einsum("bhts,bhsj->bhtj", (scores * mask[None]).real, v)
    assert relerr(orc.lrpe_fwd_quad(q, k, v, lam, th), o_ref) < 1e-12


@pytest.mark.parametrize("pos0", [0, 1000])
def test_lrpe_separates_into_position_features(pos0):
    """cos(a - b) = cos a cos b + sin a sin b: the plain operator on doubled features [x cos, x sin], evaluated at
    absolute positions (any common offset), equals the relative-position definition, for outputs and for the
    gradients with respect to v."""
    B, H, N, d, e = 2, 2, 50, 4, 3
    q, k, v, do = rand_inputs(B, H, N, d, e, seed=7)
    lam = np.array([1.0, 0.8])
    th = inputs.make_theta(H, d, seed=4).double().numpy() * 20.0
    qf, kf = lrpe_features(q, th, pos0), lrpe_features(k, th, pos0)
    o = orc.lrpe_fwd_quad(q, k, v, lam, th)
    assert relerr(orc.fwd_quad(qf.astype(np.float32), kf.astype(np.float32), v, lam), o) < 1e-5   # fp32 containers
    # in fp64 throughout (the recurrence takes fp32 containers, so use the einsum definition here)
    t = np.arange(N)
    mask = np.tril(np.power(lam[:, None, None], (t[:, None] - t[None, :]).clip(min=0)[None]))
    o2 = np.einsum("bhts,bhsj->bhtj", np.einsum("bhti,bhsi->bhts", qf, kf) * mask[None], np.asarray(v, np.float64))
    assert relerr(o2, o) < 1e-12
    dv = orc.lrpe_bwd_quad(q, k, v, do, lam, th)[2]
    dv2 = np.einsum("bhts,bhtj->bhsj", np.einsum("bhti,bhsi->bhts", qf, kf) * mask[None], np.asarray(do, np.float64))
    assert relerr(dv2, dv) < 1e-12


def test_lrpe_finite_differences():
    B, H, N, d, e = 2, 2, 12, 3, 4
    q, k, v, do = (np.asarray(x, np.float64) for x in rand_inputs(B, H, N, d, e, seed=8))
    lam = np.array([0.95, 0.5])
    th = np.array([[0.3, 1.1, 2.0], [0.05, 0.7, 1.6]])

    def loss(q_, k_, v_, th_):
        return float(np.sum(orc.lrpe_fwd_quad(q_, k_, v_, lam, th_) * do))

    dq, dk, dv, dth = orc.lrpe_bwd_quad(q, k, v, do, lam, th)
    rng = np.random.default_rng(0)
    # inputs are carried in fp32 containers: perturb by values exactly representable there
    h = 2.0 ** -10
    for name, x, g in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        for _ in range(6):
            idx = tuple(rng.integers(0, n) for n in x.shape)
            xp, xm = x.copy(), x.copy()
            xp[idx] += h
            xm[idx] -= h
            args_p = {"q": (xp, k, v), "k": (q, xp, v), "v": (q, k, xp)}[name]
            args_m = {"q": (xm, k, v), "k": (q, xm, v), "v": (q, k, xm)}[name]
            fd = (loss(*args_p, th) - loss(*args_m, th)) / (2 * h)      # exact: the loss is linear in each of q, k, v
            assert abs(fd - g[idx]) < 1e-9 * (1 + abs(fd)), (name, idx)
    for hh in range(H):
        for i in range(d):
            tp, tm = th.copy(), th.copy()
            tp[hh, i] += 1e-5
            tm[hh, i] -= 1e-5
            fd = (loss(q, k, v, tp) - loss(q, k, v, tm)) / 2e-5
            assert abs(fd - dth[hh, i]) < 1e-6 * (1 + abs(fd)), (hh, i)


def test_lrpe_brute_force_loops():
    B, H, N, d, e = 1, 2, 7, 2, 2
    q, k, v, _ = (np.asarray(x, np.float64) for x in rand_inputs(B, H, N, d, e, seed=9))
    lam = [0.9, 0.3]
    th = [[0.4, 1.3], [2.2, 0.01]]
    o = np.zeros((B, H, N, e))
    for h in range(H):
        for t in range(N):
            for s in range(t + 1):
                a = 0.0
                for i in range(d):
                    a += q[0, h, t, i] * k[0, h, s, i] * np.cos(th[h][i] * (t - s))
                for j in range(e):
                    o[0, h, t, j] += lam[h] ** (t - s) * a * v[0, h, s, j]
    np.testing.assert_allclose(orc.lrpe_fwd_quad(q, k, v, np.array(lam), np.array(th)), o, rtol=0, atol=1e-13)
