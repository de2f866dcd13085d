"""Pins of the DPQ quantizer oracle (Algorithm 1, Eq. 6-12, Sec. 3.2-3.3) against what the paper
and the mathematics fix: a hand-worked example, the reduction to round-to-nearest when the Hessian
is the identity, the elimination identity W - W^ = E U, the drop of the layer-output error it
exists for, and the structure Group-Aware Reordering must keep."""
import os

import numpy as np
import pytest

import oracle
from helpers import e4m3_value_table, unpack_codes

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "dpq_tiny.txt")


def _golden():
    out = {}
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, *v = line.split()
        out[k] = np.array([float(x) for x in v])
    return out


def _dequant16(codes, gscale, gzero, s_w, group):
    """The BF16-domain weights inference sees: Eq. 10 (rounded to E4M3) then Eq. 11."""
    w8 = oracle.dequant_weight(codes, gscale, gzero, group)
    vals = e4m3_value_table()[w8]
    sw = s_w.astype(np.float64)
    return vals * (sw[:, None] if sw.size > 1 else sw[0])


def _case(N, K, seed, tokens=512, hot_every=7, hot=6.0):
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    X = rng.standard_normal((tokens, K))
    X[:, ::hot_every] *= hot                    # a few input features that matter much more
    X += 0.5 * rng.standard_normal((tokens, 1))  # and a common component: correlated features
    return W, X


def test_hand_worked_example():
    g = _golden()
    W = g["W"].astype(np.float32)[None, :]
    U = g["U"].astype(np.float32).reshape(2, 2)
    codes, gs, gz, s_w, err, what = oracle.dpq_quantize(W, U, group=2, symmetric=False, debug=True)
    assert list(unpack_codes(codes)[0]) == list(g["codes"].astype(int))
    scale = (gs.astype(np.uint32) << 16).view(np.float32)[0, 0]
    assert scale == np.float32(g["gscale"][0])
    assert gz[0, 0] == int(g["gzero"][0])
    assert np.allclose(err[0], g["err"], rtol=0, atol=2e-8)
    assert np.allclose(what[0], g["what"], rtol=0, atol=1e-8)
    rtn = oracle.quantize_weight_rtn(W, group=2, symmetric=False)
    assert list(unpack_codes(rtn[0])[0]) == list(g["rtn_codes"].astype(int))


@pytest.mark.parametrize("symmetric", [True, False])
@pytest.mark.parametrize("per_channel", [False, True])
def test_identity_hessian_reduces_to_round_to_nearest(symmetric, per_channel):
    # with H = I nothing is propagated (U = I): Algorithm 1 is Eq. 6 -> 7 -> 8 -> 9 per weight
    W, _ = _case(24, 384, 1)
    a = oracle.dpq_quantize(W, np.eye(384, dtype=np.float32), symmetric=symmetric, per_channel=per_channel)
    b = oracle.quantize_weight_rtn(W, symmetric=symmetric, per_channel=per_channel)
    for x, y in zip(a, b):
        assert (x is None and y is None) or np.array_equal(x, y)


@pytest.mark.parametrize("symmetric,mse_steps,use_gar", [(False, 0, False), (False, 6, True), (True, 11, True)])
def test_elimination_identity(symmetric, mse_steps, use_gar):
    # every weight ends as w - sum_{p<q} e_p U_pq and is replaced by that minus e_q U_qq: W - W^ = E U
    W, X = _case(16, 256, 2)
    H = X.T @ X
    perm = oracle.gar_permutation(np.diag(H)) if use_gar else None
    U = oracle.hessian_upper_cholesky(H, perm)
    codes, gs, gz, s_w, err, what = oracle.dpq_quantize(W, U, perm, symmetric=symmetric, mse_steps=mse_steps,
                                                        debug=True)
    Wp = (W if perm is None else W[:, perm]).astype(np.float64)
    resid = Wp - what - err.astype(np.float64) @ np.triu(U.astype(np.float64))
    assert np.abs(resid).max() < 1e-6 * np.abs(Wp).max()
    # and `what` is what the stored format dequantizes to (Eq. 10, Eq. 11), back in the original order
    w16 = _dequant16(codes, gs, gz, s_w, 128)
    back = np.empty_like(what)
    if perm is None:
        back = what
    else:
        back[:, perm] = what
    assert np.allclose(w16, back, rtol=1e-6, atol=0)


@pytest.mark.parametrize("symmetric", [True, False])
def test_error_compensation_lowers_the_layer_output_error(symmetric):
    # the objective of Eq. 5: || W X - W^ X ||^2 on the calibration inputs, against round-to-nearest
    ratios = []
    for seed in range(4):
        W, X = _case(32, 256, 10 + seed)
        H = X.T @ X
        rtn = oracle.quantize_weight_rtn(W, symmetric=symmetric)
        e_rtn = np.linalg.norm((W - _dequant16(*rtn, 128)) @ X.T) ** 2
        plain = oracle.dpq_quantize(W, oracle.hessian_upper_cholesky(H), symmetric=symmetric)
        e_plain = np.linalg.norm((W - _dequant16(*plain, 128)) @ X.T) ** 2
        perm = oracle.gar_permutation(np.diag(H))
        gar = oracle.dpq_quantize(W, oracle.hessian_upper_cholesky(H, perm), perm, symmetric=symmetric, mse_steps=6)
        e_gar = np.linalg.norm((W - _dequant16(*gar, 128)) @ X.T) ** 2
        assert e_plain < 0.8 * e_rtn
        ratios.append(e_gar / e_plain)
    assert np.mean(ratios) < 1.05   # reordering with the scale search does not hurt on average


def test_scale_search_never_raises_the_group_error():
    # with H = I the groups are independent: the searched scale's squared error on the FP8 weights
    # is at most that of the plain Eq. 8 scale, group by group
    W, _ = _case(16, 512, 3)
    U = np.eye(512, dtype=np.float32)
    tab = e4m3_value_table()
    errs = []
    for steps in (0, 11):
        codes, gs, gz, s_w = oracle.dpq_quantize(W, U, symmetric=False, mse_steps=steps)
        w8 = tab[oracle.e4m3_encode_array(W / s_w[0])]
        w8hat = tab[oracle.dequant_weight(codes, gs, gz)]
        errs.append(((w8 - w8hat) ** 2).reshape(16, 4, 128).sum(axis=2))
    assert np.all(errs[1] <= errs[0])
    assert np.any(errs[1] < errs[0])


def test_group_aware_reordering_structure():
    # hand example, group = 2: diag = [1,5 | 9,2 | 3,3] -> inside groups [1,0] [2,3] [4,5];
    # group maxima 5, 9, 3 -> groups in order 1, 0, 2
    perm = oracle.gar_permutation(np.array([1.0, 5.0, 9.0, 2.0, 3.0, 3.0]), group=2)
    assert list(perm) == [2, 3, 1, 0, 4, 5]
    rng = np.random.default_rng(5)
    d = rng.random(1024)
    perm = oracle.gar_permutation(d, 128)
    assert sorted(perm) == list(range(1024))
    blocks = perm.reshape(8, 128)
    assert np.all(blocks // 128 == (blocks[:, :1] // 128))          # whole groups move
    assert np.all(np.diff(d[blocks], axis=1) <= 0)                  # descending inside a group
    assert np.all(np.diff(d[blocks].max(axis=1)) <= 0)              # groups by descending maximum


def test_rejects_an_order_that_splits_groups():
    W, _ = _case(2, 256, 4)
    perm = np.arange(256, dtype=np.int32)
    perm[[0, 200]] = perm[[200, 0]]
    with pytest.raises(ValueError):
        oracle.dpq_quantize(W, np.eye(256, dtype=np.float32), perm)


def _damped_permuted(H, perm, damp):
    """The matrix Sec. 3.3 inverts, built here entry by entry (not with the oracle's indexing)."""
    K = H.shape[0]
    order = list(range(K)) if perm is None else [int(v) for v in perm]
    Hp = np.empty((K, K), dtype=np.float64)
    for a in range(K):
        for b in range(K):
            Hp[a, b] = H[order[a], order[b]]
    for a in range(K):
        if Hp[a, a] == 0.0:
            Hp[a, a] = 1.0
    mean_diag = sum(Hp[a, a] for a in range(K)) / K
    for a in range(K):
        Hp[a, a] += damp * mean_diag
    return Hp


@pytest.mark.parametrize("use_perm,damp", [(False, 0.01), (True, 0.01), (True, 0.1)])
def test_hessian_factor_inverts_the_dampened_permuted_hessian(use_perm, damp):
    # U is upper triangular with a positive diagonal and U^T U is the inverse of the dampened
    # Hessian in processing order: (U^T U) (H_perm + damp * mean(diag) * I) = I.  An asymmetric H
    # ordering (rows permuted but not columns), a missing or doubled dampening, a lower factor or a
    # factor of H instead of its inverse all fail one of the asserts.
    rng = np.random.default_rng(5)
    K = 96
    X = rng.standard_normal((200, K)) * np.linspace(0.2, 3.0, K)   # distinct column energies
    X[:, 7] = 0.0                                                  # a dead input feature
    X[:, 40] = 0.0
    H = X.T @ X
    perm = rng.permutation(K).astype(np.int32) if use_perm else None
    U = oracle.hessian_upper_cholesky(H, perm, damp=damp)
    assert U.dtype == np.float32 and U.shape == (K, K)
    assert np.array_equal(U, np.triu(U)) and (np.diag(U) > 0).all()
    Hp = _damped_permuted(H, perm, damp)
    U64 = U.astype(np.float64)
    resid = U64.T @ U64 @ Hp - np.eye(K)
    # U is stored in float32: 2^-24 relative per entry, amplified by the condition number (< 1e4 here)
    assert np.abs(resid).max() < 2e-3
    # the same identity without the amplification: R = U^-1 is upper triangular and R R^T = Hp
    R = np.linalg.inv(U64)                      # upper triangular
    assert np.abs(np.tril(R, -1)).max() < 1e-12
    assert np.abs(R @ R.T - Hp).max() < 2e-6 * np.abs(Hp).max()
    # (Hp carries the dead-column rule -- unit diagonal before the dampening, wherever the
    # permutation put the column -- so a factor computed without it fails the identity above)


def test_hessian_factor_of_a_diagonal_hessian_in_closed_form():
    # H = diag(d): the dampened matrix is diag(d + damp * mean(d)), its inverse factor is
    # diag(1 / sqrt(d + damp * mean(d))), permuted like the columns.
    d = np.array([4.0, 1.0, 9.0, 16.0, 25.0, 0.25])
    perm = np.array([2, 0, 5, 1, 4, 3], dtype=np.int32)
    U = oracle.hessian_upper_cholesky(np.diag(d), perm, damp=0.05)
    want = 1.0 / np.sqrt(d[perm] + 0.05 * d.mean())
    assert np.allclose(np.diag(U), want, rtol=1e-6, atol=0)
    assert np.array_equal(U, np.diag(np.diag(U)))


def test_hessian_is_the_sum_of_outer_products_and_prepare_follows_its_three_rules():
    # oracle.hessian: X^T X written out as a sum of outer products of the token rows (no matmul), its
    # diagonal the column sums of squares; a one-hot X gives a diagonal count matrix.  oracle.hessian_prepare
    # against the three rules applied entry by entry: permutation of rows AND columns, unit diagonal for dead
    # columns, damp * mean(diag) on the diagonal.
    rng = np.random.default_rng(12)
    T, K = 37, 24
    X = (rng.standard_normal((T, K)) * 3).astype(np.float32)
    X[:, 5] = 0.0
    xb = oracle.f32_to_bf16(X)
    Xr = oracle.bf16_to_f32(xb).astype(np.float64)
    H = oracle.hessian(xb)
    want = np.zeros((K, K))
    for t in range(T):
        want += np.outer(Xr[t], Xr[t])
    assert np.allclose(H, want, rtol=1e-13, atol=1e-12)
    assert np.allclose(np.diag(H), (Xr ** 2).sum(axis=0), rtol=1e-13)
    onehot = np.zeros((10, 4), dtype=np.float32)
    onehot[np.arange(10), [0, 1, 1, 3, 3, 3, 0, 1, 3, 3]] = 1.0
    assert np.array_equal(oracle.hessian(oracle.f32_to_bf16(onehot)), np.diag([2.0, 3.0, 0.0, 5.0]))
    perm = rng.permutation(K).astype(np.int32)
    Hp = oracle.hessian_prepare(H, perm, damp=0.05)
    dd = np.array([H[perm[a], perm[a]] if H[perm[a], perm[a]] != 0 else 1.0 for a in range(K)])
    for a in range(K):
        for b in range(K):
            v = H[perm[a], perm[b]]
            if a == b:
                v = dd[a] + 0.05 * dd.mean()
            assert Hp[a, b] == pytest.approx(v, rel=1e-14, abs=1e-300)
