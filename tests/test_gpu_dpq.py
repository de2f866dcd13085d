"""GPU parity: w4a8_gar_permutation and w4a8_dpq_quantize against the oracle (Algorithm 1,
Eq. 6-12; Sec. 3.2-3.3).  Integer work: the permutation, the INT4 codes, the BF16 group scales,
the zero-points and the FP32 weight scale must be bit-exact.  Both sides get the same Cholesky
factor U (a library factorization is an input of the method, not part of it) and take every
rounding decision in fp32, one operation at a time."""
import numpy as np
import pytest
import torch

import oracle
from gpu_utils import bf16_bits, dev, hessian_upper_cholesky_dev
from paper_2505_14638_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _hessian(K, seed, tokens=384):
    xb = inputs.make_activation(tokens, K, seed, 0.01, 20.0)          # BF16 N(0,1) with outlier channels
    X = inputs.bf16_bits_to_f32(xb).astype(np.float64)
    rng = np.random.default_rng(seed)
    X += 0.5 * rng.standard_normal((tokens, 1))                        # correlated input features
    return X.T @ X


def _compare(W, U, perm, **kw):
    ref = oracle.dpq_quantize(W, U, perm, **kw)
    got = binding.dpq_quantize(dev(W), dev(U), None if perm is None else dev(perm), **kw)
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    codes, gscale, gzero, s_w = got
    assert np.array_equal(s_w.cpu().numpy().view(np.uint32), ref[3].view(np.uint32))
    assert np.array_equal(bf16_bits(gscale), ref[1])
    if ref[2] is None:
        assert gzero is None
    else:
        assert np.array_equal(gzero.cpu().numpy(), ref[2])
    assert np.array_equal(codes.cpu().numpy(), ref[0])


@pytest.mark.parametrize("K", [128, 1024, 4096])
def test_gar_permutation_matches(K):
    rng = np.random.default_rng(K)
    d = rng.random(K).astype(np.float32)
    d[rng.choice(K, K // 16, replace=False)] = d[0]      # ties
    d[5] = 0.0
    perm = binding.gar_permutation(dev(d))
    torch.cuda.synchronize()
    assert np.array_equal(perm.cpu().numpy(), oracle.gar_permutation(d))


@pytest.mark.parametrize("N,K", [(8, 128), (24, 384), (100, 1024), (37, 256), (1, 128)])
@pytest.mark.parametrize("symmetric", [False, True])
def test_dpq_matches_oracle_in_original_order(N, K, symmetric):
    W = inputs.make_weight(N, K, 0.02, seed=N + K)
    U = oracle.hessian_upper_cholesky(_hessian(K, N))
    _compare(W, U, None, symmetric=symmetric)
    _compare(W, U, None, symmetric=symmetric, per_channel=True)


@pytest.mark.parametrize("mse_steps", [0, 6, 11])
def test_dpq_with_reordering_and_scale_search(mse_steps):
    N, K = 64, 1024
    W = inputs.make_weight(N, K, 0.02, seed=77)
    H = _hessian(K, 78)
    perm = oracle.gar_permutation(np.diag(H))
    U = oracle.hessian_upper_cholesky(H, perm)
    _compare(W, U, perm, symmetric=False, mse_steps=mse_steps)
    _compare(W, U, perm, symmetric=True, mse_steps=mse_steps)


def test_dpq_identity_factor_is_round_to_nearest():
    N, K = 40, 512
    W = inputs.make_weight(N, K, 0.02, seed=5)
    Wd = dev(W)
    a = binding.dpq_quantize(Wd, torch.eye(K, dtype=torch.float32, device="cuda"))
    b = binding.quantize_weight_rtn(Wd, symmetric=False)
    torch.cuda.synchronize()
    for x, y in zip(a, b):
        assert torch.equal(x.view(torch.uint8) if x.dtype != torch.float32 else x.view(torch.int32),
                           y.view(torch.uint8) if y.dtype != torch.float32 else y.view(torch.int32))


def test_dpq_layer_size_and_the_device_side_factorization():
    # a Llama-sized layer slice: N = 512 rows of the K = 4096 o-projection; the codes must match the
    # oracle when both get the SAME factor (here one computed on the device by the caller's library routines) ...
    N, K = 512, 4096
    W = inputs.make_weight(N, K, 0.02, seed=9)
    H = _hessian(K, 10, tokens=1024)
    Hd = dev(H.astype(np.float64))
    perm = binding.gar_permutation(torch.diagonal(Hd).to(torch.float32).contiguous())
    U = hessian_upper_cholesky_dev(Hd, perm)
    torch.cuda.synchronize()
    assert np.array_equal(perm.cpu().numpy(), oracle.gar_permutation(np.diag(H).astype(np.float32)))
    _compare(W, U.cpu().numpy(), perm.cpu().numpy(), symmetric=False, mse_steps=6)
    # ... and the quantized layer must beat round-to-nearest on the objective of Eq. 5
    codes, gscale, gzero, s_w = binding.dpq_quantize(dev(W), U, perm, symmetric=False, mse_steps=6)
    rtn = binding.quantize_weight_rtn(dev(W), symmetric=False)
    torch.cuda.synchronize()

    def out_err(q):
        c, gs, gz, sw = q
        w8 = binding.dequant_weight(c, gs, gz)
        w16 = w8.view(torch.float8_e4m3fn).to(torch.float64) * sw.to(torch.float64)
        D = torch.from_numpy(W).cuda().to(torch.float64) - w16
        return float(torch.einsum("nk,kj,nj->", D, Hd, D))    # || (W - W^) X^T ||^2 = tr(D H D^T)
    assert out_err((codes, gscale, gzero, s_w)) < 0.8 * out_err(rtn)


@pytest.mark.parametrize("T,K", [(100, 128), (384, 640), (1000, 1096)])
def test_hessian_accumulate_and_prepare_match_oracle(T, K):
    # w4a8_hessian_accumulate: FP32 sums over T products per entry against the oracle's float64 X^T X
    # (tolerance: T rounding errors of 2^-24 relative to the entry's sum of magnitudes, bounded by
    # sqrt(H_ii H_jj)); two batches accumulated = one pass; the matrix is exactly symmetric.
    # w4a8_hessian_prepare: permutation, dead-feature rule, dampening -- against the oracle's.
    rng = np.random.default_rng(T + K)
    X = rng.standard_normal((T, K)).astype(np.float32) * np.linspace(0.1, 4.0, K, dtype=np.float32)
    X[:, 3] = 0.0
    X[:, K - 1] = 0.0
    xb = oracle.f32_to_bf16(X)
    xd = torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16).cuda()
    H = binding.hessian_accumulate(xd)
    half = T // 2
    H2 = binding.hessian_accumulate(xd[:half].contiguous())
    H2 = binding.hessian_accumulate(xd[half:].contiguous(), H2)
    torch.cuda.synchronize()
    ref = oracle.hessian(xb)
    got = H.cpu().numpy().astype(np.float64)
    assert np.array_equal(H.cpu().numpy(), H.cpu().numpy().T)
    bound = np.sqrt(np.outer(np.diag(ref), np.diag(ref)))
    assert np.all(np.abs(got - ref) <= 4.0 * T * 2.0 ** -24 * bound + 1e-30)
    assert np.all(np.abs(H2.cpu().numpy().astype(np.float64) - ref) <= 4.0 * T * 2.0 ** -24 * bound + 1e-30)
    assert np.all(got[3] == 0) and np.all(got[:, K - 1] == 0)
    perm = rng.permutation(K).astype(np.int32)
    for pm in (None, perm):
        Hp = binding.hessian_prepare(H, None if pm is None else torch.from_numpy(pm).cuda(), damp=0.02)
        torch.cuda.synchronize()
        want = oracle.hessian_prepare(H.cpu().numpy(), pm, damp=0.02)
        assert np.allclose(Hp.cpu().numpy().astype(np.float64), want, rtol=3e-7, atol=0)


def test_quantizer_pipeline_from_activations_through_the_c_abi():
    # X -> H (w4a8_hessian_accumulate) -> order (w4a8_gar_permutation) -> prepared Hessian
    # (w4a8_hessian_prepare) -> [library: inverse and Cholesky factor] -> w4a8_dpq_quantize: the stored
    # layer must beat round-to-nearest on the layer's output error by the margin the oracle's
    # quantizer shows on such inputs (>= 20 %).
    N, K, T = 256, 512, 1024
    rng = np.random.default_rng(5)
    mix = rng.standard_normal((K, K)).astype(np.float32) * 0.2 + np.eye(K, dtype=np.float32)
    X = (rng.standard_normal((T, K)).astype(np.float32) @ mix) * np.linspace(0.3, 3.0, K, dtype=np.float32)
    xb = oracle.f32_to_bf16(X)
    xd = torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16).cuda()
    W = torch.from_numpy(inputs.make_weight(N, K, 0.02, 6)).cuda()
    H = binding.hessian_accumulate(xd)
    perm = binding.gar_permutation(H.diagonal().contiguous())
    Hp = binding.hessian_prepare(H, perm, damp=0.01).to(torch.float64)
    Hinv = torch.cholesky_inverse(torch.linalg.cholesky(Hp))
    U = torch.linalg.cholesky(0.5 * (Hinv + Hinv.T), upper=True).to(torch.float32).contiguous()
    cq = binding.dpq_quantize(W, U, perm, symmetric=True, mse_steps=6)
    rq = binding.quantize_weight_rtn(W, symmetric=True)
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0

    def out_err(q):
        w8 = binding.dequant_weight(q[0], q[1], q[2]).view(torch.float8_e4m3fn).float() * q[3]
        D = (W - w8).double()
        return float(torch.einsum("nk,kj,nj->", D, H.double(), D))
    assert out_err(cq) <= 0.8 * out_err(rq)
