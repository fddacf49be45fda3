"""Compression front-end on the device (Section 4.1 with S = I; Eq. 3, Eq. 6-8): rank-r factors of a dense weight
from the library's Jacobi SVD, against the oracle's fp64 Jacobi SVD and the Eckart-Young value.  Factor entries
are never compared (singular vectors are unique only up to sign and to rotations inside near-equal subspaces):
singular values, the product U V and MLP outputs are."""
import numpy as np
import pytest
import torch

from paper_2510_25977_b200 import binding, inputs

import _gpu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu_ready():
    _gpu.require_gpu()


@pytest.mark.parametrize("shape,r", [((688, 256), 32), ((256, 688), 32), ((300, 255), 40), ((96, 96), 96)])
def test_factors_against_the_oracle_svd(oracle, shape, r):
    g = torch.Generator().manual_seed(shape[0] * 1000 + shape[1])
    W = (torch.randn(shape, generator=g) * 0.02).float()
    U, V, sigma = binding.svdmlp_compress(W.cuda(), r)
    _, S_ref, _ = oracle.svd_jacobi(W.numpy().astype(np.float64))
    S = sigma.numpy().astype(np.float64)
    assert S.shape == S_ref.shape and np.all(np.diff(S) <= 1e-7)          # all of them, descending
    assert np.abs(S - S_ref).max() <= 2e-5 * S_ref[0]
    Wd = W.numpy().astype(np.float64)
    rec = oracle.reconstruct(U.cpu(), V.cpu())
    err = np.linalg.norm(rec - Wd)
    tail = np.sqrt((S_ref[r:] ** 2).sum())                                  # Eckart-Young: the best any rank-r product can do
    rounding = 2.0 ** -8 * np.sqrt((S_ref[:r] ** 2).sum())                  # bf16 storage of the two factors
    assert err >= tail * (1 - 1e-6) - 1e-12
    assert err <= np.sqrt(tail ** 2 + rounding ** 2) * 1.01 + 1e-9
    VV = V.double().cpu().numpy() @ V.double().cpu().numpy().T             # rows of V orthonormal (to bf16 precision)
    assert np.abs(VV - np.eye(r)).max() <= 2e-2


def test_sqrt_split_of_the_singular_values(oracle):
    g = torch.Generator().manual_seed(7)
    W = (torch.randn((320, 200), generator=g) * 0.05).float().cuda()
    U1, V1, s1 = binding.svdmlp_compress(W, 24)
    U2, V2, s2 = binding.svdmlp_compress(W, 24, flags=binding.COMPRESS_SPLIT_SQRT)
    assert torch.equal(s1, s2)
    r1, r2 = oracle.reconstruct(U1.cpu(), V1.cpu()), oracle.reconstruct(U2.cpu(), V2.cpu())
    assert np.abs(r1 - r2).max() <= 2e-2 * np.abs(r1).max()                # same product, different bf16 roundings
    un = U2.double().norm(dim=0).cpu().numpy()                             # Eq. 6: columns of U' carry sqrt(sigma)
    assert np.abs(un - np.sqrt(s2.numpy()[:24])).max() <= 1e-2 * un.max()
    vn = V2.double().norm(dim=1).cpu().numpy()                             # Eq. 7: so do the rows of V'
    assert np.abs(vn - np.sqrt(s2.numpy()[:24])).max() <= 1e-2 * vn.max()


def test_config1_from_dense_weights_on_the_device(oracle):
    """The tiny configuration end to end on the device: dense weights -> device SVD -> factors -> forward; compared
    with the oracle on the stored factors (parity) and with the oracle's own truncation of the same weights
    (the two rank-32 MLPs agree to the precision of the bf16 factors)."""
    d, ffn, r, T = 256, 688, 32, 16
    Wg, Wu, Wd = inputs.dense_weights(d, ffn, seed=0)
    fac = []
    for W in (Wg, Wu, Wd):
        U, V, _ = binding.svdmlp_compress(W.float().cuda().contiguous(), r)
        fac += [U, V]
    Ug, Vg, Uu, Vu, Ud, Vd = fac
    X = inputs.activations(T, d, seed=0, device="cuda")
    h = binding.svdmlp_create(Ug, Vg, Uu, Vu, Ud, Vd, max_T=T)
    Y = binding.svdmlp_forward(h, X)
    torch.cuda.synchronize()
    assert binding.svdmlp_last_device_status(h) == 0
    binding.svdmlp_destroy(h)
    _gpu.assert_close(Y, oracle.svdmlp(X, Ug, Vg, Uu, Vu, Ud, Vd), "forward on device-made factors")
    f = inputs.svd_factors(d, ffn, r, seed=0)                             # host LAPACK truncation of the same weights
    ref = oracle.svdmlp(X, *f.tensors())
    got = oracle.svdmlp(X, Ug, Vg, Uu, Vu, Ud, Vd)
    assert np.abs(got - ref).sum() <= 2e-2 * np.abs(ref).sum()


def test_argument_checks():
    L = binding.lib()
    assert L.svdmlp_compress_workspace_bytes(0, 8) == 0
    W = torch.zeros((64, 32), dtype=torch.float32, device="cuda")
    U = torch.empty((64, 8), dtype=torch.bfloat16, device="cuda")
    V = torch.empty((8, 32), dtype=torch.bfloat16, device="cuda")
    need = L.svdmlp_compress_workspace_bytes(64, 32)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    assert L.svdmlp_compress(W.data_ptr(), 64, 32, 40, U.data_ptr(), V.data_ptr(), None, ws.data_ptr(), need, 0, None) == -1   # r > min
    assert L.svdmlp_compress(W.data_ptr(), 64, 32, 8, U.data_ptr(), V.data_ptr(), None, ws.data_ptr(), need - 1, 0, None) == -6
    assert L.svdmlp_compress(W.data_ptr(), 64, 32, 8, U.data_ptr(), V.data_ptr(), None, ws.data_ptr(), need, 0, None) == 0     # zero matrix: sigma = 0, factors 0
    torch.cuda.synchronize()
    assert bool((U == 0).all()) and bool((V.float().abs() <= 1).all())
