"""Unit tests of the tensor-core contraction kernel in isolation (through the debug entry point of the
C ABI), against fp64 numpy matmuls of the same bf16 inputs.  Covers every operand form the layer uses:
K-major/K-major (forward), K-major/MN-major (input gradients), MN-major/MN-major (weight gradients),
dense and expert-grouped (row segments padded to 128), all epilogues."""
import numpy as np
import pytest
from scipy.special import erf

from paper_2502_16927_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _dev_bf16(a):
    import torch
    return torch.from_numpy(wl.to_bf16_bits(wl.bf16_round(a)).view(np.int16)).cuda().view(torch.bfloat16)


def _np(t):
    import torch
    return t.to(torch.float32).cpu().numpy().astype(np.float64)


def _layer():
    from paper_2502_16927_b200 import binding
    return binding.Layer(64, 64, 64, 8, 1, 16, 1, 1)


def _q(**kw):
    from paper_2502_16927_b200 import binding
    q = binding.bigmac_debug_gemm_t()
    for key, val in kw.items():
        if hasattr(val, "data_ptr"):
            val = val.data_ptr()
        setattr(q, key, val)
    return q


def _rand(shape, seed, scale=1.0):
    return wl.bf16_round((np.random.default_rng(seed).standard_normal(shape) * scale).astype(np.float32))


def _close(got, ref, out_bf16=True, abs_tol=0.0):
    """Elementwise: one rounding of the output dtype, relative to max(|ref|, rms(ref)), after `abs_tol` of absolute
    error (the stated bound of an approximation inside the kernel) has been taken off."""
    if ref.size == 0:
        return
    scale = np.sqrt(np.mean(ref ** 2)) + 1e-30
    tol = (2.0 ** -8 if out_bf16 else 1e-5)
    err = np.max(np.maximum(np.abs(got - ref) - abs_tol, 0.0) / np.maximum(np.abs(ref), scale))
    assert err <= tol * 1.01 + 1e-6, err


# The tensor-core epilogue evaluates Phi(z) by a saturating polynomial: |Phi error| <= 3.2e-5, |z Phi(z) error| <= 1.1e-4.
GELU_ABS_ERR = 1.1e-4


def _run(layer, q, tc=True):
    import torch
    from paper_2502_16927_b200 import binding
    binding.bigmac_debug_gemm(layer.handle, q, tc)
    torch.cuda.synchronize()
    assert layer.status() == 0


@pytest.mark.parametrize("M,N,K", [(128, 128, 64), (300, 192, 256), (1000, 64, 4096), (77, 320, 128), (333, 1024, 192),
                                   (20000, 2048, 64),
                                   # long contractions at least 512 wide
                                   (700, 512, 2048), (1300, 640, 2112), (520, 896, 4096), (300, 1100, 2048)])
def test_dense_kmajor_kmajor(M, N, K):
    import torch
    A, B = _rand((M, K), 1), _rand((N, K), 2, K ** -0.5)
    dA, dB = _dev_bf16(A), _dev_bf16(B)
    C = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    layer = _layer()
    _run(layer, _q(A=dA, B=dB, C=C, lda=K, ldb=K, ldc=N, M=M, N=N, K=K, a_kmajor=1, b_kmajor=1))
    _close(_np(C), A.astype(np.float64) @ B.astype(np.float64).T)


@pytest.mark.parametrize("M,N,K", [(1000, 1024, 192), (777, 320, 512), (300, 2048, 64), (500, 384, 256), (260, 400, 128)])
def test_pair_kernel_gives_the_same_bits_with_four_two_or_one_working_epilogue_warps(M, N, K):
    """Plain epilogues let two of the four epilogue warps of a lane quadrant do all its columns (the default) so that
    fewer warps compete with the MMA-issuing thread; who drains a column does not change its value.  N = 320, 384 and
    400 end in a partly filled column tile."""
    import torch
    A, B = _rand((M, K), 5), _rand((N, K), 6, K ** -0.5)
    dA, dB = _dev_bf16(A), _dev_bf16(B)
    layer = _layer()
    outs = []
    for mode in (3, 4, 5, 1):                      # 4, 2, 1 working warps per quadrant, then the default choice
        C = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        _run(layer, _q(A=dA, B=dB, C=C, lda=K, ldb=K, ldc=N, M=M, N=N, K=K, a_kmajor=1, b_kmajor=1), mode)
        outs.append(C)
    _close(_np(outs[0]), A.astype(np.float64) @ B.astype(np.float64).T)
    for other in outs[1:]:
        assert torch.equal(outs[0].view(torch.int16), other.view(torch.int16))


def test_gelu_epilogue_error_bound_over_a_sweep_of_z():
    """z = A I through the expert-GEMM1 epilogue for z across [-6, 6] and, in the last quarter of the rows, for
    magnitudes from 3 up to 1e38 of both signs (the polynomial's argument is not clamped: it has to saturate by itself,
    also where z^2 overflows): sigma(z) within one bf16 rounding plus the stated absolute bound of the Phi polynomial,
    sigma'(z) within half a quantisation step."""
    import torch
    M, N, K = 2048, 256, 256
    z = np.linspace(-6.0, 6.0, M * N).astype(np.float32)
    far = np.logspace(np.log10(3.0), 38.0, M * N // 4).astype(np.float32)
    far[1::2] *= -1.0
    z[-far.size:] = far
    z = wl.bf16_round(z.reshape(M, N))
    eye = np.eye(N, K, dtype=np.float32)
    C = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    Z = torch.zeros((M, N), dtype=torch.uint8, device="cuda")
    layer = _layer()
    _run(layer, _q(A=_dev_bf16(z), B=_dev_bf16(eye), C=C, Z=Z, lda=K, ldb=K, ldc=N, M=M, N=N, K=K, a_kmajor=1, b_kmajor=1,
                   epilogue=1, act=1))
    z64 = z.astype(np.float64)
    ref = _gelu(z64)
    assert np.all(np.abs(_np(C) - ref) <= 2.0 ** -8 * np.abs(ref) * 1.01 + GELU_ABS_ERR)
    got_z = (Z.cpu().numpy().astype(np.float64) - 27.0) / 200.0
    assert np.max(np.abs(got_z - _dgelu(z64))) <= 0.0026


@pytest.mark.parametrize("N", [32, 8, 5])
def test_dense_fp32_output_with_narrow_n(N):
    import torch
    M, K = 200, 1024
    A, B = _rand((M, K), 3), _rand((N, K), 4, K ** -0.5)
    C = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    layer = _layer()
    _run(layer, _q(A=_dev_bf16(A), B=_dev_bf16(B), C=C, lda=K, ldb=K, ldc=N, M=M, N=N, K=K, a_kmajor=1, b_kmajor=1,
                   out_f32=1))
    _close(_np(C), A.astype(np.float64) @ B.astype(np.float64).T, out_bf16=False)


@pytest.mark.parametrize("M,N,K", [(256, 128, 192), (130, 256, 64), (200, 192, 32), (900, 512, 2048), (270, 768, 2304)])
def test_dense_kmajor_mnmajor_with_accumulate(M, N, K):
    import torch
    A, Bt = _rand((M, K), 5), _rand((K, N), 6, K ** -0.5)       # B(n,k) = Bt[k,n]
    lda = max(K, 64)
    A_pad = np.zeros((M, lda), dtype=np.float32); A_pad[:, :K] = A
    C0 = _rand((M, N), 7)
    C = _dev_bf16(C0)
    layer = _layer()
    _run(layer, _q(A=_dev_bf16(A_pad), B=_dev_bf16(Bt), C=C, lda=lda, ldb=N, ldc=N, M=M, N=N, K=K, a_kmajor=1,
                   b_kmajor=0, accumulate=1))
    _close(_np(C), C0.astype(np.float64) + A.astype(np.float64) @ Bt.astype(np.float64))


@pytest.mark.parametrize("M,N,K", [(128, 128, 128), (192, 256, 1000), (40, 320, 300)])
def test_dense_mnmajor_mnmajor(M, N, K):
    import torch
    ldm = (M + 63) // 64 * 64
    At, Bt = _rand((K, M), 8), _rand((K, N), 9, K ** -0.5)       # A(m,k) = At[k,m]
    At_pad = np.zeros((K, ldm), dtype=np.float32); At_pad[:, :M] = At
    C = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    layer = _layer()
    _run(layer, _q(A=_dev_bf16(At_pad), B=_dev_bf16(Bt), C=C, lda=ldm, ldb=N, ldc=N, M=M, N=N, K=K, a_kmajor=0,
                   b_kmajor=0))
    _close(_np(C), At.astype(np.float64).T @ Bt.astype(np.float64))


def _segments(counts):
    """Padded layout tables for expert row counts."""
    pad = [(c + 127) // 128 * 128 for c in counts]
    poff = np.concatenate([[0], np.cumsum(pad)]).astype(np.int32)
    tile_expert = np.concatenate([np.full(p // 128, e, dtype=np.int32) for e, p in enumerate(pad)] + [np.zeros(0, np.int32)])
    return poff, tile_expert


def _gelu(z):
    return 0.5 * z * (1.0 + erf(z / np.sqrt(2.0)))


def _dgelu(z):
    return 0.5 * (1.0 + erf(z / np.sqrt(2.0))) + z * np.exp(-0.5 * z * z) / np.sqrt(2 * np.pi)


@pytest.mark.parametrize("N", [192, 1024])       # 1024: wide outputs leave through shared memory and TMA stores
def test_grouped_rows_forward_and_backward_epilogues(N):
    import torch
    counts = [130, 0, 5, 256, 1]
    E, K = len(counts), 128
    poff, tile_expert = _segments(counts)
    P = int(poff[-1]) + 256                                     # buffer larger than the live tiles
    A = np.zeros((P, K), dtype=np.float32)
    for e, c in enumerate(counts):
        A[poff[e]:poff[e] + c] = _rand((c, K), 20 + e)
    W = _rand((E, N, K), 11, K ** -0.5)                          # K-major weights [E,N,K]
    d_te = torch.from_numpy(np.concatenate([tile_expert, np.full(8, 99, np.int32)])).cuda()
    d_nt = torch.tensor([len(tile_expert)], dtype=torch.int32, device="cuda")
    d_po = torch.from_numpy(poff).cuda()
    C = torch.full((P, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    Z = torch.full((P, N), 255, dtype=torch.uint8, device="cuda")     # tensor-core path: sigma' as bytes, (q - 27) / 200
    layer = _layer()
    _run(layer, _q(A=_dev_bf16(A), B=_dev_bf16(W), C=C, Z=Z, lda=K, ldb=K, ldc=N, M=P, N=N, K=K, a_kmajor=1, b_kmajor=1,
                   epilogue=1, act=1, group=1, num_experts=E, b_stride=N * K, tile_expert=d_te, n_tiles=d_nt, poffsets=d_po))
    got_c, got_z = _np(C), (Z.cpu().numpy().astype(np.float64) - 27.0) / 200.0
    for e, c in enumerate(counts):
        rows = slice(poff[e], poff[e + 1])
        z = A[rows].astype(np.float64) @ W[e].astype(np.float64).T
        if z.size:
            assert np.max(np.abs(got_z[rows] - _dgelu(z))) <= 0.0026       # half a quantisation step (+ fp32 noise)
        _close(got_c[rows], _gelu(z), abs_tol=GELU_ABS_ERR)
    assert np.isnan(got_c[poff[-1]:]).all()                     # nothing beyond the live tiles is touched

    # input-gradient form: K-major A, MN-major per-expert weights, multiply by the saved sigma' bytes
    G = np.zeros((P, N), dtype=np.float32)                       # "du": [P, N] now the contraction side
    for e, c in enumerate(counts):
        G[poff[e]:poff[e] + c] = _rand((c, N), 40 + e)
    N2 = K if N == 192 else 1024                                 # output width
    Wt = _rand((E, N, N2), 12, N ** -0.5)                        # B(n2, k=n) = Wt[e][n, n2]
    q_in = np.random.default_rng(13).integers(0, 256, size=(P, N2)).astype(np.uint8)
    Zin = (q_in.astype(np.float64) - 27.0) / 200.0
    Zd = torch.from_numpy(q_in).cuda()
    Cd = torch.full((P, N2), float("nan"), dtype=torch.bfloat16, device="cuda")
    _run(layer, _q(A=_dev_bf16(G), B=_dev_bf16(Wt), C=Cd, Z=Zd, lda=N, ldb=N2, ldc=N2, M=P, N=N2, K=N, a_kmajor=1,
                   b_kmajor=0, epilogue=2, act=1, group=1, num_experts=E, b_stride=N * N2, tile_expert=d_te, n_tiles=d_nt, poffsets=d_po))
    got = _np(Cd)
    for e in range(E):
        rows = slice(poff[e], poff[e + 1])
        ref = (G[rows].astype(np.float64) @ Wt[e].astype(np.float64)) * Zin[rows].astype(np.float64)
        _close(got[rows], ref)


@pytest.mark.parametrize("accumulate", [0, 1])
def test_grouped_contraction_over_expert_rows(accumulate):
    import torch
    counts = [200, 0, 64, 1, 300]
    E, M, N = len(counts), 192, 128
    poff, _ = _segments(counts)
    P = int(poff[-1]) + 128
    rng = np.random.default_rng(5)
    At = rng.standard_normal((P, M)).astype(np.float32)         # rows beyond each segment's padding hold junk
    Bt = rng.standard_normal((P, N)).astype(np.float32)
    for e, c in enumerate(counts):                               # padding rows are zero by contract
        At[poff[e] + c:poff[e + 1]] = 0
        Bt[poff[e] + c:poff[e + 1]] = 0
    At, Bt = wl.bf16_round(At), wl.bf16_round(Bt)
    C0 = _rand((E, M, N), 6)
    C = _dev_bf16(C0)
    layer = _layer()
    _run(layer, _q(A=_dev_bf16(At), B=_dev_bf16(Bt), C=C, lda=M, ldb=N, ldc=N, M=M, N=N, K=P, a_kmajor=0, b_kmajor=0,
                   accumulate=accumulate, group=2, num_experts=E, c_stride=M * N,
                   poffsets=torch.from_numpy(poff).cuda()))
    got = _np(C)
    for e in range(E):
        rows = slice(poff[e], poff[e + 1])
        ref = At[rows].astype(np.float64).T @ Bt[rows].astype(np.float64) + accumulate * C0[e].astype(np.float64)
        if counts[e] == 0 and not accumulate:
            assert not got[e].any()
        else:
            _close(got[e], ref)
