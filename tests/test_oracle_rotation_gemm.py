"""Pins for the oracle's rotation (Algorithm 3 steps 1-3), block-scaled GEMM (step 5) and
the offline weight fusion, against special cases with textbook answers, brute force in
pure Python, and the invariants the paper states (orthogonal transforms conserve the
total variance summed over blocks; the rotate / inverse-rotate chain is the identity in
full precision)."""
import numpy as np
import pytest

import oracle as O
from paper_2605_19561_b200 import inputs as I


def _bits(a):
    return I.to_bf16_bits(np.asarray(a, dtype=np.float32))


def _rand_bf16(shape, seed):
    g = np.random.default_rng(seed)
    return _bits(g.standard_normal(shape))


def test_identity_rotation_is_a_decode():
    xb = _rand_bf16((5, 64), 0)
    z = O.rotate(xb, None, None)
    assert (z == O.decode_bf16(xb)).all()
    eye = _bits(np.eye(64))
    eyes = _bits(np.stack([np.eye(32)] * 2))
    assert (O.rotate(xb, eye, eyes) == O.decode_bf16(xb)).all()


def test_permutations_pin_orientation_and_block_indexing():
    d = 96
    g = np.random.default_rng(5)
    xb = _rand_bf16((4, d), 1)
    x = O.decode_bf16(xb)
    perm = g.permutation(d)                       # P[i, perm[i]] = 1  ->  y[:, perm[i]] = x[:, i]
    P = np.zeros((d, d)); P[np.arange(d), perm] = 1
    y = O.rotate(xb, _bits(P), None)
    want = np.empty_like(x); want[:, perm] = x
    assert (y == want).all()
    # intra: a different permutation in each block, applied after the inter step
    q = np.stack([g.permutation(32) for _ in range(d // 32)])
    Q = np.zeros((d // 32, 32, 32))
    for b in range(d // 32):
        Q[b, np.arange(32), q[b]] = 1
    z = O.rotate(xb, _bits(P), _bits(Q))
    want2 = np.empty_like(want)
    for b in range(d // 32):
        want2[:, 32 * b + q[b]] = want[:, 32 * b:32 * b + 32]
    assert (z == want2).all()


def _fwht(v):
    """Textbook in-place fast Walsh-Hadamard transform (natural order), pure Python."""
    v = list(v)
    h = 1
    while h < len(v):
        for i in range(0, len(v), 2 * h):
            for j in range(i, i + h):
                a, b = v[j], v[j + h]
                v[j], v[j + h] = a + b, a - b
        h *= 2
    return v


def _hadamard(n):
    H = np.array([[1.0]])
    while H.shape[0] < n:
        H = np.block([[H, H], [H, -H]])
    return H


def test_walsh_hadamard_inter_rotation_and_energy():
    d = 256
    H = _hadamard(d) / 16.0                       # entries +-2^-4: exact in bfloat16, exactly orthogonal
    xb = _rand_bf16((6, d), 2)
    x = O.decode_bf16(xb)
    y = O.rotate(xb, _bits(H), None)
    for m in range(6):
        ref = np.array(_fwht(x[m])) / 16.0
        assert np.allclose(y[m], ref, rtol=0, atol=1e-13 * np.abs(x[m]).sum())
    # total variance over blocks is conserved by an orthogonal transform (Appendix A.1, step 1)
    eb_x = (x.reshape(6, 8, 32) ** 2).sum(-1)
    eb_y = (y.reshape(6, 8, 32) ** 2).sum(-1)
    assert np.allclose(eb_x.sum(1), eb_y.sum(1), rtol=1e-12)
    assert not np.allclose(eb_x, eb_y)            # energy really moved between blocks
    # intra rotation by H32/sqrt(32)... not exact in bf16; use H32 * 2^-2 * (exactly orthogonal up to factor 2)
    H32 = _hadamard(32) / 4.0                     # = sqrt(2) * orthogonal; energy doubles exactly
    z = O.rotate(xb, _bits(H), _bits(np.stack([H32] * 8)))
    eb_z = (z.reshape(6, 8, 32) ** 2).sum(-1)
    assert np.allclose(eb_z, 2.0 * eb_y, rtol=1e-12)   # intra step never moves energy across blocks


def test_rotation_against_pure_python_loops():
    M, d = 3, 64
    xb, rb, rib = _rand_bf16((M, d), 3), _rand_bf16((d, d), 4), _rand_bf16((2, 32, 32), 5)
    x, r, ri = O.decode_bf16(xb), O.decode_bf16(rb), O.decode_bf16(rib)
    z = O.rotate(xb, rb, rib)
    for m in range(M):
        y = [sum(x[m, i] * r[i, j] for i in range(d)) for j in range(d)]
        for b in range(2):
            for j in range(32):
                ref = sum(y[32 * b + i] * ri[b, i, j] for i in range(32))
                assert abs(z[m, 32 * b + j] - ref) <= 1e-12 * (1 + abs(ref))


def test_generated_rotations_are_orthogonal_and_conserve_energy():
    cfg = I.CONFIGS["tiny"]
    rb, rib, r64, ri64 = I.rotations(cfg)
    assert np.abs(r64.T @ r64 - np.eye(cfg.d)).max() < 1e-12
    for b in range(cfg.d // 32):
        assert np.abs(ri64[b].T @ ri64[b] - np.eye(32)).max() < 1e-12
    xb = I.activations(cfg)
    x = O.decode_bf16(xb)
    z = O.rotate(xb, rb, rib)
    # bfloat16-rounded rotations are orthogonal to ~2^-9: energy conserved to that order
    ex, ez = (x ** 2).sum(1), (z ** 2).sum(1)
    assert np.abs(ez / ex - 1).max() < 2e-2
    rt = O.merged_rotation(rb, rib)
    assert np.abs(rt.T @ rt - np.eye(cfg.d)).max() < 2e-2
    # merged operator equals the two-step application
    assert np.allclose(x @ rt, z, rtol=1e-12, atol=1e-12 * np.abs(x).max())


def test_unquantized_chain_is_identity_with_exact_rotations():
    d, N = 256, 40
    H = _hadamard(d) / 16.0
    g = np.random.default_rng(6)
    P = np.zeros((8, 32, 32))
    for b in range(8):
        P[b, np.arange(32), g.permutation(32)] = 1
    xb = _rand_bf16((7, d), 7)
    w = g.standard_normal((d, N))
    z = O.rotate(xb, _bits(H), _bits(P))
    rt = O.merged_rotation(_bits(H), _bits(P))
    ref = O.decode_bf16(xb) @ w
    assert np.allclose(z @ (rt.T @ w), ref, rtol=1e-12, atol=1e-12 * np.abs(ref).max())


def test_prepare_weights_is_transposed_fused_and_quantized_along_k():
    cfg = I.CONFIGS["tiny"]
    rb, rib, _, _ = I.rotations(cfg)
    w = I.weights(cfg, N=48)
    codes, sb = O.prepare_weights(rb, rib, w)
    assert codes.shape == (48, cfg.d) and sb.shape == (48, cfg.d // 32)
    rt = O.merged_rotation(rb, rib)
    wp = (rt.T @ w.astype(np.float64)).T
    deq = O.dequantize(codes, sb)
    # MXFP4 keeps about 2-3 significant bits: relative Frobenius error well under 20 %
    assert np.linalg.norm(deq - wp) / np.linalg.norm(wp) < 0.2
    # and a quantized end-to-end layer approximates the float layer
    xb = I.activations(cfg)
    out, _, _ = O.rotated_linear(xb, rb, rib, codes, sb)
    ref = O.decode_bf16(xb) @ w.astype(np.float64)
    assert np.linalg.norm(out - ref) / np.linalg.norm(ref) < 0.3


def _rand_q(rows, k, seed):
    g = np.random.default_rng(seed)
    return g.integers(0, 16, size=(rows, k), dtype=np.uint8), g.integers(118, 134, size=(rows, k // 32), dtype=np.uint8)


def test_gemm_against_pure_python_loops():
    M, N, K = 3, 4, 64
    ac, asb = _rand_q(M, K, 8)
    wc, wsb = _rand_q(N, K, 9)
    out = O.gemm_dequant(ac, asb, wc, wsb)
    val = [0, .5, 1, 1.5, 2, 3, 4, 6]
    def deq(c, s):
        return (-1 if c & 8 else 1) * val[c & 7] * 2.0 ** (int(s) - 127)
    for m in range(M):
        for n in range(N):
            ref = sum(deq(ac[m, k], asb[m, k // 32]) * deq(wc[n, k], wsb[n, k // 32]) for k in range(K))
            assert out[m, n] == ref                 # everything is exact in float64 here


def test_gemm_one_hot_and_power_of_two_sums():
    M, N, K = 4, 5, 128
    wc, wsb = _rand_q(N, K, 10)
    ac = np.zeros((M, K), np.uint8); asb = np.full((M, K // 32), 127, np.uint8)
    hot = [3, 40, 77, 127]
    for m, k in enumerate(hot):
        ac[m, k] = 2                                # the value 1.0
    out = O.gemm_dequant(ac, asb, wc, wsb)
    wd = O.dequantize(wc, wsb)
    for m, k in enumerate(hot):
        assert (out[m] == wd[:, k]).all()           # selects column k of W^ (orientation: out = A W^T)
    # all elements 1.0, scales vary per block: out = 32 * sum_b 2^(ea_b + ew_b)
    ac[:] = 2; wc[:] = 2
    g = np.random.default_rng(11)
    asb = g.integers(120, 130, size=(M, K // 32), dtype=np.uint8)
    wsb = g.integers(120, 130, size=(N, K // 32), dtype=np.uint8)
    out = O.gemm_dequant(ac, asb, wc, wsb)
    for m in range(M):
        for n in range(N):
            assert out[m, n] == 32.0 * sum(2.0 ** (int(asb[m, b]) + int(wsb[n, b]) - 254) for b in range(K // 32))


def test_round_to_bf16_matches_library_cast():
    g = np.random.default_rng(12)
    y = g.standard_normal(5000) * np.exp(g.normal(0, 4, 5000))
    y32 = y.astype(np.float32).astype(np.float64)   # avoid double-rounding differences: start on the f32 grid
    lib = O.decode_bf16(I.to_bf16_bits(y32))
    assert (O.round_to_bf16(y32) == lib).all()
    assert O.round_to_bf16(np.array([1.00390625]))[0] == 1.0        # 1 + 2^-8: tie -> even
    assert O.round_to_bf16(np.array([1.01171875]))[0] == 1.015625   # 1 + 3*2^-8: tie -> even (up)


# ------------------------------------------------------------------ structured rotation (paper's form)
def _structured_case(M, nb, seed):
    g = np.random.default_rng(seed)
    xb = I.to_bf16_bits(g.standard_t(3.0, size=(M, nb * 32)))
    rb = I.to_bf16_bits(I.orthogonal(nb, g))
    ri = I.to_bf16_bits(I.orthogonal(32, g))
    return xb, rb, ri


def test_structured_rotation_equals_the_dense_one_with_kronecker_operands():
    """R_B acting across blocks is the dense inter rotation kron(R_B^T, I_32) in the row-vector
    convention, and one shared R_intra is the same matrix in every block: the two oracle
    functions must agree to summation-order rounding."""
    for M, nb in [(5, 4), (3, 8), (7, 16)]:
        xb, rb, ri = _structured_case(M, nb, seed=nb)
        z = O.rotate_structured(xb, rb, ri)
        RB, RI = O.decode_bf16(rb), O.decode_bf16(ri)
        dense = np.kron(RB.T, np.eye(32))                 # [32b+k, 32b'+k'] = R_B[b', b] delta(k, k')
        # the dense oracle takes bf16 bit patterns; every entry of `dense` is an entry of R_B or 0
        zd = O.rotate(xb, I.to_bf16_bits(dense), I.to_bf16_bits(np.stack([RI] * nb)))
        np.testing.assert_allclose(z, zd, rtol=1e-12, atol=1e-12)
        # each step alone
        np.testing.assert_allclose(O.rotate_structured(xb, rb, None), O.rotate(xb, I.to_bf16_bits(dense), None),
                                   rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(O.rotate_structured(xb, None, ri),
                                   O.rotate(xb, None, I.to_bf16_bits(np.stack([RI] * nb))), rtol=1e-12, atol=1e-12)


def test_structured_rotation_against_pure_python_loops_and_exact_cases():
    xb, rb, ri = _structured_case(2, 4, seed=99)
    x, RB, RI = O.decode_bf16(xb), O.decode_bf16(rb), O.decode_bf16(ri)
    z = O.rotate_structured(xb, rb, ri)
    for t in range(2):
        for bo in range(4):
            for j in range(32):
                acc = 0.0
                for k in range(32):
                    y = 0.0
                    for b in range(4):
                        y += RB[bo, b] * x[t, 32 * b + k]        # Y = R_B X: mixes blocks, keeps position k
                    acc += y * RI[k, j]                            # Z = Y R_intra: mixes positions
                assert abs(z[t, 32 * bo + j] - acc) <= 1e-12 * max(1.0, abs(acc))
    # a block permutation moves whole blocks, a position permutation acts inside every block alike
    g = np.random.default_rng(1)
    xi = g.integers(-8, 9, size=(3, 4 * 32)).astype(np.float64)
    pb, pk = g.permutation(4), g.permutation(32)
    PB = np.zeros((4, 4)); PB[np.arange(4), pb] = 1                # (PB X)[b'] = X[pb[b']]
    PK = np.zeros((32, 32)); PK[pk, np.arange(32)] = 1             # (Y PK)[., j] = Y[., pk[j]]
    z = O.rotate_structured(I.to_bf16_bits(xi), I.to_bf16_bits(PB), I.to_bf16_bits(PK))
    want = xi.reshape(3, 4, 32)[:, pb][:, :, pk].reshape(3, 128)
    assert np.array_equal(z, want)
    # energy conservation (total variance across blocks, App. A.1) with the float64 orthogonal factors
    Q, P = I.orthogonal(4, g), I.orthogonal(32, g)
    xt = O.decode_bf16(xb)[0].reshape(4, 32)
    zt = Q @ xt @ P
    assert abs((zt ** 2).sum() - (xt ** 2).sum()) <= 1e-10 * (xt ** 2).sum()
