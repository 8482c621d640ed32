"""Pins of the CPU oracle against things other than itself (no GPU needed).

P1 brute force over the six 2-of-4 patterns, P2 structural invariants, P3 Lemma 1,
P4 numpy fp64 matmul on masked dense matrices, P5 central finite differences,
P7 fused-adapter identity of Eq. (concat), P8 metadata reorder properties.
"""
import itertools
import math
import os

import numpy as np
import pytest

from paper_2608_24070_b200 import inputs as si

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16(x):
    return si.f32_to_bf16_bits(np.asarray(x, np.float32))


def f64(bits):
    return si.bf16_bits_to_f32(bits).astype(np.float64)


# ----------------------------------------------------------------------------- P1
def brute_pair(vals4):
    """Max sum of |w| over the six pairs, exact in fp64; ties -> lexicographically smallest pair."""
    best, best_pair = None, None
    for pair in itertools.combinations(range(4), 2):
        s = abs(vals4[pair[0]]) + abs(vals4[pair[1]])
        if best is None or s > best:
            best, best_pair = s, pair
    return best_pair


def test_p1_worked_groups(oracle):
    # hand-derived from the selection rule (largest magnitude first, lower index wins ties)
    W = bf16([[0.5, -0.5, 0.25, 0.5, 1, 2, 2, 3]])
    vals, nib, mask = oracle.prune24(W)
    assert nib.tolist() == [[0x4, 0xD]]
    assert f64(vals).tolist() == [[0.5, -0.5, 2.0, 3.0]]
    assert mask.tolist() == [[0b10100011]]


def test_p1_exhaustive_small_alphabet(oracle):
    alphabet = [0.0, -0.0, 1.0, -1.0, 2.0, -2.0]
    groups = list(itertools.product(alphabet, repeat=4))
    W = bf16(np.array(groups, np.float32).reshape(1, -1))
    pad = (-W.shape[1]) % 8
    W = np.concatenate([W, np.zeros((1, pad), np.uint16)], axis=1)
    vals, nib, mask = oracle.prune24(W)
    for g, grp in enumerate(groups):
        p0, p1 = brute_pair(grp)
        assert nib[0, g] == (p0 | (p1 << 2)), (grp, nib[0, g])
        # bit copies (sign of zero preserved)
        assert vals[0, 2 * g] == W[0, 4 * g + p0] and vals[0, 2 * g + 1] == W[0, 4 * g + p1]


def test_p1_random_bf16_matches_brute_force(oracle):
    W = si.gaussian_bf16((64, 256), 0.02, 7)
    # inject exact ties and zeros
    W[3, 8:12] = bf16([0.25, 0.25, -0.25, 0.25])
    W[5, 0:4] = 0
    vals, nib, mask = oracle.prune24(W)
    Wd = f64(W)
    mb = oracle.mask_to_bool(mask, 256)
    for i in range(64):
        for g in range(64):
            p0, p1 = brute_pair(Wd[i, 4 * g:4 * g + 4])
            assert nib[i, g] == (p0 | (p1 << 2))
            assert mb[i, 4 * g:4 * g + 4].tolist() == [t in (p0, p1) for t in range(4)]


def test_p1_second_pass_brute_force(oracle):
    W = si.gaussian_bf16((128, 64), 0.02, 11)
    _, _, mask1 = oracle.prune24(W)
    valsT, nibT, mask2 = oracle.double_prune(W, mask1)
    m1 = oracle.mask_to_bool(mask1, 64)
    m2 = oracle.mask_to_bool(mask2, 64)
    WR = np.where(m1, f64(W), 0.0)
    for j in range(64):
        for h in range(32):
            col = WR[4 * h:4 * h + 4, j]
            q0, q1 = brute_pair(col)
            assert nibT[j, h] == (q0 | (q1 << 2))
            assert f64(valsT[j, 2 * h:2 * h + 2]).tolist() == [col[q0], col[q1]]
            expect = [(t in (q0, q1)) and bool(m1[4 * h + t, j]) for t in range(4)]
            assert m2[4 * h:4 * h + 4, j].tolist() == expect


def test_p1_second_pass_worked_column(oracle):
    # column group of W^R = [pruned, pruned, 0.1, pruned] -> keys [0,0,k,0] -> keep (0,2)
    W = np.zeros((4, 8), np.uint16)
    W[:, 0] = bf16([0.3, 0.2, 0.1, 0.4])
    mask1 = np.zeros((4, 1), np.uint8)
    mask1[2, 0] = 1  # only (2, 0) survived pass 1 in column 0
    valsT, nibT, mask2 = oracle.double_prune(W, mask1)
    assert nibT[0, 0] == 0x8
    assert valsT[0, 0] == 0 and valsT[0, 1] == W[2, 0]
    assert mask2[:, 0].tolist() == [0, 0, 1, 0]


# ----------------------------------------------------------------------------- P2
def test_p2_structure(oracle):
    W = si.gaussian_bf16((256, 384), 0.02, 3)
    vals, nib, mask1 = oracle.prune24(W)
    valsT, nibT, mask2 = oracle.double_prune(W, mask1)
    m1 = oracle.mask_to_bool(mask1, 384)
    m2 = oracle.mask_to_bool(mask2, 384)
    assert (m1.reshape(256, 96, 4).sum(-1) == 2).all()
    assert not (m2 & ~m1).any()
    assert (m2.T.reshape(384, 64, 4).sum(-1) <= 2).all()
    legal = {0x4, 0x8, 0xC, 0x9, 0xD, 0xE}
    assert set(np.unique(nib)) <= legal and set(np.unique(nibT)) <= legal
    Wd = f64(W)
    assert np.array_equal(oracle.decompress(vals, nib), np.where(m1, Wd, 0.0))
    assert np.array_equal(oracle.decompress(valsT, nibT), np.where(m2, Wd, 0.0).T)


# ----------------------------------------------------------------------------- P3
def lemma1(n, m):
    s = n / m
    return sum(math.comb(m, j) * s ** j * (1 - s) ** (m - j) * (j - n) / m for j in range(n + 1, m + 1))


def read_golden_lemma():
    out = {}
    with open(os.path.join(GOLDEN, "lemma1_extra_zeros.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                out[k] = float(v)
    return out


def test_p3_lemma1_printed_values():
    g = read_golden_lemma()
    assert lemma1(1, 2) == pytest.approx(g["1:2"], abs=1e-12)
    assert lemma1(2, 4) == pytest.approx(g["2:4"], abs=1e-12)


def test_p3_lemma1_on_gaussian(oracle):
    g = read_golden_lemma()["2:4"]
    W = si.gaussian_bf16((2048, 2048), 0.02, si.seed_for(3, 0, "W"))
    _, _, mask1 = oracle.prune24(W)
    _, _, mask2 = oracle.double_prune(W, mask1)
    m1 = oracle.mask_to_bool(mask1, 2048)
    m2 = oracle.mask_to_bool(mask2, 2048)
    assert m1.mean() == 0.5
    extra = m1.mean() - m2.mean()
    assert abs(extra - g) < 1e-3, extra
    # proof of Lemma 1: non-zeros per 4-group of the transposed matrix ~ Binomial(4, 1/2)
    hist = np.bincount(m1.T.reshape(2048, 512, 4).sum(-1).ravel(), minlength=5) / (2048 * 512)
    assert np.allclose(hist, np.array([1, 4, 6, 4, 1]) / 16, atol=3e-3)


# ----------------------------------------------------------------------------- P4
def _small_problem(seed=5, b=48, d_in=64, d_out=96, r=8):
    W = si.gaussian_bf16((d_out, d_in), 0.02, seed)
    X = si.gaussian_bf16((b, d_in), 1.0, seed + 1)
    dY = si.gaussian_bf16((b, d_out), 1.0, seed + 2)
    L = si.gaussian_bf16((d_in, r), 0.01, seed + 3)
    R = si.gaussian_bf16((r, d_out), 0.01, seed + 4)
    return W, X, dY, L, R


def test_p4_gemms_equal_numpy_on_masked_dense(oracle):
    W, X, dY, L, R = _small_problem()
    b, d_in = X.shape
    d_out = W.shape[0]
    _, nib, mask1 = oracle.prune24(W)
    _, _, mask2 = oracle.double_prune(W, mask1)
    m1 = oracle.mask_to_bool(mask1, d_in)
    m2 = oracle.mask_to_bool(mask2, d_in)
    Wd, Xd, dYd, Ld, Rd = map(f64, (W, X, dY, L, R))
    WR, WRC = np.where(m1, Wd, 0), np.where(m2, Wd, 0)
    rows = np.arange(b)

    def close(a, ref):
        return np.abs(a - ref).max() <= 1e-12 * np.abs(ref).max()

    assert close(oracle.fwd_rows(X, W, mask1, rows), Xd @ WR.T)
    assert close(oracle.fwd_rows(X, W, mask1, rows, L, R), Xd @ WR.T + (Xd @ Ld) @ Rd)
    assert close(oracle.dx_rows(dY, W, mask2, rows), dYd @ WRC)
    assert close(oracle.dx_rows(dY, W, mask2, rows, L, R), dYd @ WRC + (dYd @ Rd.T) @ Ld.T)
    dW = dYd.T @ Xd
    dWc_ref = dW[m1].reshape(d_out, d_in // 2)      # row-major boolean gather = ascending columns
    assert close(oracle.dw_rows(dY, X, mask1, np.arange(d_out)), dWc_ref)
    assert close(oracle.adapter_T_rows(X, L, rows), Xd @ Ld)
    assert close(oracle.adapter_dT_rows(dY, R, rows), dYd @ Rd.T)
    assert close(oracle.adapter_dL_rows(X, dY, R, np.arange(d_in)), Xd.T @ (dYd @ Rd.T))
    assert close(oracle.adapter_dR_cols(X, L, dY, np.arange(d_out)), (Xd @ Ld).T @ dYd)
    # a transposed operand or a swapped mask would not survive these:
    assert not close(oracle.dx_rows(dY, W, mask1, rows), dYd @ WRC)


def test_p4_row_sampling_is_exact(oracle):
    W, X, dY, L, R = _small_problem(seed=9)
    _, _, mask1 = oracle.prune24(W)
    full = oracle.fwd_rows(X, W, mask1, np.arange(X.shape[0]), L, R)
    pick = np.array([0, 5, 17, 47], np.int32)
    assert np.array_equal(oracle.fwd_rows(X, W, mask1, pick, L, R), full[pick])
    cols = np.array([0, 3, 95], np.int32)
    assert np.array_equal(oracle.adapter_dR_cols(X, L, dY, cols),
                          oracle.adapter_dR_cols(X, L, dY, np.arange(96))[:, cols])


# ----------------------------------------------------------------------------- P5
def _grid(shape, seed, lo=-16, hi=16, scale=1 / 8):
    rng = np.random.Generator(np.random.PCG64(seed))
    return (rng.integers(lo, hi + 1, size=shape) * scale).astype(np.float32)


def test_p5_finite_differences(oracle):
    """l = <Y(X, W, L, R), dY> is linear in each argument, so central differences with a
    step that stays on the bf16 grid are exact up to fp64 rounding."""
    b, d_in, d_out, r, h = 6, 8, 8, 2, 0.125
    Wf, Xf, dYf = _grid((d_out, d_in), 1), _grid((b, d_in), 2), _grid((b, d_out), 3)
    Lf, Rf = _grid((d_in, r), 4), _grid((r, d_out), 5)
    # make magnitudes within groups distinct enough that the mask is what we think
    W, X, dY, L, R = map(bf16, (Wf, Xf, dYf, Lf, Rf))
    _, _, mask1 = oracle.prune24(W)
    _, _, mask2 = oracle.double_prune(W, mask1)
    m1 = oracle.mask_to_bool(mask1, d_in)
    rows = np.arange(b)
    dYd = f64(dY)

    def loss(Xb=X, Wb=W, Lb=L, Rb=R):
        return float((oracle.fwd_rows(Xb, Wb, mask1, rows, Lb, Rb) * dYd).sum())

    def fd(base_f, which):
        g = np.zeros_like(base_f, dtype=np.float64)
        for idx in np.ndindex(base_f.shape):
            p, m = base_f.copy(), base_f.copy()
            p[idx] += h
            m[idx] -= h
            g[idx] = (loss(**{which: bf16(p)}) - loss(**{which: bf16(m)})) / (2 * h)
        return g

    # dW on kept entries (mask held fixed), compressed in ascending column order
    gW = fd(Wf, "Wb")
    assert np.allclose(oracle.dw_rows(dY, X, mask1, np.arange(d_out)), gW[m1].reshape(d_out, d_in // 2),
                       rtol=0, atol=1e-9)
    assert np.allclose(gW[~m1], 0.0)
    # dL, dR
    assert np.allclose(oracle.adapter_dL_rows(X, dY, R, np.arange(d_in)), fd(Lf, "Lb"), rtol=0, atol=1e-9)
    assert np.allclose(oracle.adapter_dR_cols(X, L, dY, np.arange(d_out)), fd(Rf, "Rb"), rtol=0, atol=1e-9)
    # true input gradient uses W^R (first mask) ...
    gX = fd(Xf, "Xb")
    assert np.allclose(oracle.dx_rows(dY, W, mask1, rows, L, R), gX, rtol=0, atol=1e-9)

    # ... the double-pruned dX is the exact gradient of X -> X (W^{R,C})^T + (X L) R
    def loss_rc(Xb):
        return float((oracle.fwd_rows(Xb, W, mask2, rows, L, R) * dYd).sum())

    gX_rc = np.zeros((b, d_in))
    for idx in np.ndindex(Xf.shape):
        p, m = Xf.copy(), Xf.copy()
        p[idx] += h
        m[idx] -= h
        gX_rc[idx] = (loss_rc(bf16(p)) - loss_rc(bf16(m))) / (2 * h)
    assert np.allclose(oracle.dx_rows(dY, W, mask2, rows, L, R), gX_rc, rtol=0, atol=1e-9)


# ----------------------------------------------------------------------------- P7
def test_p7_adapter_identity(oracle):
    W, X, dY, L, R = _small_problem(seed=21)
    _, _, mask1 = oracle.prune24(W)
    rows = np.arange(X.shape[0])
    plain = oracle.fwd_rows(X, W, mask1, rows)
    fused = oracle.fwd_rows(X, W, mask1, rows, L, R)
    lr = f64(X) @ f64(L) @ f64(R)
    assert np.allclose(fused - plain, lr, rtol=0, atol=1e-12)
    # linearity in X: Y(2X) = 2 Y(X) exactly (scaling by 2 is exact in bf16 and fp64)
    X2 = bf16(2 * si.bf16_bits_to_f32(X))
    assert np.array_equal(oracle.fwd_rows(X2, W, mask1, rows, L, R), 2 * fused)


# ----------------------------------------------------------------------------- P8
def test_p8_metadata_reorder_is_a_permutation(oracle):
    rng = np.random.Generator(np.random.PCG64(1))
    rows, cols = 256, 384
    canon = rng.integers(0, 1 << 16, size=(rows, cols // 16), dtype=np.uint16)
    hw = oracle.canonical_to_hw(canon)
    assert hw.size == rows * cols // 8
    # same multiset of 16-bit units, every destination written once
    assert sorted(hw.view(np.uint16).tolist()) == sorted(canon.ravel().tolist())
    tag = np.arange(rows * cols // 16, dtype=np.uint16).reshape(rows, cols // 16)
    assert np.unique(oracle.canonical_to_hw(tag).view(np.uint16)).size == tag.size


def test_p8_metadata_layout_spot_values(oracle):
    """Hand-placed units: row rr, 16-column slot cs of block (rb, cb) must land in 32-bit word
    (16*(rr//16) + 8*(cs%2) + rr%8) * 4 + cs//2, low half for rows with (rr//8)%2 == 0."""
    rows, cols = 256, 256
    canon = np.zeros((rows, cols // 16), np.uint16)
    canon[0, 0] = 0x1111      # block (0,0), rr=0,  cs=0 -> word 0 low
    canon[8, 0] = 0x2222      # rr=8            -> word 0 high
    canon[1, 1] = 0x3333      # rr=1, cs=1      -> lane 9, col 0 -> word 36 low
    canon[17, 6] = 0x4444     # rr=17, cs=6     -> lane 17, col 3 -> word 71 low
    canon[128 + 31, 8 + 3] = 0x5555  # block (1,1): rr=31, cs=3 -> lane 16+8+7=31, col 1, high
    hw = oracle.canonical_to_hw(canon).view(np.uint16)
    assert hw[0] == 0x1111 and hw[1] == 0x2222
    assert hw[36 * 2] == 0x3333
    assert hw[71 * 2] == 0x4444
    blk = (1 * 2 + 1) * 1024
    assert hw[blk + (31 * 4 + 1) * 2 + 1] == 0x5555
    assert np.count_nonzero(hw) == 5


# The tensor-core order written out as a TABLE instead of a formula (a slip in the oracle's index
# arithmetic fails here on the CPU; the GPU exact case X = I pins the same order through the MMA).
# tcgen05.cp.128x128b moves 128 shared-memory rows of 16 bytes into 128 tensor-memory lanes x 4
# 32-bit columns: byte 16*lane + 4*column + 2*half of a 2 KB block.  One column serves two
# consecutive K = 32 sparse MMAs of a 128-row operand; within each run of 16 operand rows the
# metadata of a 16-column slot sits as follows (row within the 16 -> lane within the 16, half-word):
_LANE_EVEN_SLOT = (0, 1, 2, 3, 4, 5, 6, 7, 0, 1, 2, 3, 4, 5, 6, 7)          # slots 0, 2, 4, 6 of a block
_LANE_ODD_SLOT = (8, 9, 10, 11, 12, 13, 14, 15, 8, 9, 10, 11, 12, 13, 14, 15)  # slots 1, 3, 5, 7
_HALF_WORD = (0, 0, 0, 0, 0, 0, 0, 0, 1, 1, 1, 1, 1, 1, 1, 1)
_COLUMN_OF_SLOT = (0, 0, 1, 1, 2, 2, 3, 3)


def test_p8_metadata_layout_against_the_lane_table(oracle):
    rng = np.random.Generator(np.random.PCG64(8))
    rows, cols = 384, 256
    canon = rng.integers(0, 1 << 16, size=(rows, cols // 16), dtype=np.uint16)
    want = np.zeros(rows * cols // 8, np.uint8)
    for i in range(rows):
        for u in range(cols // 16):
            block = (i // 128) * (cols // 128) + u // 8
            r16, slot = i % 16, u % 8
            lane = 16 * ((i % 128) // 16) + (_LANE_ODD_SLOT if slot % 2 else _LANE_EVEN_SLOT)[r16]
            byte = 2048 * block + 16 * lane + 4 * _COLUMN_OF_SLOT[slot] + 2 * _HALF_WORD[r16]
            want[byte] = int(canon[i, u]) & 0xFF
            want[byte + 1] = int(canon[i, u]) >> 8
    assert np.array_equal(oracle.canonical_to_hw(canon), want)


def test_pack_canonical(oracle):
    nib = np.array([[0x4, 0xD, 0x9, 0xE]], np.uint8)
    assert oracle.pack_canonical(nib).tolist() == [[0xE9D4]]


# ----------------------------------------------------------------------------- optimizer tail (Algorithm 1)
def test_sparse_add_equals_numpy(oracle):
    A = si.gaussian_bf16((64, 96), 1.0, 41)
    Bv = si.gaussian_bf16((64, 96), 0.02, 42)
    beta, gamma = 1.0 / 1024.0, 0.01
    got = oracle.sparse_add(A, Bv, beta, gamma)
    assert np.array_equal(got, beta * f64(A) + gamma * f64(Bv))
    assert np.array_equal(oracle.sparse_add(A, Bv, 1.0, 0.0), f64(A))


def test_update_transposed_reproduces_double_prune(oracle):
    """Feeding the forward copy's own values back must rebuild exactly what the second pruning
    pass wrote; with the masks held fixed the map is linear in the values (scale by 2, negate)."""
    W = si.gaussian_bf16((256, 384), 0.02, 43)
    vals, nib, mask1 = oracle.prune24(W)
    valsT, nibT, mask2 = oracle.double_prune(W, mask1)
    assert np.array_equal(oracle.update_transposed(vals, mask1, mask2, nibT), valsT)
    W2 = bf16(-2.0 * si.bf16_bits_to_f32(W))            # same magnitudes order -> same masks
    vals2, nib2, mask1b = oracle.prune24(W2)
    valsT2, nibT2, mask2b = oracle.double_prune(W2, mask1b)
    assert np.array_equal(mask1b, mask1) and np.array_equal(mask2b, mask2) and np.array_equal(nibT2, nibT)
    assert np.array_equal(oracle.update_transposed(vals2, mask1, mask2, nibT), valsT2)
    # entries dropped by the second pass stay +0 whatever the new values are
    junk = np.full_like(vals, 0x3F80)
    out = oracle.update_transposed(junk, mask1, mask2, nibT)
    m2T = oracle.mask_to_bool(mask2, 384).T
    sel = np.zeros_like(out, bool)
    for t in range(2):
        q = (nibT >> (2 * t)) & 3
        rows = 4 * np.arange(64)[None, :] + q
        sel[:, t::2] = m2T[np.arange(384)[:, None], rows]
    assert np.array_equal(out != 0, sel)


# ----------------------------------------------------------------------------- P9: general N:M (O9, O10)
NM_PATTERNS = [(1, 2), (2, 4), (1, 4), (2, 8), (4, 8), (3, 8), (4, 16)]


def _brute_force_group(keys, n):
    """All n-subsets of one group: largest sum of magnitudes, ties -> lexicographically smallest."""
    best, best_sum = None, -1
    for comb in itertools.combinations(range(len(keys)), n):
        s = int(sum(int(keys[t]) for t in comb))
        if s > best_sum:                                  # combinations come in lexicographic order
            best, best_sum = comb, s
    return best


def test_p9_nm_equals_the_2_4_path(oracle):
    W = si.gaussian_bf16((64, 128), 0.02, 91)
    vals, nib, mask1 = oracle.prune24(W)
    WR, m1 = oracle.prune_nm(W, 2, 4)
    assert np.array_equal(m1, mask1)
    keep = oracle.mask_to_bool(mask1, 128)
    assert np.array_equal(WR, np.where(keep, W, 0).astype(np.uint16))
    assert np.array_equal(WR[keep].reshape(64, 64), vals)
    _, _, mask2 = oracle.double_prune(W, mask1)
    WRC, m2 = oracle.double_prune_nm(W, m1, 2, 4)
    assert np.array_equal(m2, mask2)
    assert np.array_equal(WRC, np.where(oracle.mask_to_bool(mask2, 128), W, 0).astype(np.uint16))


@pytest.mark.parametrize("n,m", NM_PATTERNS)
def test_p9_nm_brute_force_with_ties(oracle, n, m):
    """Tie-heavy alphabet (few distinct magnitudes, both signs and zeros) against subset enumeration,
    for both passes."""
    rng = np.random.Generator(np.random.PCG64(900 + 10 * m + n))
    alphabet = si.f32_to_bf16_bits(np.array([0.0, -0.0, 0.5, -0.5, 1.0, -1.0, 1.5, 3.0], np.float32))
    d_out, d_in = 2 * m, 16 * max(1, m // 8) * 2
    d_in = max(d_in, 2 * m)
    W = rng.choice(alphabet, size=(d_out, d_in)).astype(np.uint16)
    WR, mask1 = oracle.prune_nm(W, n, m)
    keep1 = oracle.mask_to_bool(mask1, d_in)
    key = (W & 0x7FFF).astype(np.int64)
    for i in range(d_out):
        for g in range(d_in // m):
            want = _brute_force_group(key[i, m * g:m * g + m], n)
            got = tuple(np.flatnonzero(keep1[i, m * g:m * g + m]))
            assert got == want, (i, g, key[i, m * g:m * g + m], got, want)
    assert np.array_equal(WR, np.where(keep1, W, 0).astype(np.uint16))
    WRC, mask2 = oracle.double_prune_nm(W, mask1, n, m)
    keep2 = oracle.mask_to_bool(mask2, d_in)
    keyR = np.where(keep1, key, 0)
    for j in range(d_in):
        for h in range(d_out // m):
            col = keyR[m * h:m * h + m, j]
            want = set(_brute_force_group(col, n))
            got = set(np.flatnonzero(keep2[m * h:m * h + m, j]))
            # second-pass picks that the first pass had removed (zeros filling up the n slots) are not in mask2
            assert got == {t for t in want if keep1[m * h + t, j]}, (j, h, col, got, want)
    assert np.array_equal(WRC, np.where(keep2, W, 0).astype(np.uint16))


@pytest.mark.parametrize("n,m", NM_PATTERNS)
def test_p9_nm_structure_and_lemma1(oracle, n, m):
    """Exactly n per row group, at most n per column group, mask2 inside mask1, and the extra zeros of
    Eq. (sparsity_ratio) on Gaussian data (for 1:2 and 2:4 also the values the text prints)."""
    d = 1024
    W = si.gaussian_bf16((d, d), 0.02, 9000 + 10 * m + n)
    WR, mask1 = oracle.prune_nm(W, n, m)
    WRC, mask2 = oracle.double_prune_nm(W, mask1, n, m)
    k1, k2 = oracle.mask_to_bool(mask1, d), oracle.mask_to_bool(mask2, d)
    assert np.all(k1.reshape(d, d // m, m).sum(-1) == n)
    assert np.all(k2.T.reshape(d, d // m, m).sum(-1) <= n)
    assert not np.any(k2 & ~k1)
    assert np.array_equal(WR, np.where(k1, W, 0).astype(np.uint16))
    assert np.array_equal(WRC, np.where(k2, W, 0).astype(np.uint16))
    extra = k1.mean() - k2.mean()
    assert abs(extra - lemma1(n, m)) < 1.5e-3, (extra, lemma1(n, m))
    printed = read_golden_lemma().get(f"{n}:{m}")
    if printed is not None:
        assert abs(extra - printed) < 1.5e-3
    # the proof's premise: kept entries per column group ~ Binomial(m, n/m)
    hist = np.bincount(k1.T.reshape(d, d // m, m).sum(-1).ravel(), minlength=m + 1) / (d * d // m)
    binom = np.array([math.comb(m, j) * (n / m) ** j * (1 - n / m) ** (m - j) for j in range(m + 1)])
    assert np.allclose(hist, binom, atol=4e-3)


# ----------------------------------------------------------------------------- P10: mask difference (O11)
def test_p10_mask_difference(oracle):
    rng = np.random.Generator(np.random.PCG64(1001))
    a = rng.integers(0, 256, size=(24, 40), dtype=np.uint8)
    b = rng.integers(0, 256, size=(24, 40), dtype=np.uint8)
    want = int((np.unpackbits(a, axis=1, bitorder="little") != np.unpackbits(b, axis=1, bitorder="little")).sum())
    assert oracle.mask_difference(a, b) == want
    assert oracle.mask_difference(a, a) == 0
    assert oracle.mask_difference(a, ~a) == 24 * 320
    # a worked case: the 2:4 masks of two matrices that differ in one group only, (1,2 kept) -> (0,3 kept):
    # all four positions of that group change
    W = si.f32_to_bf16_bits(np.tile(np.array([0.1, 2.0, 3.0, 0.2], np.float32), (4, 8)))
    V = W.copy()
    V[2, 4:8] = si.f32_to_bf16_bits(np.array([5.0, 0.2, 0.1, 4.0], np.float32))
    _, _, m1 = oracle.prune24(W)
    _, _, m2 = oracle.prune24(V)
    assert oracle.mask_difference(m1, m2) == 4
