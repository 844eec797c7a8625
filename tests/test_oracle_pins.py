"""Pins for the float64 oracle: each checks it against something the paper or the
mathematics fixes (closed forms, the SVD polar factor, brute force on tiny inputs,
printed values), never against the oracle's own formula retyped."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle as O

RNG = np.random.default_rng(20260516)


def f_scalar(x, k):
    """Scalar Newton-Schulz map x -> x (3 - x^2) / 2 applied k times (what Alg. 4 does to a singular value)."""
    for _ in range(k):
        x = 0.5 * x * (3.0 - x * x)
    return x


# ----------------------------------------------------------------------------- momentum
def test_momentum_constant_gradient_closed_form():
    g = RNG.normal(size=(5, 7))
    w = RNG.normal(size=(5, 7))
    beta = 0.9
    mom = np.zeros_like(g)
    for t in range(1, 13):
        mom = O.momentum_update(mom, g, w, beta, 0.0)
        assert np.allclose(mom, (1.0 - beta ** t) * g, rtol=1e-13, atol=0)


def test_momentum_beta_zero_and_weight_decay():
    g = RNG.normal(size=(4, 3))
    w = RNG.normal(size=(4, 3))
    old = RNG.normal(size=(4, 3))
    out = O.momentum_update(old, g, w, 0.0, 0.25)
    assert np.allclose(out, g + 0.25 * w, rtol=1e-15)
    # one hand-computed entry: beta=0.5, lambda=0.1, mom=2, g=4, w=10 -> 0.5*2 + 0.5*(4+1) = 3.5
    assert O.momentum_update(np.array([[2.0]]), np.array([[4.0]]), np.array([[10.0]]), 0.5, 0.1)[0, 0] == 3.5


# ----------------------------------------------------------------------------- Newton-Schulz
@pytest.mark.parametrize("shape", [(3, 5), (8, 8), (16, 4), (1, 9), (7, 1)])
@pytest.mark.parametrize("K", [0, 1, 3, 5])
def test_polar_ns_matches_svd_closed_form(shape, K):
    x = RNG.normal(size=shape)
    u, s, vt = np.linalg.svd(x, full_matrices=False)
    sigma = math.sqrt(np.sum(s ** 2))
    expect = (u * f_scalar(s / sigma, K)) @ vt
    got = O.polar_ns(x, K, 1e-12)
    assert np.allclose(got, expect, rtol=1e-10, atol=1e-13)
    got_short = O.polar_ns_short_side(x, K, 1e-12)
    assert np.allclose(got_short, expect, rtol=1e-10, atol=1e-13)


def test_polar_ns_literal_equals_short_side_larger():
    x = RNG.normal(size=(24, 70))
    a = O.polar_ns(x, 5)
    b = O.polar_ns_short_side(x, 5)
    assert np.max(np.abs(a - b)) <= 1e-13 * np.max(np.abs(a))


@pytest.mark.parametrize("shape,K", [((6, 40), 5), ((40, 6), 3), ((9, 9), 2), ((3, 17), 7)])
def test_gram_space_evaluation_is_the_same_map_as_alg4(shape, K):
    """The reading the CUDA path relies on for short sides: with A_k = Y_k Y_k^T and P_k = 3/2 I - A_k / 2, Alg. 4's
    step gives A_{k+1} = P_k A_k P_k = 9/4 A_k - 3/2 A_k^2 + 1/4 A_k^3 and Y_K = (P_{K-1} ... P_0) Y_0; with
    T_k = (3/2)^k I + F_k the product obeys F_{k+1} = 3/2 F_k - (3/2)^k / 2 A_k - 1/2 A_k F_k, F_0 = 0.  Written out here in
    numpy (not in the oracle) and compared with the oracle's literal iteration."""
    x = RNG.normal(size=shape)
    wide = shape[0] <= shape[1]
    y0 = x / np.linalg.norm(x)
    a = y0 @ y0.T if wide else y0.T @ y0
    f = np.zeros_like(a)
    t = 1.0
    for _ in range(K):
        f, a = 1.5 * f - 0.5 * t * a - 0.5 * a @ f, 2.25 * a - 1.5 * a @ a + 0.25 * a @ a @ a
        t *= 1.5
    tk = t * np.eye(a.shape[0]) + f
    y_gram_space = tk @ y0 if wide else y0 @ tk
    y_literal = O.polar_ns(x, K)
    assert np.max(np.abs(y_gram_space - y_literal)) <= 1e-12 * np.max(np.abs(y_literal))
    # and the s x s matrix the chain carries is the Gram matrix of the literal iterate
    yk_minus_1 = O.polar_ns(x, K - 1)
    a_lit = yk_minus_1 @ yk_minus_1.T if wide else yk_minus_1.T @ yk_minus_1
    a_chain = y0 @ y0.T if wide else y0.T @ y0
    for _ in range(K - 1):
        a_chain = 2.25 * a_chain - 1.5 * a_chain @ a_chain + 0.25 * a_chain @ a_chain @ a_chain
    assert np.max(np.abs(a_chain - a_lit)) <= 1e-12


@pytest.mark.parametrize("shape,K", [((6, 40), 5), ((40, 6), 3), ((9, 14), 2), ((5, 17), 7)])
def test_gram_space_chain_of_symmetric_products_is_the_same_map_as_alg4(shape, K):
    """The form of the same reading that the CUDA path runs through memory for longer short sides: with Q_k = -A_k / 2
    and T_k = (3/2)^k (I + H_k):  R_k = Q_k Q_k + 3 Q_k,  Q_{k+1} = Q_k R_k + 9/4 Q_k,
    H_{k+1} = 2/3 (Q_k H_k + Q_k + 3/2 H_k) with H_1 = 2/3 Q_0,  Y_K = (3/2)^K (Y_0 + H_K Y_0);  every matrix of the
    chain is symmetric (only its upper tiles are computed there).  Written out in numpy and compared with the oracle's
    literal iteration."""
    x = RNG.normal(size=shape)
    wide = shape[0] <= shape[1]
    y0 = x / np.linalg.norm(x)
    q = -0.5 * (y0 @ y0.T if wide else y0.T @ y0)
    h = (2.0 / 3.0) * q
    for k in range(K - 1):                 # Q_{k+1} from Q_k; H_{k+2} from Q_{k+1}, H_{k+1}
        r = q @ q + 3.0 * q
        q = q @ r + 2.25 * q
        h = (2.0 / 3.0) * (q @ h + q + 1.5 * h)
        for m in (r, q, h):
            assert np.max(np.abs(m - m.T)) <= 1e-14
    f = 1.5 ** K * h
    y_chain = 1.5 ** K * y0 + (f @ y0 if wide else y0 @ f)
    y_literal = O.polar_ns(x, K)
    assert np.max(np.abs(y_chain - y_literal)) <= 1e-12 * np.max(np.abs(y_literal))
    # Q_{K-1} is -1/2 times the Gram matrix of the literal iterate Y_{K-1}
    yk = O.polar_ns(x, K - 1)
    assert np.max(np.abs(-2.0 * q - (yk @ yk.T if wide else yk.T @ yk))) <= 1e-12


@pytest.mark.parametrize("K", [1, 2, 3, 4, 5])
def test_newton_schulz_polar_error_bound(K):
    # tall 9 x 2 with singular values 0.8, 0.6: ||X||_F = 1, rho = ||I - X^T X||_op = 0.64
    q1, _ = np.linalg.qr(RNG.normal(size=(9, 2)))
    q2, _ = np.linalg.qr(RNG.normal(size=(2, 2)))
    x = (q1 * np.array([0.8, 0.6])) @ q2.T
    polar = q1 @ q2.T
    rho = np.linalg.norm(np.eye(2) - x.T @ x, 2)
    assert abs(rho - 0.64) < 1e-12
    y = O.polar_ns(x, K)                      # Frobenius scaling is the identity here
    assert np.linalg.norm(y, 2) <= 1.0 + 1e-12
    assert np.linalg.norm(y - polar, 2) <= rho ** (2 ** K) + 1e-12
    if K == 5:
        # <X, polar(X)> = nuclear norm
        assert abs(np.sum(x * y) - 1.4) < 1e-6


def test_newton_schulz_bare_loop_band():
    # Alg. 6 with a caller-chosen scaling: singular values in [0.6, 1.0] -> rho = 0.64
    u, _ = np.linalg.qr(RNG.normal(size=(10, 6)))
    v, _ = np.linalg.qr(RNG.normal(size=(6, 6)))
    s = np.array([1.0, 0.95, 0.9, 0.8, 0.7, 0.6])
    y0 = (u * s) @ v.T
    y5 = O.newton_schulz(y0, 5)
    assert np.linalg.norm(y5 - u @ v.T, 2) <= 0.64 ** 32 + 1e-12
    sv = np.linalg.svd(y5, compute_uv=False)
    assert np.all(sv <= 1 + 1e-12) and np.all(sv >= f_scalar(0.6, 5) - 1e-12)


def test_polar_ns_special_cases():
    # orthogonal s x s: all singular values 1 -> after fro scaling 1/sqrt(s)
    q, _ = np.linalg.qr(RNG.normal(size=(6, 6)))
    assert np.allclose(O.polar_ns(q, 4), f_scalar(1 / math.sqrt(6), 4) * q, rtol=1e-11, atol=1e-14)
    # diagonal matrix: entrywise scalar recurrence, signs preserved
    dvals = np.array([3.0, -2.0, 0.5, 1.0])
    sigma = math.sqrt(np.sum(dvals ** 2))
    got = O.polar_ns(np.diag(dvals), 3)
    assert np.allclose(np.diag(got), np.sign(dvals) * f_scalar(np.abs(dvals) / sigma, 3), rtol=1e-12)
    assert np.allclose(got - np.diag(np.diag(got)), 0, atol=1e-15)
    # 1 x n: positive multiple of the input (so its sign pattern is that of the input)
    row = RNG.normal(size=(1, 11))
    out = O.polar_ns(row, 5)
    ratio = out / row
    assert np.all(ratio > 0) and np.allclose(ratio, ratio[0, 0], rtol=1e-12)
    # K = 0: plain Frobenius normalisation
    x = RNG.normal(size=(3, 4))
    assert np.allclose(O.polar_ns(x, 0), x / np.linalg.norm(x), rtol=1e-15)
    # all-zero input: sigma = 0 -> divide by eps -> zeros -> every bit is 1
    z = O.polar_ns(np.zeros((3, 3)), 5)
    assert np.all(z == 0) and np.all(O.encode_bits(z) == 1)


def test_planted_mistakes_fail_the_svd_pin():
    """The SVD pin has teeth: plausible slips in the iteration give different results."""
    x = RNG.normal(size=(5, 5))
    u, s, vt = np.linalg.svd(x)
    expect = (u * f_scalar(s / np.linalg.norm(x), 2)) @ vt
    y = x / np.linalg.norm(x)
    wrong_sign = y.copy()
    wrong_side = y.copy()
    for _ in range(2):
        wrong_sign = 0.5 * wrong_sign @ (3 * np.eye(5) + wrong_sign.T @ wrong_sign)
        wrong_side = 0.5 * wrong_side @ (3 * np.eye(5) - wrong_side @ wrong_side.T)
    assert not np.allclose(wrong_sign, expect, rtol=1e-6)
    assert not np.allclose(wrong_side, expect, rtol=1e-6)
    assert np.allclose(O.polar_ns(x, 2), expect, rtol=1e-11)


# ----------------------------------------------------------------------------- sign / pack
def test_sign_and_encoding_table():
    u = np.array([3.0, -2.0, 0.0, -0.0, np.nan, 1e-300, -1e-300])
    assert O.sign_pm1(u).tolist() == [1, -1, 1, 1, -1, 1, -1]
    assert O.encode_bits(u).tolist() == [1, 0, 1, 1, 0, 1, 0]
    assert O.decode_bits(np.array([0, 1])).tolist() == [-1, 1]
    assert np.array_equal(O.decode_bits(O.encode_bits(u)), O.sign_pm1(u))


def test_pack_bit_order_hand_example():
    bits = [1, 0, 0, 0, 0, 0, 0, 0,   0, 1, 0, 0, 0, 0, 0, 1,   1]
    assert O.pack_bits(bits).tolist() == [0x01, 0x82, 0x01]
    assert O.bytes_to_words(O.pack_bits(bits)).tolist() == [0x00018201]


@pytest.mark.parametrize("d", [1, 7, 8, 9, 31, 32, 33, 64, 1000, 4099])
def test_pack_roundtrip_and_size(d):
    bits = RNG.integers(0, 2, size=d).astype(np.uint8)
    packed = O.pack_bits(bits)
    assert packed.size == math.ceil(d / 8) == O.payload_bytes(d)
    assert np.array_equal(O.unpack_bits(packed, d), bits)
    # independent library check: numpy's own bit packer in little-endian bit order
    assert np.array_equal(packed, np.packbits(bits, bitorder="little"))
    # pad bits are zero
    if d % 8:
        assert packed[-1] >> (d % 8) == 0
    assert np.array_equal(O.words_to_bytes(O.bytes_to_words(packed), d), packed)


def test_payload_ratios_and_worked_example():
    d = 2 ** 20
    assert 4 * d / O.payload_bytes(d, 1) == 32       # bit-packed vs float32
    assert 4 * d / O.payload_bytes(d, 8) == 4        # int8 vs float32
    path = os.path.join(os.path.dirname(__file__), "golden", "payload_worked_example.txt")
    vals = {}
    for line in open(path):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            vals[k] = float(v)
    dd = int(vals["d_entries"])
    assert round(4 * dd / 1e6) == vals["fp32_megabytes"]
    assert round(O.payload_bytes(dd, 1) / 2 ** 20, 1) == vals["onebit_mebibytes"]
    assert O.payload_bytes(dd, 8) / 1e6 == vals["int8_megabytes"]
    assert 4 * dd / O.payload_bytes(dd, 1) == vals["ratio_onebit"]
    assert 4 * dd / O.payload_bytes(dd, 8) == vals["ratio_int8"]


# ----------------------------------------------------------------------------- vote
def brute_force_vote(bits_per_worker):
    """Count +1 and -1 ballots entry by entry in plain Python."""
    M = len(bits_per_worker)
    d = len(bits_per_worker[0])
    out = []
    for i in range(d):
        plus = sum(1 for m in range(M) if bits_per_worker[m][i] == 1)
        minus = M - plus
        out.append(1 if plus >= minus else 0)
    return out


@pytest.mark.parametrize("M", [1, 2, 3, 4, 5, 8, 16, 31, 32])
def test_vote_matches_brute_force_and_int8_sum(M):
    d = 77
    bits = RNG.integers(0, 2, size=(M, d)).astype(np.uint8)
    packed = [O.pack_bits(b) for b in bits]
    vote = O.majority_vote_popcount(packed, d)
    assert vote.tolist() == brute_force_vote(bits.tolist())
    # Alg. 2 formulation: sign of the int8 sum of +-1 signs
    s = O.majority_vote_sum(O.decode_bits(bits))
    assert np.array_equal(O.decode_bits(vote), s)
    if M == 1:
        assert np.array_equal(vote, bits[0])
    if M % 2 == 1:
        comp = [O.pack_bits(1 - b) for b in bits]
        assert np.array_equal(O.majority_vote_popcount(comp, d), 1 - vote)


def test_vote_exhaustive_tiny():
    for M in (1, 2, 3, 4):
        for ballots in itertools.product([0, 1], repeat=M):
            packed = [O.pack_bits([b]) for b in ballots]
            got = int(O.majority_vote_popcount(packed, 1)[0])
            assert got == (1 if 2 * sum(ballots) >= M else 0)


def test_vote_even_tie_goes_to_plus():
    bits = np.array([[1, 0, 1, 0], [0, 1, 1, 0]], dtype=np.uint8)
    packed = [O.pack_bits(b) for b in bits]
    assert O.majority_vote_popcount(packed, 4).tolist() == [1, 1, 1, 0]
    assert O.majority_vote_sum(O.decode_bits(bits)).tolist() == [1, 1, 1, -1]


# ----------------------------------------------------------------------------- local polar / update
def test_local_polar_norm_and_bound():
    s = O.decode_bits(RNG.integers(0, 2, size=(6, 10))).astype(np.float64)
    assert O.frobenius_norm(s) == math.sqrt(60)
    d = O.local_polar(s, 5)
    assert np.allclose(d, O.newton_schulz(s / math.sqrt(60), 5), rtol=1e-13)
    assert np.linalg.norm(d, 2) <= 1 + 1e-12
    u, sv, vt = np.linalg.svd(s, full_matrices=False)
    assert np.allclose(d, (u * f_scalar(sv / math.sqrt(60), 5)) @ vt, rtol=1e-10, atol=1e-13)


def test_round_to_bf16_matches_torch_and_fixes_double_rounding():
    x32 = RNG.normal(size=4096).astype(np.float32) * np.float32(0.02)
    ours = O.round_to_bf16(x32.astype(np.float64))
    ref = torch.from_numpy(x32).to(torch.bfloat16).float().numpy()
    assert np.array_equal(ours, ref)
    # 1 + 2^-8 is a bf16 tie (between 1 and 1 + 2^-7); a float64 just below it must round down,
    # although float32 rounding alone would land exactly on the tie and then round to even (up? no: 1.0 is even)
    tie = 1.0 + 2.0 ** -8
    assert O.round_to_bf16(np.array([tie]))[0] == 1.0                        # tie -> even
    assert O.round_to_bf16(np.array([tie + 2.0 ** -40]))[0] == np.float32(1.0 + 2.0 ** -7)
    tie_odd = 1.0 + 3 * 2.0 ** -8                                             # between 1+2^-7 (odd) and 1+2^-6 (even)
    assert O.round_to_bf16(np.array([tie_odd]))[0] == np.float32(1.0 + 2.0 ** -6)
    assert O.round_to_bf16(np.array([tie_odd - 2.0 ** -40]))[0] == np.float32(1.0 + 2.0 ** -7)


def signum_reference_python(w, g, mom, beta, lr):
    """Textbook signSGD with momentum, scalar loops: m = beta m + (1-beta) g ; w -= lr * sign(m), sign(0)=+1."""
    new_w = [row[:] for row in w]
    new_m = [row[:] for row in mom]
    for i in range(len(w)):
        for j in range(len(w[0])):
            new_m[i][j] = beta * mom[i][j] + (1 - beta) * g[i][j]
            new_w[i][j] = w[i][j] - lr * (1.0 if new_m[i][j] >= 0 else -1.0)
    return new_w, new_m


def test_step_reduces_to_signum_for_single_worker_no_ns():
    spec = O.ParamSpec(4, 6, "matrix")
    cfg = O.OracleConfig(num_workers=1, momentum=0.9, lr=0.01, ns_steps=0, local_polar=False)
    st = O.init_state([spec], cfg)
    w = RNG.normal(size=(4, 6))
    mom_py = [[0.0] * 6 for _ in range(4)]
    w_py = w.tolist()
    for t in range(4):
        g = RNG.normal(size=(1, 4, 6))
        new_w, _ = O.step([spec], cfg, st, [w], [g])
        w_py, mom_py = signum_reference_python(w_py, g[0].tolist(), mom_py, 0.9, 0.01)
        w = new_w[0]
        assert np.allclose(w, np.array(w_py), rtol=0, atol=1e-15)
        assert np.allclose(st.mom[0][0], np.array(mom_py), rtol=1e-15)


def test_step_update_is_plus_minus_eta_and_plain_kind():
    for kind in ("matrix", "plain"):
        spec = O.ParamSpec(5, 8, kind)
        cfg = O.OracleConfig(num_workers=3, lr=0.125, ns_steps=3)
        st = O.init_state([spec], cfg)
        w = RNG.normal(size=(5, 8))
        g = RNG.normal(size=(3, 5, 8))
        new_w, tr = O.step([spec], cfg, st, [w], [g])
        delta = new_w[0] - w
        assert set(np.unique(np.round(delta / 0.125, 12)).tolist()) <= {-1.0, 1.0}
        assert np.array_equal(delta < 0, tr[0].vote_bits.reshape(5, 8) == 1)
        # the vote of the trace equals brute force over the per-worker bits
        assert tr[0].vote_bits.tolist() == brute_force_vote(tr[0].bits.tolist())
        if kind == "plain":
            assert np.array_equal(tr[0].bits, (tr[0].mom.reshape(3, -1) >= 0).astype(np.uint8))


def test_step_hands_weight_decay_to_the_momentum():
    """Alg. 2 "Apply weight decay" at step level: beta = 0 and a constant gradient give Mom = G + lambda W,
    worked by hand on a 2 x 2 plain parameter (so that no Newton-Schulz intervenes):
        W = [[1, -2], [4, 0.5]], G = [[0.5, 0.1], [-1.5, -0.1]], lambda = 0.25
        Mom = [[0.75, -0.4], [-0.5, 0.025]]  -> bits [[1, 0], [0, 1]]  -> W' = W - 0.5 * [[+1, -1], [-1, +1]].
    Without the decay term the signs of the entries (1,0) and (1,1) would flip."""
    spec = O.ParamSpec(2, 2, "plain")
    cfg = O.OracleConfig(num_workers=2, momentum=0.0, lr=0.5, ns_steps=0, weight_decay=0.25)
    st = O.init_state([spec], cfg)
    w = np.array([[1.0, -2.0], [4.0, 0.5]])
    g = np.array([[0.5, 0.1], [-1.5, -0.1]])
    new_w, tr = O.step([spec], cfg, st, [w], [np.stack([g, g])])
    assert np.allclose(tr[0].mom[0], np.array([[0.75, -0.4], [-0.5, 0.025]]), rtol=1e-15, atol=1e-17)
    assert np.array_equal(tr[0].mom[1], tr[0].mom[0]) and np.array_equal(st.mom[0], tr[0].mom)
    assert tr[0].vote_bits.tolist() == [1, 0, 0, 1]
    assert np.array_equal(new_w[0], np.array([[0.5, -1.5], [4.5, 0.0]]))
    # matrix kind, K = 3: the decayed momentum is what enters PolarNS
    spec_m = O.ParamSpec(2, 2, "matrix")
    cfg_m = O.OracleConfig(num_workers=1, momentum=0.0, lr=0.5, ns_steps=3, weight_decay=0.25)
    _, tr_m = O.step([spec_m], cfg_m, O.init_state([spec_m], cfg_m), [w], [g[None]])
    u, sv, vt = np.linalg.svd(np.array([[0.75, -0.4], [-0.5, 0.025]]))
    expect = (u * f_scalar(sv / math.sqrt(np.sum(sv ** 2)), 3)) @ vt
    assert np.allclose(tr_m[0].polar[0], expect, rtol=1e-12, atol=1e-15)


def test_step_matrix_sign_is_scale_invariant_and_eq2_scale():
    spec = O.ParamSpec(6, 4, "matrix")
    w = RNG.normal(size=(6, 4))
    g = RNG.normal(size=(2, 6, 4))
    outs = []
    for scale in (1.0, 1e-6):
        cfg = O.OracleConfig(num_workers=2, lr=0.5, ns_steps=5)
        st = O.init_state([spec], cfg)
        _, tr = O.step([spec], cfg, st, [w], [g * scale])
        outs.append(tr[0].bits)
    assert np.array_equal(outs[0], outs[1])
    cfg = O.OracleConfig(num_workers=2, lr=0.5, ns_steps=5, update_scale=1)
    st = O.init_state([spec], cfg)
    new_w, tr = O.step([spec], cfg, st, [w], [g])
    assert np.allclose(np.abs(new_w[0] - w), 0.5 / math.sqrt(24), rtol=1e-12)
    assert abs(O.frobenius_norm(tr[0].direction) - 1.0) < 1e-12      # ||D||_F = 1 (Eq. 2)


def test_step_local_polar_direction():
    spec = O.ParamSpec(8, 5, "matrix")
    cfg = O.OracleConfig(num_workers=4, lr=0.1, ns_steps=5, local_polar=True)
    st = O.init_state([spec], cfg)
    w = RNG.normal(size=(8, 5))
    g = RNG.normal(size=(4, 8, 5))
    new_w, tr = O.step([spec], cfg, st, [w], [g])
    s_bar = O.decode_bits(tr[0].vote_bits).reshape(8, 5).astype(np.float64)
    u, sv, vt = np.linalg.svd(s_bar, full_matrices=False)
    expect_d = (u * f_scalar(sv / math.sqrt(40), 5)) @ vt
    assert np.allclose(tr[0].direction, expect_d, rtol=1e-10, atol=1e-13)
    assert np.allclose(new_w[0], w - 0.1 * expect_d, rtol=1e-12, atol=1e-15)
    # override path: feeding another vote changes the direction accordingly
    flipped = 1 - tr[0].vote_bits
    tr2 = O.step_param(spec, cfg, np.zeros((4, 8, 5)), w, g, vote_bits_override=flipped)
    assert np.allclose(tr2.direction, -expect_d, rtol=1e-10, atol=1e-13)


def test_muon_step_direction_is_the_svd_form_of_the_mean_gradient():
    """Full-precision Muon (Sec. 5.1's comparison optimizer; Alg. 1 without the sign): with beta = 0 the direction is
    PolarNS of the workers' mean gradient, whose K-step closed form comes from a float64 SVD; with singular values in
    the band where the iteration has converged it is the polar factor U V^T itself."""
    rng = np.random.default_rng(7)
    spec = O.ParamSpec(6, 9, "matrix")
    cfg = O.OracleConfig(num_workers=3, momentum=0.0, lr=0.25, ns_steps=4)
    w = rng.normal(size=(6, 9))
    g = rng.normal(size=(3, 6, 9))
    mom, u, new_w = O.muon_step_param(spec, cfg, np.zeros((6, 9)), w, g)
    mean = (g[0] + g[1] + g[2]) / 3.0
    assert np.allclose(mom, mean, rtol=1e-15, atol=1e-17)
    uu, sv, vt = np.linalg.svd(mean, full_matrices=False)
    expect = (uu * f_scalar(sv / math.sqrt(np.sum(sv ** 2)), 4)) @ vt
    assert np.allclose(u, expect, rtol=1e-10, atol=1e-13)
    assert np.allclose(new_w, w - 0.25 * expect, rtol=1e-12, atol=1e-15)
    # momentum carried over: second step from the returned momentum, beta = 0.9, weight decay coupled
    cfg2 = O.OracleConfig(num_workers=3, momentum=0.9, lr=0.25, ns_steps=0, weight_decay=0.5)
    mom2, u2, _ = O.muon_step_param(spec, cfg2, mom, w, g)
    assert np.allclose(mom2, 0.9 * mean + 0.1 * (mean + 0.5 * w), rtol=1e-14)
    assert np.allclose(u2, mom2 / np.linalg.norm(mom2), rtol=1e-14)          # K = 0: the normalised momentum
    # converged band: a rank-2 gradient with singular values (0.8, 0.6) of the normalised matrix -> U V^T
    q1, _ = np.linalg.qr(rng.normal(size=(7, 2)))
    q2, _ = np.linalg.qr(rng.normal(size=(5, 2)))
    x = 3.0 * (q1 * np.array([0.8, 0.6])) @ q2.T
    cfg3 = O.OracleConfig(num_workers=1, momentum=0.0, lr=1.0, ns_steps=8)
    _, u3, w3 = O.muon_step_param(O.ParamSpec(7, 5, "matrix"), cfg3, np.zeros((7, 5)), np.zeros((7, 5)), x[None])
    assert np.linalg.norm(u3 - q1 @ q2.T, 2) <= 0.64 ** (2 ** 8) + 1e-12
    assert np.allclose(w3, -(q1 @ q2.T), atol=1e-10)
    # short-side route gives the same step; a plain parameter is refused
    _, u_s, _ = O.muon_step_param(spec, cfg, np.zeros((6, 9)), w, g, short_side=True)
    assert np.allclose(u_s, u, rtol=1e-10, atol=1e-13)
    with pytest.raises(ValueError):
        O.muon_step_param(O.ParamSpec(1, 9, "plain"), cfg, np.zeros((1, 9)), w[:1], g[:, :1])


# --------------------------------------------------------------------------- #
# Alg. 5 (PowerIter) and Alg. 4 with scale = spectral
# --------------------------------------------------------------------------- #
def test_power_iter_rank_one_is_exact_after_one_round():
    # X = a b^T has one non-zero singular value ||a|| ||b||; X^T X v is parallel to b for any v not orthogonal to b.
    rng = np.random.default_rng(3)
    a, b, v0 = rng.standard_normal(7), rng.standard_normal(11), rng.standard_normal(11)
    x = np.outer(a, b)
    want = np.linalg.norm(a) * np.linalg.norm(b)
    assert abs(O.power_iter(x, 1, 1e-300, v0) - want) <= 1e-12 * want
    assert abs(O.power_iter(x, 4, 1e-300, v0) - want) <= 1e-12 * want
    # P = 0: just ||X v0 / ||v0|| || = ||a|| |b . v0| / ||v0||
    want0 = np.linalg.norm(a) * abs(b @ v0) / np.linalg.norm(v0)
    assert abs(O.power_iter(x, 0, 1e-300, v0) - want0) <= 1e-12 * want0


def test_power_iter_diagonal_closed_form():
    # X = diag(s): after P rounds v is proportional to s^(2P) * v0, so the estimate is ||s^(2P+1) v0|| / ||s^(2P) v0||.
    s = np.array([3.0, 2.0, 1.0, 0.5])
    v0 = np.array([0.2, -0.7, 1.1, 0.4])
    for P in (0, 1, 2, 5):
        want = np.linalg.norm(s ** (2 * P + 1) * v0) / np.linalg.norm(s ** (2 * P) * v0)
        assert abs(O.power_iter(np.diag(s), P, 1e-300, v0) - want) <= 1e-12 * want


def test_power_iter_is_a_lower_bound_that_rises_to_sigma_max():
    rng = np.random.default_rng(4)
    x = rng.standard_normal((9, 14))
    v0 = rng.standard_normal(14)
    smax = np.linalg.svd(x, compute_uv=False)[0]
    est = [O.power_iter(x, P, 1e-300, v0) for P in (0, 1, 2, 4, 8, 400)]
    assert all(e <= smax * (1 + 1e-12) for e in est)                    # ||X v|| <= sigma_max for ||v|| <= 1
    assert all(b >= a * (1 - 1e-12) for a, b in zip(est, est[1:]))      # Rayleigh quotients of (X^T X)^P v0 rise
    assert abs(est[-1] - smax) <= 1e-9 * smax                           # and converge (spectral gap)
    # a transposed operand or a missing normalisation would break either the bound or the limit
    assert abs(O.power_iter(x.T, 400, 1e-300, rng.standard_normal(9)) - smax) <= 1e-9 * smax


def test_power_iter_eps_enters_as_a_sum_and_zero_matrix_is_safe():
    v0 = np.array([3.0, 4.0])
    x = np.eye(2)
    # v <- v0 / (5 + eps): with eps = 5 the start vector has norm 1/2; one round renormalises with (1/2 + 5)
    got = O.power_iter(x, 0, 5.0, v0)
    assert abs(got - 0.5) <= 1e-15
    assert O.power_iter(np.zeros((3, 2)), 2, 1e-12, v0) == 0.0
    assert np.all(O.polar_ns(np.zeros((3, 2)), 3, 1e-12, sigma=0.0) == 0.0)


def test_spectral_scaling_reaches_the_polar_factor():
    # With sigma ~ ||X||_op the singular values of Y0 lie in (0, ~1]; for a well-conditioned matrix K = 5
    # cubic steps bring all of them to 1 within the theorem's bound.
    rng = np.random.default_rng(5)
    u, _ = np.linalg.qr(rng.standard_normal((6, 6)))
    v, _ = np.linalg.qr(rng.standard_normal((10, 10)))
    sv = np.array([1.0, 0.95, 0.9, 0.85, 0.8, 0.75])
    x = 3.7 * (u * sv) @ v[:, :6].T
    sigma = O.power_iter(x, 200, 1e-12, rng.standard_normal(10))
    assert abs(sigma - 3.7) <= 1e-9
    y = O.polar_ns(x, 5, 1e-12, sigma=sigma)
    polar = u @ v[:, :6].T
    rho = 1.0 - 0.75 ** 2                                               # ||I - Y0^T Y0||_op on the row space
    assert np.linalg.norm(y - polar, 2) <= rho ** (2 ** 5) + 1e-12
    # the step routes sigma through PowerIter when asked to
    cfg = O.OracleConfig(num_workers=1, ns_steps=5, ns_scale="spectral", power_iters=200)
    tr = O.step_param(O.ParamSpec(6, 10), cfg, np.zeros((1, 6, 10)), np.zeros((6, 10)), x[None] / (1 - cfg.momentum),
                      power_start=rng.standard_normal((1, 10)))
    assert np.linalg.norm(tr.polar[0] - polar, 2) <= 1e-6
