"""Pins for the CPU oracle: everything here checks the oracle against something other than
itself -- values the paper prints for its worked example, the plain definition evaluated by a
library routine (numpy / torch in float64), closed forms, invariants, brute force on tiny grids.
"""
import itertools
import os

import numpy as np
import pytest
import torch

GOLD = os.path.join(os.path.dirname(__file__), "golden")

# the paper's toy generators (Section "Pre-processing"): G_r = [I | P_r], G_c = [I | P_c]
P_R_TOY = np.array([[1, 1], [1, -1]], np.float32)
P_C_TOY = np.array([[1, 1], [1, 2]], np.float32)


def _toy_layer(orc, W, **kw):
    return orc.Layer(W, 2, 2, 2, 2, P_row=P_R_TOY, P_col=P_C_TOY, **kw)


def _rel(a, b):
    return float(np.max(np.abs(np.asarray(a, np.float64) - np.asarray(b, np.float64))) /
                 max(np.max(np.abs(np.asarray(b, np.float64))), 1e-300))


# ---------------------------------------------------------------------------------------------
# random numbers
# ---------------------------------------------------------------------------------------------

def test_philox_known_answers(orc):
    n = 0
    for line in open(os.path.join(GOLD, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        assert orc.philox(w[0:4], w[4:6]) == w[6:10]
        n += 1
    assert n == 3


def test_noise_is_unit_variance_scaled_by_sigma(orc):
    v = np.array([orc.noise(3, 1, 0, 7, 5, e, 10.0) for e in range(20000)], np.float64)
    assert abs(v.mean()) < 0.3                      # 3 sigma of the mean is 0.21
    assert abs(v.var() - 100.0) < 5.0
    # Irwin-Hall(12) support: |v| <= 6 sigma
    assert np.max(np.abs(v)) <= 60.0
    # the sample is a multiple of sigma * 2^-16 (integer until the last product)
    q = v / (10.0 / 65536.0)
    assert np.allclose(q, np.round(q), atol=1e-3)


def test_noise_streams_are_distinct(orc):
    base = orc.noise(0, 0, 0, 0, 0, 0, 1.0)
    others = [orc.noise(1, 0, 0, 0, 0, 0, 1.0), orc.noise(0, 1, 0, 0, 0, 0, 1.0),
              orc.noise(0, 0, 1, 0, 0, 0, 1.0), orc.noise(0, 0, 0, 1, 0, 0, 1.0),
              orc.noise(0, 0, 0, 0, 1, 0, 1.0), orc.noise(0, 0, 0, 0, 0, 1, 1.0)]
    assert len(set([base] + others)) == 7


def test_hit_frequency_and_exactly_one(orc):
    f = orc.make_fault(seed=5, layer=2, mode=orc.FAULT_BERNOULLI, p=0.05)
    hits = sum(orc.node_hit(f, 0, it, node, node, 16) for it in range(2000) for node in range(16))
    assert abs(hits / 32000.0 - 0.05) < 0.005
    f1 = orc.make_fault(seed=5, layer=2, mode=orc.FAULT_EXACTLY_ONE)
    victims = []
    for it in range(300):
        h = [orc.node_hit(f1, 1, it, 99, a, 6) for a in range(6)]
        assert sum(h) == 1
        victims.append(h.index(True))
    assert set(victims) == set(range(6))            # every node gets picked eventually
    f0 = orc.make_fault(mode=orc.FAULT_NONE)
    assert not any(orc.node_hit(f0, 0, it, 0, 0, 4) for it in range(50))


# ---------------------------------------------------------------------------------------------
# codes
# ---------------------------------------------------------------------------------------------

def test_toy_generators_are_mds_and_annihilated_by_h():
    for P in (P_R_TOY, P_C_TOY):
        P = P.astype(np.float64)
        G = np.hstack([np.eye(2), P])
        H = np.hstack([P.T, -np.eye(2)])
        assert np.all(H @ G.T == 0)
        for cols in itertools.combinations(range(4), 2):
            assert abs(np.linalg.det(G[:, cols])) > 1e-12
        # Spark(H) = 2t + 1 = 3: every pair of columns independent, some triple dependent
        for cols in itertools.combinations(range(4), 2):
            assert np.linalg.matrix_rank(H[:, cols]) == 2
        assert any(np.linalg.matrix_rank(H[:, cols]) < 3 for cols in itertools.combinations(range(4), 3))


def test_node_count_matches_theorem_1(orc):
    # P^ = P + 2 (m + n) t populated nodes for r = 2t parity rows and columns
    for (m, n, t) in [(2, 2, 1), (3, 2, 1), (4, 4, 1), (2, 3, 2)]:
        W = np.zeros((m * 2, n * 2), np.float32)
        lay = orc.Layer(W, m, n, 2 * t, 2 * t, P_row=np.random.default_rng(0).standard_normal((m, 2 * t)),
                        P_col=np.random.default_rng(1).standard_normal((n, 2 * t)))
        count = sum(lay.has_node(i, j) for i in range(lay.M) for j in range(lay.Nn))
        assert count == m * n + 2 * (m + n) * t
        with pytest.raises(IndexError):
            lay.block(lay.M - 1, lay.Nn - 1)        # corner: no node


# ---------------------------------------------------------------------------------------------
# initial encoding (Claim 1)
# ---------------------------------------------------------------------------------------------

def test_encoding_reproduces_the_papers_toy_grid(orc):
    k = 3
    primes = {"W00": 2.0, "W01": 3.0, "W10": 5.0, "W11": 7.0}
    eye = np.eye(k, dtype=np.float32)
    W = np.block([[primes["W00"] * eye, primes["W01"] * eye], [primes["W10"] * eye, primes["W11"] * eye]])
    lay = _toy_layer(orc, W)
    seen = 0
    for line in open(os.path.join(GOLD, "toy_example.txt")):
        t = line.split()
        if not t or t[0] in "#SXD":
            continue
        i, j = int(t[0]), int(t[1])
        if t[2] == "x":
            assert not lay.has_node(i, j)
        else:
            c = [float(x) for x in t[2:6]]
            want = (c[0] * 2.0 + c[1] * 3.0 + c[2] * 5.0 + c[3] * 7.0) * eye
            assert np.array_equal(lay.block(i, j), want)
        seen += 1
    assert seen == 16


@pytest.mark.parametrize("m,n,rr,rc,no,ni", [(2, 2, 2, 2, 8, 12), (3, 2, 1, 1, 9, 8), (4, 4, 1, 1, 10, 18),
                                             (2, 3, 2, 1, 6, 9), (2, 2, 0, 0, 4, 4)])
def test_encoding_equals_kronecker_definition(orc, m, n, rr, rc, no, ni):
    rng = np.random.default_rng(11)
    W = rng.standard_normal((no, ni)).astype(np.float32)
    Pr = rng.standard_normal((m, rr)).astype(np.float32)
    Pc = rng.standard_normal((n, rc)).astype(np.float32)
    lay = orc.Layer(W, m, n, rr, rc, P_row=Pr, P_col=Pc)
    br, bc = lay.b_r, lay.b_c
    Wp = np.zeros((br * m, bc * n))
    Wp[:no, :ni] = W
    Gr = np.hstack([np.eye(m), Pr.astype(np.float64)])
    Gc = np.hstack([np.eye(n), Pc.astype(np.float64)])
    full = np.kron(Gr.T, np.eye(br)) @ Wp @ np.kron(Gc, np.eye(bc))
    for i in range(lay.M):
        for j in range(lay.Nn):
            if not lay.has_node(i, j):
                continue
            want = full[i * br:(i + 1) * br, j * bc:(j + 1) * bc]
            got = lay.block(i, j)
            assert np.allclose(got, want, rtol=2e-7, atol=1e-7)
            # inner checksums are column / row sums of the stored block
            assert np.allclose(lay.u(i, j)[0], got.astype(np.float64).sum(0), rtol=1e-6, atol=1e-6)
            assert np.allclose(lay.v(i, j)[0], got.astype(np.float64).sum(1), rtol=1e-6, atol=1e-6)


def test_inner_checksum_slices(orc):
    rng = np.random.default_rng(2)
    W = rng.standard_normal((16, 8)).astype(np.float32)
    lay = orc.Layer(W, 2, 2, 1, 1, check_rows=4, check_cols=2)
    assert (lay.T, lay.ns, lay.Tc, lay.nsc) == (4, 2, 2, 2)
    blk = lay.block(2, 1).astype(np.float64)
    assert np.allclose(lay.u(2, 1), blk.reshape(2, 4, 4).sum(1), rtol=1e-6, atol=1e-6)
    assert np.allclose(lay.v(2, 1), blk.reshape(8, 2, 2).sum(2).T, rtol=1e-6, atol=1e-6)


# ---------------------------------------------------------------------------------------------
# vector encoding, products
# ---------------------------------------------------------------------------------------------

def test_vector_encoding_matches_the_toy_example(orc):
    rng = np.random.default_rng(3)
    W = rng.standard_normal((6, 4)).astype(np.float32)
    lay = _toy_layer(orc, W)
    x = rng.standard_normal((1, 4)).astype(np.float32)
    d = rng.standard_normal((1, 6)).astype(np.float32)
    xt = lay.encode_x(x)[0].reshape(4, 2)
    dt = lay.encode_delta(d)[0].reshape(4, 3)
    x0, x1 = x[0, :2], x[0, 2:]
    d0, d1 = d[0, :3], d[0, 3:]
    coef = {}
    for line in open(os.path.join(GOLD, "toy_example.txt")):
        t = line.split()
        if t and t[0] in "XD":
            coef[(t[0], int(t[1]))] = (float(t[2]), float(t[3]))
    assert np.array_equal(xt[0], x0) and np.array_equal(xt[1], x1)
    assert np.array_equal(dt[0], d0) and np.array_equal(dt[1], d1)
    for k in (2, 3):
        a, b = coef[("X", k)]
        assert np.allclose(xt[k], a * x0 + b * x1, rtol=1e-6)
        a, b = coef[("D", k)]
        assert np.allclose(dt[k], a * d0 + b * d1, rtol=1e-6)


def test_toy_forward_outputs_and_subset_consistency(orc):
    """Row outputs are [s0, s1, s0+s1, s0-s1]; with s1 corrupted only {s0, s~2, s~3} is
    consistent and s1 = s~2 - s0 (the paper's four subset checks)."""
    rng = np.random.default_rng(4)
    W = rng.standard_normal((8, 6)).astype(np.float32)
    x = rng.standard_normal((1, 6)).astype(np.float32)
    lay = _toy_layer(orc, W)
    Y = lay.forward_products(x)                      # (n, M, b_r, 1)
    rows = Y.astype(np.float64).sum(axis=0)[:, :, 0]  # (M, b_r): sum over j
    s = (W.astype(np.float64) @ x[0].astype(np.float64)).reshape(2, 4)
    coef = {}
    for line in open(os.path.join(GOLD, "toy_example.txt")):
        t = line.split()
        if t and t[0] == "S":
            coef[int(t[1])] = (float(t[2]), float(t[3]))
    for i in range(4):
        a, b = coef[i]
        assert np.allclose(rows[i], a * s[0] + b * s[1], rtol=1e-5, atol=1e-5)
    out = rows.copy()
    out[1] += rng.standard_normal(4) * 10.0          # s1 -> s1 + e1
    tol = 1e-4
    checks = {
        (0, 1, 2): np.max(np.abs(out[0] + out[1] - out[2])) < tol,
        (0, 2, 3): np.max(np.abs(2 * out[0] - (out[2] + out[3]))) < tol,
        (0, 1, 3): np.max(np.abs(out[0] - out[1] - out[3])) < tol,
        (1, 2, 3): np.max(np.abs(2 * out[1] - (out[2] - out[3]))) < tol,
    }
    assert checks == {(0, 1, 2): False, (0, 2, 3): True, (0, 1, 3): False, (1, 2, 3): False}
    assert np.allclose(out[2] - out[0], s[1], rtol=1e-5, atol=1e-5)


@pytest.mark.parametrize("B", [1, 3])
@pytest.mark.parametrize("m,n,rr,rc,no,ni", [(2, 2, 2, 2, 8, 12), (4, 4, 1, 1, 10, 18), (1, 1, 0, 0, 5, 7),
                                             (2, 3, 2, 1, 6, 9)])
def test_decoded_products_equal_plain_products(orc, B, m, n, rr, rc, no, ni):
    """s = W x and c = W^T delta (proof of Lemma 2: the node outputs are a codeword of s)."""
    rng = np.random.default_rng(5)
    W = rng.standard_normal((no, ni)).astype(np.float32)
    X = rng.standard_normal((B, ni)).astype(np.float32)
    D = rng.standard_normal((B, no)).astype(np.float32)
    lay = orc.Layer(W, m, n, rr, rc, P_row=rng.standard_normal((m, rr)), P_col=rng.standard_normal((n, rc)))
    S, rep = lay.forward(X)
    assert rep.decisions()[:5] == (0, 0, 0, 0, 0)
    assert _rel(S, X.astype(np.float64) @ W.astype(np.float64).T) < 1e-6
    Cc, rep = lay.backward_update(D, X, 0.0)
    assert rep.decisions()[:5] == (0, 0, 0, 0, 0)
    assert _rel(Cc, D.astype(np.float64) @ W.astype(np.float64)) < 1e-6


def test_node_outputs_form_a_codeword(orc):
    rng = np.random.default_rng(6)
    m, n, r = 3, 2, 2
    W = rng.standard_normal((9, 8)).astype(np.float32)
    Pr = rng.standard_normal((m, r)).astype(np.float32)
    Pc = rng.standard_normal((n, r)).astype(np.float32)
    lay = orc.Layer(W, m, n, r, r, P_row=Pr, P_col=Pc)
    X = rng.standard_normal((2, 8)).astype(np.float32)
    D = rng.standard_normal((2, 9)).astype(np.float32)
    Y = lay.forward_products(X).astype(np.float64)   # (n, M, b_r, B)
    H = np.hstack([Pr.T.astype(np.float64), -np.eye(r)])
    assert np.max(np.abs(np.einsum("qk,jkrb->jqrb", H, Y))) < 1e-5
    Z = lay.backward_products(D).astype(np.float64)  # (m, Nn, b_c, B)
    Hc = np.hstack([Pc.T.astype(np.float64), -np.eye(r)])
    assert np.max(np.abs(np.einsum("qk,ikcb->iqcb", Hc, Z))) < 1e-5
    # un-reduced node outputs against the plain block products
    Wd = W.astype(np.float64)
    for j in range(n):
        for i in range(m):
            want = Wd[i * 3:(i + 1) * 3, j * 4:(j + 1) * 4] @ X[:, j * 4:(j + 1) * 4].astype(np.float64).T
            assert np.allclose(Y[j, i], want, rtol=1e-6, atol=1e-6)
    for i in range(m):
        for j in range(n):
            want = Wd[i * 3:(i + 1) * 3, j * 4:(j + 1) * 4].T @ D[:, i * 3:(i + 1) * 3].astype(np.float64).T
            assert np.allclose(Z[i, j], want, rtol=1e-6, atol=1e-6)


# ---------------------------------------------------------------------------------------------
# coded update (step O3)
# ---------------------------------------------------------------------------------------------

def test_update_identity_for_block_0_3(orc):
    """W~_{0,3} + eta d0 x~3^T = (W00 + eta d0 x0^T) + 2 (W01 + eta d0 x1^T)."""
    rng = np.random.default_rng(7)
    W = rng.standard_normal((6, 8)).astype(np.float32)
    x = rng.standard_normal((1, 8)).astype(np.float32)
    d = rng.standard_normal((1, 6)).astype(np.float32)
    lay = _toy_layer(orc, W)
    lay.update(d, x, 0.05)
    Wd, xd, dd = W.astype(np.float64), x[0].astype(np.float64), d[0].astype(np.float64)
    new = Wd + 0.05 * np.outer(dd, xd)
    want = new[0:3, 0:4] + 2.0 * new[0:3, 4:8]
    assert np.allclose(lay.block(0, 3), want, rtol=1e-6, atol=1e-6)
    assert np.allclose(lay.block(0, 0), new[0:3, 0:4], rtol=1e-6, atol=1e-6)
    assert np.allclose(lay.block(3, 1), new[0:3, 4:8] - new[3:6, 4:8], rtol=1e-6, atol=1e-6)


@pytest.mark.parametrize("B", [1, 4])
def test_update_preserves_the_code_and_follows_uncoded_sgd(orc, B):
    rng = np.random.default_rng(8)
    m, n = 2, 3
    W = (rng.standard_normal((8, 9)) / 3).astype(np.float32)
    lay = orc.Layer(W, m, n, 2, 1, P_row=rng.standard_normal((m, 2)), P_col=rng.standard_normal((n, 1)),
                    check_rows=2, check_cols=3)
    shadow = W.copy()
    for it in range(30):
        X = rng.standard_normal((B, 9)).astype(np.float32)
        D = (rng.standard_normal((B, 8)) / B).astype(np.float32)
        Cc, rep = lay.backward_update(D, X, 0.01)
        assert _rel(Cc, D.astype(np.float64) @ shadow.astype(np.float64)) < 1e-6   # pre-update weights
        shadow = (shadow.astype(np.float64) + np.float64(np.float32(0.01)) *
                  (D.astype(np.float64).T @ X.astype(np.float64))).astype(np.float32)
        assert rep.status == orc.CLEAN
    assert np.array_equal(lay.decode_weights(), shadow)      # same arithmetic on the same values
    assert lay.check_invariance() < 5e-6


def test_corrupted_stored_block_breaks_invariance_and_is_detected(orc):
    rng = np.random.default_rng(9)
    W = rng.standard_normal((8, 8)).astype(np.float32)
    lay = orc.Layer(W, 2, 2, 1, 1)
    assert lay.check_invariance() < 1e-6
    blk = lay.block(1, 0)
    blk[2, 1] += 3.0
    lay.set_block(1, 0, blk)
    assert lay.check_invariance() > 1e-2
    X = rng.standard_normal((1, 8)).astype(np.float32)
    S, rep = lay.forward(X)
    # an erroneous stored sub-matrix shows up as noise in that node's next output
    assert rep.n_detected_cw == 1 and rep.flagged_mask[0] == 0b010
    assert _rel(S, X.astype(np.float64) @ W.astype(np.float64).T) < 1e-5


# ---------------------------------------------------------------------------------------------
# detection, location, correction
# ---------------------------------------------------------------------------------------------

def _corrupt(Y, cw, node, rng, sigma=10.0):
    Y[cw, node] += (rng.standard_normal(Y[cw, node].shape) * sigma).astype(np.float32)


@pytest.mark.parametrize("r", [1, 2])
@pytest.mark.parametrize("phase", [0, 1])
def test_all_hit_patterns_on_tiny_grids(orc, r, phase):
    """Brute force over every pattern of corrupted nodes in a 2x2 data grid with r parities:
    <= r hits per codeword are located and corrected, more are detected and fall back."""
    rng = np.random.default_rng(10 + r)
    W = rng.standard_normal((8, 8)).astype(np.float32)
    X = rng.standard_normal((2, 8)).astype(np.float32)
    D = rng.standard_normal((2, 8)).astype(np.float32)
    Pr = rng.standard_normal((2, r)) if r > 1 else None
    Pc = rng.standard_normal((2, r)) if r > 1 else None
    lay = orc.Layer(W, 2, 2, r, r, P_row=Pr, P_col=Pc)
    clean = lay.forward_products(X) if phase == 0 else lay.backward_products(D)
    V = X if phase == 0 else D
    K = 2 + r
    for pat0 in range(1 << K):
        for pat1 in (0, 1 << (K - 1), 0b11):
            Y = clean.copy()
            inj = [pat0, pat1]
            for cw in range(2):
                for k in range(K):
                    if (inj[cw] >> k) & 1:
                        _corrupt(Y, cw, k, rng)
            rep = lay.detect_decode(phase, Y, V, Yclean=clean, injected=inj + [0] * 62)
            for cw in range(2):
                hits = bin(inj[cw]).count("1")
                assert ((rep.detected_mask >> cw) & 1) == (1 if hits else 0)
                assert rep.flagged_mask[cw] == inj[cw]
            n_bad = sum(bin(p).count("1") > r for p in inj)
            assert rep.n_fallback_cw == n_bad
            want_status = orc.FALLBACK if n_bad else (orc.CORRECTED if any(inj) else orc.CLEAN)
            assert rep.status == want_status
            assert _rel(Y, clean) < 1e-5
            if any(inj):
                assert rep.min_margin_hit > 10.0
            assert rep.max_margin_clean < 0.1


def test_without_clean_copy_uncorrectable_is_reported_failed(orc):
    rng = np.random.default_rng(12)
    W = rng.standard_normal((8, 8)).astype(np.float32)
    X = rng.standard_normal((1, 8)).astype(np.float32)
    lay = orc.Layer(W, 2, 2, 1, 1)
    Y = lay.forward_products(X)
    _corrupt(Y, 1, 0, rng)
    _corrupt(Y, 1, 2, rng)
    rep = lay.detect_decode(0, Y, X)
    assert rep.status == orc.FAILED and rep.n_fallback_cw == 1 and rep.detected_mask == 0b10


def test_syndrome_only_location_corrects_any_single_error(orc):
    """Paper-exact blind decoding (t = 1, r = 2t = 2): every single erroneous output is located
    from the syndrome alone; two errors are detected but not corrected (Lemma 2)."""
    rng = np.random.default_rng(13)
    W = rng.standard_normal((9, 8)).astype(np.float32)
    X = rng.standard_normal((1, 8)).astype(np.float32)
    lay = orc.Layer(W, 3, 2, 2, 2, P_row=rng.standard_normal((3, 2)), P_col=P_C_TOY,
                    locate_mode=orc.LOCATE_SYNDROME)
    clean = lay.forward_products(X)
    for k in range(5):
        Y = clean.copy()
        _corrupt(Y, 0, k, rng)
        rep = lay.detect_decode(0, Y, X, Yclean=clean)
        assert rep.status == orc.CORRECTED and rep.flagged_mask[0] == 1 << k and rep.flagged_mask[1] == 0
        assert _rel(Y, clean) < 1e-5
    Y = clean.copy()
    _corrupt(Y, 1, 0, rng)
    _corrupt(Y, 1, 3, rng)
    rep = lay.detect_decode(0, Y, X, Yclean=clean)
    assert rep.status == orc.FALLBACK and rep.detected_mask == 0b10 and rep.n_fallback_cw == 1


@pytest.mark.parametrize("r", [2, 3, 4])
def test_joint_location_finds_the_support_a_brute_force_search_finds(orc, r):
    """locate_mode JOINT (supports of up to r - 1 nodes, whole sub-vectors in error) against a search written
    with numpy's least squares: every support of every size is tried in the same order and the first one whose
    residual over all elements is below the threshold the report states is the answer; planted errors in up
    to r - 1 nodes are then decoded back to the clean products, r of them only detected."""
    rng = np.random.default_rng(40 + r)
    m, n = 4, 2
    W = rng.standard_normal((4 * 5, 2 * 3)).astype(np.float32)
    X = rng.standard_normal((2, 6)).astype(np.float32)
    P = rng.standard_normal((m, r))
    lay = orc.Layer(W, m, n, r, 1, P_row=P, locate_mode=orc.LOCATE_JOINT)
    clean = lay.forward_products(X)
    K = m + r
    H = np.concatenate([P.T, -np.eye(r)], axis=1)                      # r x K, H G_r^T = 0
    for count in range(1, r + 1):
        for trial in range(4):
            support = sorted(rng.choice(K, size=count, replace=False).tolist())
            Y = clean.copy()
            for k in support:
                _corrupt(Y, 1, k, rng)
            syn = H @ Y[1].reshape(K, -1).astype(np.float64)           # r x n_el
            rep = lay.detect_decode(0, Y, X)
            # the independent search (any threshold between the rounding level and the planted errors separates
            # a support that fits from one that does not)
            tau, found = 1e-3, None
            for size in range(1, min(r - 1, 3) + 1):
                for F in itertools.combinations(range(K), size):
                    HF = H[:, list(F)]
                    resid = syn - HF @ np.linalg.lstsq(HF, syn, rcond=None)[0]
                    if np.max(np.abs(resid)) <= tau:
                        found = list(F)
                        break
                if found:
                    break
            if count <= min(r - 1, 3):
                assert found == support
                assert rep.status == orc.CORRECTED and rep.flagged_mask[1] == sum(1 << k for k in support)
                assert rep.flagged_mask[0] == 0 and _rel(Y, clean) < 1e-4
            else:
                assert found is None
                assert rep.status == orc.FAILED and rep.detected_mask == 0b10


def test_syndrome_and_node_check_agree_on_single_hits(orc):
    rng = np.random.default_rng(14)
    m = n = 4
    W = rng.standard_normal((16, 16)).astype(np.float32)
    D = rng.standard_normal((3, 16)).astype(np.float32)
    Pr, Pc = rng.standard_normal((m, 2)), rng.standard_normal((n, 2))
    a = orc.Layer(W, m, n, 2, 2, P_row=Pr, P_col=Pc, locate_mode=orc.LOCATE_SYNDROME)
    b = orc.Layer(W, m, n, 2, 2, P_row=Pr, P_col=Pc, locate_mode=orc.LOCATE_NODECHECK)
    clean = a.backward_products(D)
    for cw in range(m):
        for k in range(n + 2):
            Ya, Yb = clean.copy(), clean.copy()
            _corrupt(Ya, cw, k, np.random.default_rng(100 + k))
            _corrupt(Yb, cw, k, np.random.default_rng(100 + k))
            ra = a.detect_decode(1, Ya, D, Yclean=clean)
            rb = b.detect_decode(1, Yb, D, Yclean=clean)
            assert ra.flagged_mask[cw] == rb.flagged_mask[cw] == 1 << k
            assert ra.status == rb.status == orc.CORRECTED


def test_locate_none_detects_and_falls_back(orc):
    rng = np.random.default_rng(15)
    W = rng.standard_normal((8, 8)).astype(np.float32)
    X = rng.standard_normal((1, 8)).astype(np.float32)
    lay = orc.Layer(W, 2, 2, 1, 1, locate_mode=orc.LOCATE_NONE)
    clean = lay.forward_products(X)
    Y = clean.copy()
    _corrupt(Y, 0, 1, rng)
    rep = lay.detect_decode(0, Y, X, Yclean=clean)
    assert rep.status == orc.FALLBACK and rep.detected_mask == 1 and rep.flagged_mask[0] == 0
    assert np.array_equal(Y, clean)


def test_no_injection_means_no_detection_over_a_run(orc):
    from paper_1903_01042_b200 import workloads as wl
    cfg = wl.config("c1", scale=8)
    sp = cfg.layers[0]
    lay = orc.Layer(wl.weights(sp.n_out, sp.n_in), sp.m, sp.n, sp.r_row, sp.r_col)
    net = orc.Net([lay])
    worst = 0.0
    for it in range(60):
        x, t = wl.layer_inputs(cfg, it)
        loss, out, reps = net.step(x, t, cfg.lr, None, it)
        assert all(r.status == orc.CLEAN and r.n_detected_cw == 0 for r in reps)
        worst = max(worst, max(r.max_margin_clean for r in reps))
    assert worst < 0.1                                # >= 10x margin below the thresholds


def test_injected_run_flags_exactly_the_injected_nodes(orc):
    from paper_1903_01042_b200 import workloads as wl
    cfg = wl.config("c1", scale=8)
    sp = cfg.layers[0]
    W = wl.weights(sp.n_out, sp.n_in)
    lay = orc.Layer(W, sp.m, sp.n, sp.r_row, sp.r_col)
    net = orc.Net([lay])
    shadow = W.copy()
    f = orc.make_fault(seed=0, layer=0, mode=orc.FAULT_EXACTLY_ONE, sigma=10.0)
    for it in range(40):
        x, t = wl.layer_inputs(cfg, it)
        loss, out, reps = net.step(x, t, cfg.lr, [f], it)
        for r in reps:
            assert r.status == orc.CORRECTED and r.n_detected_cw == 1 and r.n_flagged_nodes == 1
            assert tuple(r.flagged_mask) == tuple(r.injected_mask)
            assert r.min_margin_hit > 10.0 and r.max_margin_clean < 0.1
        # fault-free uncoded shadow run (plain SGD on the mean-squared error)
        s = shadow.astype(np.float64) @ x[0].astype(np.float64)
        d = (2.0 * (t[0].astype(np.float64) - s) / s.size).astype(np.float32)
        shadow = (shadow.astype(np.float64) + np.float64(np.float32(cfg.lr)) *
                  np.outer(d.astype(np.float64), x[0].astype(np.float64))).astype(np.float32)
    assert _rel(lay.decode_weights(), shadow) < 1e-4
    assert lay.check_invariance() < 1e-5


# ---------------------------------------------------------------------------------------------
# whole-network step against torch autograd (float64)
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("loss_kind", ["mse", "ce"])
def test_step_matches_autograd_sgd(orc, loss_kind):
    rng = np.random.default_rng(16)
    dims = [12, 16, 8, 10]
    B = 3
    Ws = [(rng.standard_normal((dims[l + 1], dims[l])) / np.sqrt(dims[l])).astype(np.float32) for l in range(3)]
    layers = [orc.Layer(Ws[l], 4, 4, 1, 1) for l in range(3)]      # the 10-row head is padded to 12
    net = orc.Net(layers, activation=orc.ACT_RELU,
                  loss=orc.LOSS_MSE_MEAN if loss_kind == "mse" else orc.LOSS_SOFTMAX_CE)
    tw = [torch.tensor(w, dtype=torch.float64, requires_grad=True) for w in Ws]
    lr = 0.05
    for it in range(3):
        X = rng.standard_normal((B, dims[0])).astype(np.float32)
        if loss_kind == "mse":
            tgt = rng.standard_normal((B, dims[-1])).astype(np.float32)
        else:
            tgt = rng.integers(0, dims[-1], size=B).astype(np.int32)
        loss, out, reps = net.step(X, tgt, lr, None, it)
        h = torch.tensor(X, dtype=torch.float64)
        for l in range(3):
            h = h @ tw[l].T
            if l < 2:
                h = torch.relu(h)
        if loss_kind == "mse":
            tl = torch.mean((h - torch.tensor(tgt, dtype=torch.float64)) ** 2)
        else:
            tl = torch.nn.functional.cross_entropy(h, torch.tensor(tgt, dtype=torch.long))
        assert abs(loss - float(tl.detach())) < 1e-5 * max(1.0, abs(float(tl.detach())))
        assert _rel(out, h.detach().numpy()) < 1e-5
        tl.backward()
        with torch.no_grad():
            for w in tw:
                w -= lr * w.grad
                w.grad = None
        for l in range(3):
            assert _rel(layers[l].decode_weights(), tw[l].detach().numpy()) < 1e-5
        assert all(r.status == orc.CLEAN for r in reps)


def test_code_conditioning_closed_forms_and_brute_force(orc):
    """Conditioning of the erasure sub-systems: closed forms for the all-ones checksum code and for the
    generators of the paper's worked example, and an independent enumeration with numpy's inverse for seeded
    Gaussian codes."""
    import itertools
    from paper_1903_01042_b200 import workloads as wl
    W = np.zeros((12, 20), np.float32)
    # all-ones single parity over k data outputs: A = [1]; a decoded output is parity minus the k - 1 others
    lay = orc.Layer(W, 4, 5, 1, 1)
    assert lay.code_conditioning(0) == (1.0, 1.0, 4.0) and lay.code_conditioning(1) == (1.0, 1.0, 5.0)
    # the worked example: P_r = [[1, 1], [1, -1]], P_c = [[1, 1], [1, 2]]
    toy = orc.Layer(np.zeros((4, 4), np.float32), 2, 2, 2, 2, P_row=[[1, 1], [1, -1]], P_col=[[1, 1], [1, 2]])
    assert toy.code_conditioning(0) == (2.0, 1.0, 2.0)
    # P_c: 1 x 1 systems 1 / |p| <= 1, amplification (1 + other) / |p| <= 3; the 2 x 2 system has inverse [[2, -1], [-1, 1]]
    assert np.allclose(toy.code_conditioning(1), (3.0 * 3.0, 3.0, 3.0))
    for (k, r, seed) in [(5, 2, 0), (6, 3, 4), (4, 4, 2)]:
        P = wl.gaussian_parity(k, r, seed, 0)
        lay = orc.Layer(np.zeros((2 * k, 8), np.float32), k, 2, r, 0, P_row=P)
        worst = [0.0, 0.0, 0.0]
        P64 = P.astype(np.float64)
        for s in range(1, r + 1):
            for F in itertools.combinations(range(k), s):
                rest = [x for x in range(k) if x not in F]
                for Q in itertools.combinations(range(r), s):
                    A = P64[np.ix_(F, Q)].T
                    Ai = np.linalg.inv(A)
                    w = 1.0 + np.abs(P64[np.ix_(rest, Q)]).sum(axis=0)
                    worst[0] = max(worst[0], np.abs(A).sum(1).max() * np.abs(Ai).sum(1).max())
                    worst[1] = max(worst[1], np.abs(Ai).sum(1).max())
                    worst[2] = max(worst[2], (np.abs(Ai) @ w).max())
        assert np.allclose(lay.code_conditioning(0), worst, rtol=1e-10)
        assert np.isclose(worst[0], wl.worst_condition(P), rtol=1e-10) and worst[0] <= wl.COND_LIMIT
        assert lay.code_conditioning(1) == (0.0, 0.0, 0.0)      # no parity in that direction


def test_node_check_threshold_has_a_rounding_floor_for_cancelling_checksums(orc):
    """Blocks whose rows cancel exactly (every column sums to zero) have zero inner checksums u, so the
    checksum-side scale of the node-check threshold, tau_rel * sum|u||x|, is zero, while the sum of the stored
    (rounded) block outputs is a rounding residue of the order of 1e-7 * sum|y|.  The threshold's second term,
    (tau_rel / 512) * sum|y|, is what keeps such a fault-free node from being flagged: without it this test
    fails (the ratio is the residue over tau_abs = 1e-20).  The margin of the clean outputs stays below 0.1, and a
    hit node is still found with its margin above 10."""
    rng = np.random.default_rng(5)
    m = n = 2
    b = 48
    W = np.zeros((m * b, n * b), np.float32)
    for i in range(m):
        for j in range(n):
            a = np.round(rng.uniform(-1, 1, (b // 3, b)) * 1024) / 1024          # ten fractional bits: sums are exact
            c = np.round(rng.uniform(-1, 1, (b // 3, b)) * 1024) / 1024
            blk = np.concatenate([a, c, -(a + c)]).astype(np.float32)
            assert np.all(blk.astype(np.float64).sum(axis=0) == 0.0)
            W[i * b:(i + 1) * b, j * b:(j + 1) * b] = blk
    lay = orc.Layer(W, m, n, 1, 1, tau_rel=1e-3, tau_abs=1e-20)
    assert all(np.all(lay.u(i, j) == 0.0) for i in range(m + 1) for j in range(n))   # the checksums do cancel
    worst = 0.0
    for trial in range(20):
        X = rng.standard_normal((3, n * b)).astype(np.float32)
        S, rep = lay.forward(X)
        Y = lay.forward_products(X)
        assert np.any(Y.astype(np.float64).reshape(n, m + 1, b, 3).sum(axis=2) != 0.0)    # there is a residue to survive
        assert rep.status == orc.CLEAN and rep.n_detected_cw == 0, trial
        worst = max(worst, rep.max_margin_clean)
    assert 0.0 < worst < 0.1
    f = orc.make_fault(seed=2, mode=orc.FAULT_EXACTLY_ONE, sigma=10.0)
    for it in range(10):
        S, rep = lay.forward(rng.standard_normal((3, n * b)).astype(np.float32), f, it)
        assert tuple(rep.flagged_mask) == tuple(rep.injected_mask)
        assert rep.min_margin_hit > 10.0


# ---------------------------------------------------------------------------------------------
# soft errors in the small steps (Error Model 2 in encoding, input generation, detection, decoding)
# ---------------------------------------------------------------------------------------------

def _small_layer(orc, m=2, n=2, r=2, b=6, seed=3, mode=None):
    from paper_1903_01042_b200 import workloads as wl
    rng = np.random.default_rng(seed)
    W = rng.standard_normal((m * b, n * b)).astype(np.float32)
    Pr, Pc = wl.gaussian_parity(m, r, seed, 0), wl.gaussian_parity(n, r, seed, 1)
    lay = orc.Layer(W, m, n, r, r, P_row=Pr, P_col=Pc, locate_mode=orc.LOCATE_NODECHECK if mode is None else mode, tau_rel=1e-3)
    return lay, W, rng


def _iteration_hitting_only(orc, plan, phase, units, wanted, start=0):
    """First iteration >= start in which exactly the units in `wanted` (of all `units`) are hit."""
    for it in range(start, start + 100000):
        if {u for u in units if orc.small_hit(plan, phase, it, u)} == set(wanted):
            return it
    raise AssertionError("no such iteration")


def test_encoding_faults_surface_at_the_next_products_and_are_repaired(orc):
    """A soft error in the additional encoding (delta~_i of a parity block-row, x~_j of a parity block-column) does
    not touch the products of its own iteration; it enters the stored parity blocks through the update, and the
    next products that use those blocks show it in every codeword, at exactly that parity node (Section
    "Decentralized Implementation", last paragraph).  Every single encoding unit of the 2 x 2 + 2 + 2 grid is tried
    in turn.  Regeneration of the affected blocks (or the checkpoint) brings the layer back into the code."""
    m = n = 2
    for unit in range(4):                      # x~_2, x~_3 (units 2, 3), delta~_2, delta~_3 (units Nn + 2, Nn + 3)
        lay, W, rng = _small_layer(orc, mode=orc.LOCATE_SYNDROME)
        Nn = n + 2
        units = [n, n + 1, Nn + m, Nn + m + 1]
        plan = orc.make_small_faults(seed=5, layer=1, p_encode=0.3, sigma=10.0)
        it = _iteration_hitting_only(orc, plan, orc.PHASE_ENCODE, units, [units[unit]])
        X = rng.standard_normal((2, n * 6)).astype(np.float32)
        D = rng.standard_normal((2, m * 6)).astype(np.float32)
        lay.checkpoint_save()
        lay.set_small_faults(plan)
        S, rf = lay.forward(X, None, it)
        C, rb = lay.backward_update(D, X, 0.05, None, it)
        lay.set_small_faults(None)
        assert rf.status == orc.CLEAN and rb.status == orc.CLEAN       # nothing shows in the iteration of the fault
        assert lay.check_invariance() > 1e-2                            # but the stored parity blocks left the code
        S2, rf2 = lay.forward(X, None, it + 1)
        C2, rb2 = lay.backward_update(D, X, 0.0, None, it + 1)
        if unit < 2:      # x~_j entered the blocks of parity block-column j: the backward products show it
            j = units[unit]
            assert rf2.status == orc.CLEAN
            assert rb2.n_detected_cw == m and all(rb2.flagged_mask[i] == 1 << j for i in range(m))
            assert rb2.status == orc.CORRECTED
            for i in range(m):
                lay.regenerate_block(i, j, 1)
        else:             # delta~_i entered the blocks of parity block-row i: the feedforward products show it
            i = units[unit] - Nn
            assert rf2.n_detected_cw == n and all(rf2.flagged_mask[j] == 1 << i for j in range(n))
            assert rf2.status == orc.CORRECTED and rb2.status == orc.CLEAN
            for j in range(n):
                lay.regenerate_block(i, j, 0)
        # corrected outputs are the plain products with the (intact) data blocks
        assert _rel(S2, X.astype(np.float64) @ lay.decode_weights().astype(np.float64).T) < 1e-4
        assert lay.check_invariance() < 1e-5
        S3, rf3 = lay.forward(X, None, it + 2)
        C3, rb3 = lay.backward_update(D, X, 0.0, None, it + 2)
        assert rf3.status == orc.CLEAN and rb3.status == orc.CLEAN
        lay.checkpoint_restore()                                        # the other remedy: back to the checkpoint
        assert lay.check_invariance() < 1e-6 and _rel(lay.decode_weights(), W) == 0.0


def test_input_copy_faults_are_located_like_output_faults(orc):
    """A node whose own copy of its input sub-vector is off (an error in the activation / post-multiplication step
    that generated it) outputs W~_ij (x_j + nu): the deviation W~_ij nu is caught by the same checks as any
    erroneous output, in the same call.  Every single node of the 2 x 2 + 2 + 2 grid in turn, then a random run."""
    lay, W, rng = _small_layer(orc)
    m = n = 2
    M, Nn = 4, 4
    nodes = [i * Nn + j for i in range(M) for j in range(n)]
    plan = orc.make_small_faults(seed=9, layer=0, p_input=0.1, sigma=10.0)
    lay.set_small_faults(plan)
    X = rng.standard_normal((3, n * 6)).astype(np.float32)
    want = X.astype(np.float64) @ W.astype(np.float64).T
    for node in nodes:
        it = _iteration_hitting_only(orc, plan, orc.PHASE_INPUT, nodes, [node])
        S, rep = lay.forward(X, None, it)
        i, j = node // Nn, node % Nn
        assert rep.status == orc.CORRECTED and rep.n_detected_cw == 1
        assert rep.injected_mask[j] == 1 << i and rep.flagged_mask[j] == 1 << i
        assert rep.min_margin_hit > 10.0 and _rel(S, want) < 1e-4
    hits = 0
    for it in range(200):
        S, rep = lay.forward(X, None, it)
        truth = [sum(1 << i for i in range(M) if orc.small_hit(plan, orc.PHASE_INPUT, it, i * Nn + j)) for j in range(n)]
        assert list(rep.injected_mask[:n]) == truth
        hits += sum(bin(t).count("1") for t in truth)
        if all(bin(t).count("1") <= 2 for t in truth):
            assert list(rep.flagged_mask[:n]) == truth and _rel(S, want) < 1e-4
    assert hits > 50


def test_verification_steps_report_a_disagreement_exactly_when_an_evaluation_was_hit(orc):
    """The two verification steps: a soft error in one evaluation of a codeword's parity checks, or (for a
    detected codeword) of its list of erroneous nodes, makes the evaluations differ; the call then reports
    DISAGREE (the caller restores the last checkpoint).  Ground truth is the generator; without a plan, or with
    nothing hit, the status never appears."""
    lay, W, rng = _small_layer(orc)
    m = n = 2
    X = rng.standard_normal((2, n * 6)).astype(np.float32)
    D = rng.standard_normal((2, m * 6)).astype(np.float32)
    f = orc.make_fault(seed=4, mode=orc.FAULT_BERNOULLI, p=0.15, sigma=10.0)
    plan = orc.make_small_faults(seed=6, layer=0, p_check=0.1, p_decode=0.3, sigma=10.0)
    seen = {"check": 0, "decode": 0, "none": 0}
    for it in range(300):
        lay.set_small_faults(None)
        S0, r0 = lay.forward(X, f, it)                                   # the same call without small-step errors
        assert r0.status != orc.DISAGREE
        lay.set_small_faults(plan)
        S, rep = lay.forward(X, f, it)
        hit_c = [orc.small_hit(plan, orc.PHASE_CHECK, it, 0 * 64 + cw) for cw in range(n)]
        hit_d = [orc.small_hit(plan, orc.PHASE_DECODE, it, 0 * 64 + cw) and bool((r0.detected_mask >> cw) & 1) and not hit_c[cw]
                 for cw in range(n)]
        assert (rep.status == orc.DISAGREE) == (any(hit_c) or any(hit_d)), it
        seen["check"] += any(hit_c); seen["decode"] += any(hit_d); seen["none"] += not (any(hit_c) or any(hit_d))
        if not (any(hit_c) or any(hit_d)):
            assert rep.decisions() == r0.decisions() and np.array_equal(S, S0)
        C, rb = lay.backward_update(D, X, 0.0, f, it)
        hit_cb = [orc.small_hit(plan, orc.PHASE_CHECK, it, 1 * 64 + cw) for cw in range(m)]
        if any(hit_cb):
            assert rb.status == orc.DISAGREE
    assert min(seen.values()) > 10


# ---------------------------------------------------------------------------------------------
# bfloat16 storage
# ---------------------------------------------------------------------------------------------

def _bf16_rne_by_integers(x):
    """Round-to-nearest-even of float32 values to bfloat16 (returned as float32), in integer arithmetic on the bit
    patterns: keep the upper 16 bits, round up when the lower 16 are above half, or exactly half with an odd keeper."""
    u = np.asarray(x, np.float32).view(np.uint32).astype(np.uint64)
    low, keep = u & 0xFFFF, u >> 16
    up = (low > 0x8000) | ((low == 0x8000) & ((keep & 1) == 1))
    return ((keep + up.astype(np.uint64)) << 16).astype(np.uint32).view(np.float32)


def test_bf16_storage_rounds_to_nearest_even_in_parity_blocks_and_updates(orc):
    """The storage rounding of the oracle is round-to-nearest-even: pinned on sums that land exactly half-way
    between two bfloat16 values (even and odd keepers), just above and just below half-way, against two
    independent roundings (integer arithmetic on the bits; torch's float32 -> bfloat16 conversion).  Truncation,
    or rounding half away from zero, fails the tie cases."""
    import torch
    m = n = 2
    b = 8                                            # 8 x 8 blocks
    h = np.float32(2.0 ** -8)                        # half a bfloat16 step at 1.0
    # data blocks (all representable in bfloat16); the parity block-row holds W_0j + W_1j
    base = np.array([1.0, 1.0078125, -1.0, -1.0078125, 1.5, 2.0, 0.75, 1.0], np.float32)
    add = np.array([h, h, -h, -h, h * np.float32(1.5), h, h * np.float32(0.25), np.float32(2.0 ** -9)], np.float32)
    assert np.array_equal(base, _bf16_rne_by_integers(base)) and np.array_equal(add, _bf16_rne_by_integers(add))
    W = np.zeros((m * b, n * b), np.float32)
    for c in range(n * b):
        W[:b, c] = np.roll(base, c)
        W[b:, c] = np.roll(add, c)
    lay = orc.Layer(W, m, n, 1, 1, store_bf16=True, tau_rel=3e-2)
    for j in range(n):
        exact = (W[:b, j * b:(j + 1) * b].astype(np.float64) + W[b:, j * b:(j + 1) * b].astype(np.float64)).astype(np.float32)
        want = _bf16_rne_by_integers(exact)
        assert np.array_equal(want, torch.tensor(exact).to(torch.bfloat16).float().numpy())
        got = lay.block(m, j)                        # parity block-row m, block-column j
        assert np.array_equal(got, want), j
        # the cases really are what they claim: ties that round down to an even keeper, ties that round up,
        # and values a truncation would get wrong
        trunc = (exact.view(np.uint32) & np.uint32(0xFFFF0000)).view(np.float32)
        assert np.any(want != trunc) and np.any((exact.view(np.uint32) & 0xFFFF) == 0x8000)
    # the coded update rounds once, from the exact sum, to nearest even as well
    lr = 1.0
    D = np.zeros((1, m * b), np.float32); D[0, :] = 1.0
    X = np.zeros((1, n * b), np.float32); X[0, :] = np.tile(np.array([h, -h, h * np.float32(3.0), np.float32(2.0 ** -9)], np.float32), n * b // 4)
    before = [[lay.block(i, j).astype(np.float64) if not (i == m and j == n) else None for j in range(n + 1)]
              for i in range(m + 1)]
    lay.update(D, X, lr)
    Dt = np.concatenate([D[0, :b], D[0, b:], D[0, :b] + D[0, b:]])            # delta~ per block-row (all-ones code)
    Xt = np.concatenate([X[0, :b], X[0, b:], X[0, :b] + X[0, b:]])            # x~ per block-column
    for i in range(m + 1):
        for j in range(n + 1):
            if i == m and j == n:
                continue
            exact = (before[i][j] + lr * np.outer(Dt[i * b:(i + 1) * b], Xt[j * b:(j + 1) * b])).astype(np.float32)
            want = _bf16_rne_by_integers(exact)
            assert np.array_equal(want, torch.tensor(exact).to(torch.bfloat16).float().numpy())
            assert np.array_equal(lay.block(i, j), want), (i, j)


def test_bf16_storage_rounds_blocks_and_keeps_products_close(orc):
    from paper_1903_01042_b200 import workloads as wl
    rng = np.random.default_rng(17)
    m = n = 4
    W = wl.weights(64, 64, seed=1, bf16=True)
    Pr, Pc = wl.gaussian_parity(m, 2, 1, 0), wl.gaussian_parity(n, 2, 1, 1)
    lay = orc.Layer(W, m, n, 2, 2, P_row=Pr, P_col=Pc, store_bf16=True, tau_rel=3e-2)
    for (i, j) in [(0, 0), (4, 1), (2, 5)]:
        blk = lay.block(i, j)
        assert np.array_equal(blk, wl.bf16_round(blk))
    assert np.array_equal(lay.decode_weights(), W)
    X = rng.standard_normal((8, 64)).astype(np.float32)
    S, rep = lay.forward(X)
    assert rep.status == orc.CLEAN
    assert _rel(S, X.astype(np.float64) @ W.astype(np.float64).T) < 1e-6
    f = orc.make_fault(seed=3, mode=orc.FAULT_BERNOULLI, p=0.08)
    hit = 0
    for it in range(20):
        S, rep = lay.forward(X, f, it)
        assert tuple(rep.flagged_mask) == tuple(rep.injected_mask)
        hit += rep.n_flagged_nodes
        # a corrected output is rebuilt from parity blocks that were rounded to bfloat16
        # (2^-9 per element), amplified by the conditioning of the erasure system
        assert _rel(S, X.astype(np.float64) @ W.astype(np.float64).T) < 1e-1
    assert hit > 0


# ---------------------------------------------------------------------------------------------
# faults in the stored blocks and regeneration (Section "Experimental Results"; the "regenerate"
# step of the feedforward stage)
# ---------------------------------------------------------------------------------------------

from paper_1903_01042_b200 import workloads as wl  # seeded generators only (no arithmetic of the method)


def _intact_layer(orc, gaussian, bf16=False):
    m, n, rr, rc = 3, 2, 2, 1
    W = wl.weights(48, 40, seed=31, bf16=bf16)
    Pr = wl.gaussian_parity(m, rr, 4, 0) if gaussian else None
    Pc = wl.gaussian_parity(n, rc, 4, 1) if gaussian else None
    return W, orc.Layer(W, m, n, rr, rc, P_row=Pr, P_col=Pc, store_bf16=bf16)


@pytest.mark.parametrize("gaussian", [False, True])
def test_every_block_is_the_code_combination_of_its_column_and_of_its_row(orc, gaussian):
    """Claim 1 read block-wise: along a block-column the M blocks are a G_r codeword, along a block-row
    the Nn blocks are a G_c codeword, so rebuilding an intact block from the others reproduces it."""
    W, lay = _intact_layer(orc, gaussian)
    for i in range(lay.M):
        for j in range(lay.Nn):
            if not lay.has_node(i, j):
                continue
            for along in (0, 1):
                has_code = (j < lay.n) if along == 0 else (i < lay.m)
                before = lay.block(i, j)
                if not has_code:
                    with pytest.raises(ValueError):
                        lay.regenerate_block(i, j, along)
                    continue
                lay.regenerate_block(i, j, along)
                after = lay.block(i, j)
                assert np.max(np.abs(after - before)) <= 2e-6 * max(np.max(np.abs(before)), 1e-30), (i, j, along)
                lay.set_block(i, j, before)


def test_regeneration_matches_the_definition_with_numpy(orc):
    """A data block from the first parity of its column: (parity - sum_k P[k] other_k) / P[i], in float64."""
    W, lay = _intact_layer(orc, True)
    Pr = wl.gaussian_parity(3, 2, 4, 0).astype(np.float64)
    i, j = 1, 0
    others = [lay.block(k, j).astype(np.float64) for k in range(3)]
    parity = lay.block(3, j).astype(np.float64)
    want = (parity - sum(Pr[k, 0] * others[k] for k in range(3) if k != i)) / Pr[i, 0]
    lay.set_block(i, j, np.zeros_like(lay.block(i, j)))
    lay.regenerate_block(i, j, 0)
    assert np.array_equal(lay.block(i, j), want.astype(np.float32))


def test_sparse_fault_statistics_and_recovery(orc):
    W, lay = _intact_layer(orc, False)
    clean = lay.block(0, 1)
    n_changed = lay.corrupt_block(0, 1, seed=9, layer=0, iteration=5, density=0.05, amplitude=5.0)
    bad = lay.block(0, 1)
    diff = bad - clean
    assert n_changed == int(np.count_nonzero(diff))                 # (a zero draw has probability 2^-24)
    assert 0.02 < n_changed / diff.size < 0.09                      # density 0.05 of 16 x 20 elements
    assert np.all(np.abs(diff) <= 5.0 + 1e-6)
    assert lay.check_invariance() > 1e-2                            # the grid is no longer a codeword
    # the same call again (same counters) adds the same matrix; another iteration adds another one
    lay.set_block(0, 1, clean)
    lay.corrupt_block(0, 1, seed=9, layer=0, iteration=5, density=0.05, amplitude=5.0)
    assert np.array_equal(lay.block(0, 1), bad)
    lay.set_block(0, 1, clean)
    lay.corrupt_block(0, 1, seed=9, layer=0, iteration=6, density=0.05, amplitude=5.0)
    assert not np.array_equal(lay.block(0, 1), bad)
    # recovery in either direction restores the decoded weights
    for along in (0, 1):
        lay.set_block(0, 1, bad)
        lay.regenerate_block(0, 1, along)
        assert np.max(np.abs(lay.decode_weights() - W)) <= 2e-6 * np.max(np.abs(W))
        assert lay.check_invariance() < 1e-5


def test_a_corrupted_stored_block_is_located_at_the_next_products_until_it_is_regenerated(orc):
    """The fault sits in the weights, not in one output: the node is flagged in every following phase (the
    outputs are still corrected from the code), and no longer once the block has been rebuilt."""
    W, lay = _intact_layer(orc, False)
    lay.corrupt_block(1, 0, seed=2, layer=0, iteration=0, density=0.05, amplitude=5.0)
    X = wl.gaussian_inputs(2, 40, seed=32)
    D = wl.gaussian_inputs(2, 48, seed=33)
    for _ in range(2):
        S, rep = lay.forward(X, None, 0)
        assert rep.flagged_mask[0] == 1 << 1 and rep.flagged_mask[1] == 0 and rep.status == orc.CORRECTED
        assert np.max(np.abs(S - X @ W.T)) <= 1e-5 * np.max(np.abs(S))
    Z = lay.backward_products(D)
    Zc = Z.copy()
    rep_b = lay.detect_decode(1, Zc, D)
    assert rep_b.flagged_mask[1] == 1 << 0 and rep_b.flagged_mask[0] == 0 and rep_b.flagged_mask[2] == 0
    lay.regenerate_block(1, 0, 0)
    S, rep = lay.forward(X, None, 0)
    assert rep.status == orc.CLEAN and not any(rep.flagged_mask)
