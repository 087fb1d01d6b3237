"""Parity of the CUDA path (through the C-ABI library) with the CPU oracle, element by element
on the same seeded inputs.  Bars: reports (detected / located / corrected decisions) bit-exact;
values max|a-b| / max|b| <= 1e-5 for the fp32 FFMA paths, <= 2e-3 where tensor-core tiles or
bfloat16 storage are involved; weights <= 1e-4 after 100 steps (fp32 storage).
"""
import numpy as np
import pytest
import torch

from paper_1903_01042_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TOL_F32 = 1e-5
TOL_LOWP = 2e-3
TOL_DECODED = 1e-4   # outputs rebuilt by erasure decoding through an ill-conditioned Gaussian code


def _rel(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return float(np.max(np.abs(a - b)) / max(np.max(np.abs(b)), 1e-300))


@pytest.fixture(scope="module")
def cn():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device (there is no CPU path)")
    from paper_1903_01042_b200 import codenet
    codenet.lib()
    return codenet


def _dev(a, dtype=torch.float32):
    return torch.tensor(np.ascontiguousarray(a), device="cuda").to(dtype).contiguous()


class Pair:
    """The same coded layer held by the oracle and by the CUDA library."""

    def __init__(self, cn, orc, W, m, n, rr, rc, P_row=None, P_col=None, bf16=False, batch_max=1,
                 locate_mode=2, check_rows=None, check_cols=None, tau_rel=None, math=0):
        if tau_rel is None:
            tau_rel = 3e-2 if (bf16 or math != 0) else 1e-3
        if check_rows is None:
            check_rows = wl.check_slice(-(-W.shape[0] // m))
        if check_cols is None:
            check_cols = wl.check_slice(-(-W.shape[1] // n))
        self.o = orc.Layer(W, m, n, rr, rc, P_row=P_row, P_col=P_col, store_bf16=bf16,
                           locate_mode=locate_mode, check_rows=check_rows, check_cols=check_cols,
                           tau_rel=tau_rel)
        Wd = _dev(W, torch.bfloat16 if bf16 else torch.float32)
        self.g = cn.encode_layer(Wd, m, n, rr, rc, P_row=P_row, P_col=P_col, batch_max=batch_max,
                                 locate_mode=locate_mode, check_rows=check_rows, check_cols=check_cols,
                                 tau_rel=tau_rel, math=math)
        self.bf16 = bf16

    def compare_checksums(self, cn, tol):
        worst = 0.0
        for i in range(self.o.M):
            for j in range(self.o.Nn):
                if not self.o.has_node(i, j):
                    continue
                u, v = cn.get_checksums(self.g, i, j)
                scale = max(np.max(np.abs(self.o.u(i, j))), np.max(np.abs(self.o.v(i, j))), 1e-30)
                worst = max(worst, float(np.max(np.abs(u.cpu().numpy() - self.o.u(i, j))) / scale),
                            float(np.max(np.abs(v.cpu().numpy() - self.o.v(i, j))) / scale))
        assert worst <= tol, worst
        return worst

    def compare_blocks(self, cn, tol):
        worst = 0.0
        for i in range(self.o.M):
            for j in range(self.o.Nn):
                if not self.o.has_node(i, j):
                    continue
                got = cn.get_block(self.g, i, j).cpu().numpy()
                worst = max(worst, _rel(got, self.o.block(i, j)))
        assert worst <= tol, worst
        return worst


SHAPES = [
    # n_out, n_in, m, n, rr, rc, gaussian code
    (64, 96, 2, 2, 1, 1, False),
    (10, 72, 4, 4, 1, 1, False),       # padded head (10 -> 12 rows), b_c = 18 (not a multiple of 4)
    (250, 196, 2, 4, 1, 1, False),
    (96, 64, 3, 2, 2, 2, True),
    (128, 128, 8, 8, 2, 2, True),
    (64, 288, 2, 18, 1, 1, False),     # 18 data nodes per backward codeword (more than the one-pass sums take)
    (40, 40, 1, 1, 0, 0, False),       # uncoded
]


def _codes(m, n, rr, rc, gaussian, seed=0):
    if not gaussian:
        return None, None
    return wl.gaussian_parity(m, rr, seed, 0), wl.gaussian_parity(n, rc, seed, 1)


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("bf16", [False, True])
def test_initial_encoding(cn, orc, shape, bf16):
    no, ni, m, n, rr, rc, gauss = shape
    W = wl.weights(no, ni, seed=1, bf16=bf16)
    Pr, Pc = _codes(m, n, rr, rc, gauss)
    p = Pair(cn, orc, W, m, n, rr, rc, Pr, Pc, bf16=bf16)
    assert (p.g.b_r, p.g.b_c, p.g.M, p.g.Nn) == (p.o.b_r, p.o.b_c, p.o.M, p.o.Nn)
    # the one-off encoding sums in double on both sides: identical stored blocks
    assert p.compare_blocks(cn, 0.0) == 0.0
    p.compare_checksums(cn, 1e-6)
    assert (p.g.T, p.g.ns, p.g.Tc, p.g.nsc) == (p.o.T, p.o.ns, p.o.Tc, p.o.nsc)
    assert np.array_equal(cn.decode_weights(p.g).float().cpu().numpy(), W)
    assert cn.check_invariance(p.g) < (2e-2 if bf16 else 1e-5)


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("B", [1, 3, 8, 19])
def test_forward_and_backward_values_without_faults(cn, orc, shape, B):
    no, ni, m, n, rr, rc, gauss = shape
    W = wl.weights(no, ni, seed=2)
    Pr, Pc = _codes(m, n, rr, rc, gauss)
    p = Pair(cn, orc, W, m, n, rr, rc, Pr, Pc, batch_max=B)
    X = wl.gaussian_inputs(B, ni, seed=3)
    D = wl.gaussian_inputs(B, no, seed=4) / np.float32(B)
    rep = cn.new_reports(2)
    S = cn.forward(p.g, _dev(X), rep_dev=rep[:cn.REPORT_BYTES])
    So, ro = p.o.forward(X)
    assert _rel(S.cpu().numpy(), So) <= TOL_F32
    Cg = cn.backward_update(p.g, _dev(D), _dev(X), 0.05, rep_dev=rep[cn.REPORT_BYTES:])
    Co, rbo = p.o.backward_update(D, X, 0.05)
    assert _rel(Cg.cpu().numpy(), Co) <= TOL_F32
    rf, rb = cn.read_reports(rep)
    assert rf.decisions() == ro.decisions() and rb.decisions() == rbo.decisions()
    assert rf.status == cn.CLEAN and rb.status == cn.CLEAN
    p.compare_blocks(cn, 1e-6)                      # every stored block after the coded update
    p.compare_checksums(cn, 1e-6)                   # and the inner checksums that follow it
    assert _rel(cn.decode_weights(p.g).cpu().numpy(), p.o.decode_weights()) <= 1e-6
    # sums that nearly cancel make the relative measure noisy on the tiniest blocks
    assert cn.check_invariance(p.g) < max(1e-5, 50 * p.o.check_invariance())
    # the updated weights are used by the next forward pass, inner checksums still valid
    S2 = cn.forward(p.g, _dev(X), rep_dev=rep[:cn.REPORT_BYTES])
    S2o, r2o = p.o.forward(X)
    assert _rel(S2.cpu().numpy(), S2o) <= TOL_F32
    assert cn.read_reports(rep)[0].decisions() == r2o.decisions()


@pytest.mark.parametrize("shape", SHAPES[:6])
@pytest.mark.parametrize("B", [1, 4, 12, 32])      # 32: the blocked large-batch checks
def test_injected_faults_decisions_bit_exact(cn, orc, shape, B):
    _injected_faults_decisions(cn, orc, shape, B, 25)


# Batches of 128 and more take the shared-row checksum update; the shapes add what the list above lacks at a
# large batch: odd block sizes (no 16-byte row accesses in the update), twelve data nodes per backward codeword
# (the 4-byte-access syndrome / sums pass), three parities per code (the wide pass with four parity loads).
@pytest.mark.parametrize("shape", [SHAPES[1], SHAPES[3], SHAPES[4],
                                   (100, 132, 2, 12, 1, 1, False),
                                   (96, 60, 3, 4, 3, 3, True)])
@pytest.mark.parametrize("B", [128, 160])
def test_injected_faults_decisions_bit_exact_large_batches(cn, orc, shape, B):
    _injected_faults_decisions(cn, orc, shape, B, 10)


@pytest.mark.parametrize("B", [1, 4, 32])
def test_injected_faults_with_joint_location(cn, orc, B):
    """Training steps with injected faults under locate_mode JOINT (three parities: two hit nodes of a codeword
    are located from the syndromes alone): decisions as the oracle's, iteration after iteration."""
    _injected_faults_decisions(cn, orc, (96, 60, 3, 4, 3, 3, True), B, 12, locate_mode=4)


def _injected_faults_decisions(cn, orc, shape, B, iterations, locate_mode=2):
    no, ni, m, n, rr, rc, gauss = shape
    W = wl.weights(no, ni, seed=5)
    Pr, Pc = _codes(m, n, rr, rc, gauss)
    p = Pair(cn, orc, W, m, n, rr, rc, Pr, Pc, batch_max=B, locate_mode=locate_mode)
    it_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    rep = cn.new_reports(2)
    seen = set()
    K = max(m + rr, n + rc)
    prob = min(0.25, 1.5 / K)                 # both correctable and uncorrectable patterns occur
    for it in range(iterations):
        X = wl.gaussian_inputs(B, ni, seed=6, iteration=it)
        D = wl.gaussian_inputs(B, no, seed=7, iteration=it) / np.float32(B)
        it_dev.fill_(it)
        fg = cn.make_fault(seed=11, layer=3, mode=cn.FAULT_BERNOULLI, p=prob, sigma=10.0, iteration_dev=it_dev)
        fo = orc.make_fault(seed=11, layer=3, mode=orc.FAULT_BERNOULLI, p=prob, sigma=10.0)
        S = cn.forward(p.g, _dev(X), fault=fg, rep_dev=rep[:cn.REPORT_BYTES])
        Cg = cn.backward_update(p.g, _dev(D), _dev(X), 0.01, fault=fg, rep_dev=rep[cn.REPORT_BYTES:])
        So, ro = p.o.forward(X, fo, it)
        Co, rbo = p.o.backward_update(D, X, 0.01, fo, it)
        rf, rb = cn.read_reports(rep)
        assert rf.decisions() == ro.decisions(), ("forward", it)
        assert rb.decisions() == rbo.decisions(), ("backward", it)
        # erasure decoding with a real Gaussian generator amplifies the fp32 rounding of the node
        # outputs by the conditioning of the erasure system; checksum codes (all-ones P) do not
        tol_f = TOL_F32 if (not gauss or rf.status == cn.CLEAN) else TOL_DECODED
        tol_b = TOL_F32 if (not gauss or rb.status == cn.CLEAN) else TOL_DECODED
        if gauss:   # the looser bar stays inside what the conditioning of this code can amplify
            assert TOL_DECODED <= max(p.o.code_conditioning(0)[2], p.o.code_conditioning(1)[2]) * TOL_F32
        assert _rel(S.cpu().numpy(), So) <= tol_f
        assert _rel(Cg.cpu().numpy(), Co) <= tol_b
        seen.add(rf.status)
        seen.add(rb.status)
        for r in (rf, rb):
            if any(r.injected_mask):
                assert r.min_margin_hit > 10.0
            assert r.max_margin_clean < 0.1
        if locate_mode == 4:
            both = [(rf, p.o.M), (rb, p.o.Nn)]
            for r, K in both:
                for cw, inj in enumerate(r.injected_mask):
                    if 0 < bin(inj).count("1") <= rr - 1:
                        assert r.flagged_mask[cw] == inj, (it, cw)    # located exactly, from the syndromes alone
    assert cn.CORRECTED in seen and (cn.FALLBACK in seen or iterations < 25)   # both outcomes were exercised
    assert _rel(cn.decode_weights(p.g).cpu().numpy(), p.o.decode_weights()) <= 1e-5
    p.compare_checksums(cn, 1e-5)


@pytest.mark.parametrize("phase", [0, 1])
@pytest.mark.parametrize("mode", ["nodecheck", "syndrome", "none"])
@pytest.mark.parametrize("B", [2, 32])
def test_standalone_detect_decode(cn, orc, phase, mode, B):
    lm = {"nodecheck": 2, "syndrome": 1, "none": 0}[mode]
    m, n, r = 3, 4, 2
    W = wl.weights(48, 64, seed=8)
    Pr, Pc = wl.gaussian_parity(m, r, 2, 0), wl.gaussian_parity(n, r, 2, 1)
    p = Pair(cn, orc, W, m, n, r, r, Pr, Pc, batch_max=B, locate_mode=lm)
    X = wl.gaussian_inputs(B, 64, seed=9)
    D = wl.gaussian_inputs(B, 48, seed=10)
    clean = p.o.forward_products(X) if phase == 0 else p.o.backward_products(D)
    V = X if phase == 0 else D
    rng = np.random.default_rng(0)
    n_cw, K = clean.shape[0], clean.shape[1]
    patterns = [[0] * n_cw, [1] + [0] * (n_cw - 1), [0, 1 << (K - 1)] + [0] * (n_cw - 2),
                [0b101] + [0] * (n_cw - 1), [0b111, 0b10] + [0] * (n_cw - 2)]
    for pat in patterns:
        Y = clean.copy()
        for cw in range(n_cw):
            for k in range(K):
                if (pat[cw] >> k) & 1:
                    Y[cw, k] += (rng.standard_normal(Y[cw, k].shape) * 10).astype(np.float32)
        Yg = _dev(Y)
        rep = cn.new_reports(1)
        cn.detect_decode(p.g, phase, Yg, _dev(V), rep_dev=rep)
        Yo = Y.copy()
        ro = p.o.detect_decode(phase, Yo, V)
        rg = cn.read_reports(rep)[0]
        assert rg.decisions() == ro.decisions(), (pat, mode)
        assert _rel(Yg.cpu().numpy(), Yo) <= TOL_F32


@pytest.mark.parametrize("phase", [0, 1])
@pytest.mark.parametrize("r", [2, 3, 4])
@pytest.mark.parametrize("B", [2, 32])
def test_joint_location_of_up_to_r_minus_1_nodes(cn, orc, phase, r, B):
    """locate_mode JOINT: whole-sub-vector errors in up to r - 1 nodes of a codeword are located from the
    syndromes alone and decoded; r of them are detected and reported as not decodable.  SYNDROME (the paper's
    t = r / 2) gives up earlier on the same inputs."""
    m, n = 4, 5
    W = wl.weights(48, 60, seed=18)
    Pr, Pc = wl.gaussian_parity(m, r, 4, 0), wl.gaussian_parity(n, r, 4, 1)
    pj = Pair(cn, orc, W, m, n, r, r, Pr, Pc, batch_max=B, locate_mode=cn.LOCATE_JOINT)
    ps = Pair(cn, orc, W, m, n, r, r, Pr, Pc, batch_max=B, locate_mode=cn.LOCATE_SYNDROME)
    X = wl.gaussian_inputs(B, 60, seed=19)
    D = wl.gaussian_inputs(B, 48, seed=20)
    clean = pj.o.forward_products(X) if phase == 0 else pj.o.backward_products(D)
    V = X if phase == 0 else D
    n_cw, K = clean.shape[0], clean.shape[1]
    rng = np.random.default_rng(r)
    for count in range(1, r + 1):
        pat = [0] * n_cw
        for cw in (0, n_cw - 1):                 # two codewords, different supports (data and parity nodes mixed)
            for k in rng.choice(K, size=count, replace=False):
                pat[cw] |= 1 << int(k)
        Y = clean.copy()
        for cw in range(n_cw):
            for k in range(K):
                if (pat[cw] >> k) & 1:
                    Y[cw, k] += (rng.standard_normal(Y[cw, k].shape) * 10).astype(np.float32)
        for p, joint in ((pj, True), (ps, False)):
            Yg = _dev(Y)
            rep = cn.new_reports(1)
            cn.detect_decode(p.g, phase, Yg, _dev(V), rep_dev=rep)
            Yo = Y.copy()
            ro = p.o.detect_decode(phase, Yo, V)
            rg = cn.read_reports(rep)[0]
            assert rg.decisions() == ro.decisions(), (count, joint)
            limit = r - 1 if joint else r // 2
            if count <= min(limit, 3 if joint else 2):
                assert rg.status == cn.CORRECTED and list(rg.flagged_mask[:n_cw]) == pat
                assert _rel(Yg.cpu().numpy(), clean) <= TOL_DECODED
            else:
                assert rg.status == cn.FAILED    # detected (probability 1), not decodable, no fault-free copy here
            assert _rel(Yg.cpu().numpy(), Yo) <= TOL_DECODED


def test_code_conditioning_matches_the_oracle_and_singular_generators_are_reported(cn, orc):
    """The library's figures for the erasure sub-systems of both codes are the oracle's, and a generator with a
    singular sub-system (a zero entry: the lone parity cannot rebuild that data output; two all-ones parities)
    shows as infinite on both sides."""
    for (m, n, rr, rc, seed) in [(4, 4, 2, 2, 1), (8, 8, 2, 2, 0), (3, 5, 3, 4, 4), (4, 4, 1, 1, None)]:
        W = wl.weights(8 * m, 8 * n, seed=9)
        Pr, Pc = (None, None) if seed is None else (wl.gaussian_parity(m, rr, seed, 0), wl.gaussian_parity(n, rc, seed, 1))
        p = Pair(cn, orc, W, m, n, rr, rc, Pr, Pc)
        for phase in (0, 1):
            a, b = cn.code_conditioning(p.g, phase), p.o.code_conditioning(phase)
            assert np.allclose(a, b, rtol=1e-12, atol=0.0), (m, n, rr, rc, phase, a, b)
            assert a[0] <= wl.COND_LIMIT          # the generator the workloads draw passed the screen
    bad = np.ones((4, 1), np.float32)
    bad[2, 0] = 0.0
    for (rr, Pr) in [(1, bad), (2, None)]:
        p = Pair(cn, orc, wl.weights(32, 32, seed=9), 4, 4, rr, 1, Pr, None)
        assert cn.code_conditioning(p.g, 0)[0] == float("inf") and p.o.code_conditioning(0)[0] == float("inf")
        assert np.isfinite(cn.code_conditioning(p.g, 1)[0])


def test_a_bounded_wait_that_runs_out_is_reported_and_the_layer_recovers(cn, orc):
    """A forward launch on tensor-core tiles whose producer warp is told to issue no tile loads: the waits that
    depend on those loads give up after the (shortened) limit, the kernel releases its tensor memory and returns
    by itself, and the report of the call says TIMEOUT.  Nothing faults and nothing stays in flight.  After the
    acknowledgement the same layer runs normally again and agrees with the oracle."""
    W = wl.weights(512, 512, seed=61)
    p = Pair(cn, orc, W, 2, 2, 1, 1, batch_max=64, math=1)          # fp32 blocks, TF32 tiles, 256 x 256 blocks
    X = wl.gaussian_inputs(64, 512, seed=62)
    rep = cn.new_reports(1)
    S = cn.forward(p.g, _dev(X), rep_dev=rep)                       # a normal launch first
    So, ro = p.o.forward(X)
    assert cn.read_reports(rep)[0].status == cn.CLEAN and _rel(S.cpu().numpy(), So) <= TOL_LOWP
    try:
        cn.set_wait_limit(2_000_000)                                # two milliseconds instead of about a second
        cn.withhold_tile_loads(True)
        cn.forward(p.g, _dev(X), rep_dev=rep)
        cn.withhold_tile_loads(False)
        torch.cuda.synchronize()                                    # the kernel came back by itself
        assert cn.read_reports(rep)[0].status == cn.TIMEOUT
        cn.forward(p.g, _dev(X), rep_dev=rep)                       # the flag stays until it is acknowledged
        assert cn.read_reports(rep)[0].status == cn.TIMEOUT
    finally:
        cn.withhold_tile_loads(False)
        cn.set_wait_limit(0)
    cn.reset_timeout(p.g)
    S = cn.forward(p.g, _dev(X), rep_dev=rep)
    assert cn.read_reports(rep)[0].decisions() == ro.decisions()
    assert cn.read_reports(rep)[0].status == cn.CLEAN
    assert _rel(S.cpu().numpy(), So) <= TOL_LOWP


@pytest.mark.parametrize("shape,B,bf16,math", [((96, 60, 3, 4, 2, 2, True), 2, False, 0),
                                                ((192, 256, 2, 2, 1, 1, False), 1, False, 0),
                                                ((512, 512, 2, 2, 2, 2, True), 64, False, 1)])
def test_soft_errors_in_the_small_steps_against_the_oracle(cn, orc, shape, B, bf16, math):
    """Error Model 2 in the steps around the products (additional encoding, a node's own input copy, error
    detection, decoding) with the two verification steps: the same generator drives both sides, so the reports must
    agree step by step (DISAGREE included), outputs must agree whenever the call was not told to roll back, and
    the stored blocks, which encoding errors push out of the code, must stay equal on both sides.  After a
    DISAGREE both sides restore their checkpoint, as the method prescribes."""
    no, ni, m, n, rr, rc, gauss = shape
    W = wl.weights(no, ni, seed=71, bf16=bf16)
    Pr, Pc = _codes(m, n, rr, rc, gauss)
    p = Pair(cn, orc, W, m, n, rr, rc, Pr, Pc, bf16=bf16, batch_max=B, math=math)
    it_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    kw = dict(seed=8, layer=2, p_encode=0.04, p_input=0.03, p_check=0.04, p_decode=0.3, sigma=10.0)
    cn.set_small_faults(p.g, cn.make_small_faults(iteration_dev=it_dev, **kw))
    p.o.set_small_faults(orc.make_small_faults(**kw))
    fg = cn.make_fault(seed=12, layer=2, mode=cn.FAULT_BERNOULLI, p=0.04, sigma=10.0, iteration_dev=it_dev)
    fo = orc.make_fault(seed=12, layer=2, mode=orc.FAULT_BERNOULLI, p=0.04, sigma=10.0)
    rep = cn.new_reports(1)
    repb = cn.new_reports(1)
    tol = TOL_LOWP if math else TOL_F32
    seen = {"disagree": 0, "input": 0, "encode": 0}
    cn.checkpoint_save(p.g)
    p.o.checkpoint_save()
    for it in range(60):
        X = wl.gaussian_inputs(B, ni, seed=72, iteration=it)
        D = wl.gaussian_inputs(B, no, seed=73, iteration=it) / np.float32(B)
        it_dev.fill_(it)
        S = cn.forward(p.g, _dev(X), fault=fg, rep_dev=rep)
        Cg = cn.backward_update(p.g, _dev(D), _dev(X), 0.02, fault=fg, rep_dev=repb)
        So, ro = p.o.forward(X, fo, it)
        Co, rbo = p.o.backward_update(D, X, 0.02, fo, it)
        rf, rb = cn.read_reports(rep)[0], cn.read_reports(repb)[0]
        assert rf.decisions() == ro.decisions(), ("forward", it, rf.decisions()[:5], ro.decisions()[:5])
        assert rb.decisions() == rbo.decisions(), ("backward", it, rb.decisions()[:5], rbo.decisions()[:5])
        loose = TOL_DECODED if gauss else tol
        if rf.status != cn.DISAGREE:
            assert _rel(S.cpu().numpy(), So) <= (max(tol, loose) if rf.status != cn.CLEAN else tol), it
        if rb.status != cn.DISAGREE:
            assert _rel(Cg.cpu().numpy(), Co) <= (max(tol, loose) if rb.status != cn.CLEAN else tol), it
        Nn = n + rc
        seen["input"] += any(orc.small_hit(p.o._small, orc.PHASE_INPUT, it, i * Nn + j) for i in range(m + rr) for j in range(n))
        seen["encode"] += any(orc.small_hit(p.o._small, orc.PHASE_ENCODE, it, u) for u in list(range(n, Nn)) + [Nn + i for i in range(m, m + rr)])
        if rf.status == cn.DISAGREE or rb.status == cn.DISAGREE:
            seen["disagree"] += 1
            cn.checkpoint_restore(p.g)
            p.o.checkpoint_restore()
        elif it % 10 == 9:
            cn.checkpoint_save(p.g)
            p.o.checkpoint_save()
        if it % 10 == 0:
            # stored blocks (pushed out of the code by encoding errors, identically on both sides) and checksums
            for (i, j) in [(0, 0), (m, 0), (0, n), (m + rr - 1, n - 1), (m - 1, n + rc - 1)]:
                got = cn.get_block(p.g, i, j).cpu().numpy()
                assert _rel(got, p.o.block(i, j)) <= (1e-4 if not math else 5e-3), (it, i, j)
    assert min(seen.values()) > 0, seen


def test_regeneration_rebuilds_the_inner_checksums_of_the_block(cn, orc):
    """Everything a regenerated node stored is generated again: after an encoding error has entered a parity block
    and its inner checksums through the update, regeneration restores both, as on the oracle (up to the one
    rounding by which the two sides' updated data blocks may differ)."""
    m, n, r = 2, 3, 2
    W = wl.weights(64, 96, seed=81)
    Pr, Pc = _codes(m, n, r, r, True)
    p = Pair(cn, orc, W, m, n, r, r, Pr, Pc, batch_max=2)
    it_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    kw = dict(seed=3, layer=0, p_encode=1.0, sigma=10.0)          # every parity sub-vector is hit once
    X = wl.gaussian_inputs(2, 96, seed=82)
    D = wl.gaussian_inputs(2, 64, seed=83)
    cn.set_small_faults(p.g, cn.make_small_faults(iteration_dev=it_dev, **kw))
    p.o.set_small_faults(orc.make_small_faults(**kw))
    cn.backward_update(p.g, _dev(D), _dev(X), 0.05)
    p.o.backward_update(D, X, 0.05)
    cn.set_small_faults(p.g, None)
    p.o.set_small_faults(None)
    assert cn.check_invariance(p.g) > 1e-2 and p.o.check_invariance() > 1e-2
    for j in range(n):
        for i in range(m, m + r):
            cn.regenerate_block(p.g, i, j, 0)
            p.o.regenerate_block(i, j, 0)
    for i in range(m):
        for j in range(n, n + r):
            cn.regenerate_block(p.g, i, j, 1)
            p.o.regenerate_block(i, j, 1)
    assert cn.check_invariance(p.g) < 1e-5 and p.o.check_invariance() < 1e-5
    p.compare_checksums(cn, 1e-6)
    for i in range(m + r):
        for j in range(n + r):
            if p.o.has_node(i, j):
                assert _rel(cn.get_block(p.g, i, j).cpu().numpy(), p.o.block(i, j)) <= 1e-6, (i, j)


def test_check_rows_slices(cn, orc):
    W = wl.weights(64, 32, seed=12)
    p = Pair(cn, orc, W, 2, 2, 1, 1, batch_max=2, check_rows=8, check_cols=4)
    assert (p.g.T, p.g.ns, p.g.Tc, p.g.nsc) == (8, 4, 4, 4)
    it_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    rep = cn.new_reports(2)
    for it in range(10):
        X = wl.gaussian_inputs(2, 32, seed=13, iteration=it)
        D = wl.gaussian_inputs(2, 64, seed=14, iteration=it)
        it_dev.fill_(it)
        fg = cn.make_fault(seed=1, mode=cn.FAULT_BERNOULLI, p=0.1, iteration_dev=it_dev)
        fo = orc.make_fault(seed=1, mode=orc.FAULT_BERNOULLI, p=0.1)
        S = cn.forward(p.g, _dev(X), fault=fg, rep_dev=rep[:cn.REPORT_BYTES])
        Cg = cn.backward_update(p.g, _dev(D), _dev(X), 0.02, fault=fg, rep_dev=rep[cn.REPORT_BYTES:])
        So, ro = p.o.forward(X, fo, it)
        Co, rbo = p.o.backward_update(D, X, 0.02, fo, it)
        rf, rb = cn.read_reports(rep)
        assert rf.decisions() == ro.decisions() and rb.decisions() == rbo.decisions()
        assert _rel(S.cpu().numpy(), So) <= TOL_F32 and _rel(Cg.cpu().numpy(), Co) <= TOL_F32
    assert cn.check_invariance(p.g) < 1e-5


def test_bad_arguments(cn):
    W = torch.zeros((8, 8), device="cuda")
    with pytest.raises(cn.CodenetError):
        cn.encode_layer(W, 2, 2, 5, 1)                       # too many parities
    with pytest.raises(cn.CodenetError):
        cn.encode_layer(W, 2, 2, 1, 1, check_rows=3)         # does not divide the block height
    lay = cn.encode_layer(W, 2, 2, 1, 1, batch_max=2)
    with pytest.raises(cn.CodenetError):
        cn.forward(lay, torch.zeros((3, 8), device="cuda"))  # batch above batch_max
    with pytest.raises(cn.CodenetError):
        cn.get_block(lay, 2, 2)                              # corner: no node
    x = torch.zeros((1, 8), device="cuda")
    d = torch.zeros((1, 8), device="cuda")
    lib = cn.lib()
    # the combined call needs the next input and a place for its sums
    assert lib.codenet_backward_update_forward_next(lay.h, d.data_ptr(), x.data_ptr(), 1, 0.01, None, x.data_ptr(), None,
                                                    None, None, x.data_ptr(), None, None) != 0
    assert lib.codenet_backward_update_forward_next(lay.h, d.data_ptr(), x.data_ptr(), 1, 0.01, None, x.data_ptr(), None,
                                                    x.data_ptr(), None, None, None, None) != 0
    net = cn.net_create([lay], activation=0, loss=0)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        with pytest.raises(cn.CodenetError):
            cn.net_capture_steps(net, [], [], 0.01)          # no step to record
    gid = __import__("ctypes").c_int(-1)
    assert lib.codenet_net_capture_steps(net.h, 1, None, None, 1, 0.01, None, None, 0, None, 0, None, side.cuda_stream,
                                         __import__("ctypes").byref(gid)) != 0      # no input list
    assert lib.codenet_net_set_iteration_counter(None, None) != 0


# ---------------------------------------------------------------------------------------------
# whole configurations through codenet_step
# ---------------------------------------------------------------------------------------------

def _build_net(cn, orc, cfg, math=0, locate_mode=2):
    pairs = []
    for l, sp in enumerate(cfg.layers):
        W = wl.weights(sp.n_out, sp.n_in, seed=cfg.seed, layer=l, bf16=cfg.bf16)
        Pr, Pc = (wl.layer_codes(sp, cfg.seed, l) if sp.gaussian_code else (None, None))
        pairs.append(Pair(cn, orc, W, sp.m, sp.n, sp.r_row, sp.r_col, Pr, Pc, bf16=cfg.bf16,
                          batch_max=cfg.batch, math=math, locate_mode=locate_mode,
                          check_rows=sp.check_rows, check_cols=sp.check_cols))
    act = {"identity": 0, "relu": 1}[cfg.activation]
    loss = {"mse": 0, "softmax_ce": 1}[cfg.loss]
    gnet = cn.net_create([p.g for p in pairs], activation=act, loss=loss)
    onet = orc.Net([p.o for p in pairs], activation=act, loss=loss)
    return pairs, gnet, onet


def _fro(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def _run_config(cn, orc, cfg, iterations, tol, weight_tol, p=None, check_every=1, weight_norm="inf",
                tol_decoded=None, lookahead=False, math=0):
    pairs, gnet, onet = _build_net(cn, orc, cfg, math=math)
    L = len(pairs)
    if tol_decoded is not None:
        # an erasure-decoded output carries the deviations of the node outputs it is solved from, amplified by
        # at most the factor the code's conditioning gives: the looser bar must lie inside that envelope
        amplification = max(pr.o.code_conditioning(ph)[2] for pr in pairs for ph in (0, 1))
        assert tol <= tol_decoded <= amplification * tol, (tol_decoded, amplification)
    mode = {"bernoulli": 1, "exactly_one": 2, "none": 0}[cfg.fault_mode]
    prob = cfg.p if p is None else p
    it_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    fg = [cn.make_fault(seed=cfg.seed, layer=l, mode=mode, p=prob, sigma=cfg.sigma, iteration_dev=it_dev) for l in range(L)]
    fo = [orc.make_fault(seed=cfg.seed, layer=l, mode=mode, p=prob, sigma=cfg.sigma) for l in range(L)]
    reps = cn.new_reports(2 * L)
    loss_dev = torch.zeros(1, device="cuda")
    stats = {"corrected": 0, "fallback": 0, "detected": 0}
    xs_dev = [_dev(wl.layer_inputs(cfg, it)[0]) for it in range(iterations + 1)] if lookahead else None
    for it in range(iterations):
        X, T = wl.layer_inputs(cfg, it)
        it_dev.fill_(it)
        Td = torch.tensor(T, device="cuda")
        if lookahead:
            # the update sweep of this step also takes layer 1's products for the next input
            cn.net_set_next_input(gnet, xs_dev[it + 1])
        cn.step(gnet, xs_dev[it] if lookahead else _dev(X), Td, cfg.lr, faults=fg, reps_dev=reps, loss_dev=loss_dev)
        lo, out_o, reps_o = onet.step(X, T, cfg.lr, fo, it)
        if it % check_every == 0 or it == iterations - 1:
            rg = cn.read_reports(reps)
            for k in range(2 * L):
                assert rg[k].decisions() == reps_o[k].decisions(), (it, k)
                stats["detected"] += rg[k].n_detected_cw
                stats["corrected"] += rg[k].status == cn.CORRECTED
                stats["fallback"] += rg[k].status == cn.FALLBACK
                if any(rg[k].injected_mask):
                    assert rg[k].min_margin_hit > 10.0, (it, k, rg[k].min_margin_hit)
                assert rg[k].max_margin_clean < 0.1, (it, k, rg[k].max_margin_clean)
            decoded = any(rg[2 * l].status != cn.CLEAN for l in range(L))
            bound = tol_decoded if (decoded and tol_decoded is not None) else tol
            assert _rel(gnet.output(cfg.batch).cpu().numpy(), out_o) <= bound, it
            # the loss is a mean over outputs the tolerance `tol` bounds one by one
            assert abs(float(loss_dev.item()) - lo) <= max(1e-4, tol / 4) * max(1.0, abs(lo))
    for pr in pairs:
        wg = cn.decode_weights(pr.g).float().cpu().numpy()
        err = _fro(wg, pr.o.decode_weights()) if weight_norm == "fro" else _rel(wg, pr.o.decode_weights())
        assert err <= weight_tol, err
    return stats


def test_config1_full_size_100_iterations(cn, orc):
    """1024x1024, 2x2 + 1 + 1, batch 1, exactly one soft error per phase per iteration."""
    cfg = wl.config("c1")
    stats = _run_config(cn, orc, cfg, cfg.iterations, TOL_F32, 1e-4)
    assert stats["corrected"] == 2 * cfg.iterations and stats["fallback"] == 0


def test_config1_with_next_products_taken_in_the_update_sweep(cn, orc):
    """Same run, but each update sweep also produces the next iteration's feedforward products."""
    cfg = wl.config("c1")
    launches = cn.launch_count()
    stats = _run_config(cn, orc, cfg, cfg.iterations, TOL_F32, 1e-4, lookahead=True)
    assert stats["corrected"] == 2 * cfg.iterations and stats["fallback"] == 0
    # 1 step with its own forward sweep (8 launches), then 99 without (7 launches each)
    assert cn.launch_count() - launches < 8 * cfg.iterations - 90


@pytest.mark.parametrize("B", [1, 3, 8])
def test_next_products_batched_and_with_uncorrectable_patterns(cn, orc, B):
    cfg = wl.config("c3", scale=2)                    # 4096^2 on the 8x8+1+1 grid: 512-wide blocks
    cfg.batch = B
    stats = _run_config(cn, orc, cfg, 12, TOL_F32, 1e-4, p=4e-2, lookahead=True)
    assert stats["corrected"] > 0 and stats["fallback"] > 0


def test_next_products_are_dropped_when_another_input_arrives(cn, orc):
    W = wl.weights(256, 1024, seed=31)
    p = Pair(cn, orc, W, 2, 2, 1, 1, batch_max=1)
    X0 = wl.gaussian_inputs(1, 1024, seed=32, iteration=0)
    X1 = wl.gaussian_inputs(1, 1024, seed=32, iteration=1)
    X2 = wl.gaussian_inputs(1, 1024, seed=32, iteration=2)
    D = wl.gaussian_inputs(1, 256, seed=33)
    x1d, x2d = _dev(X1), _dev(X2)
    cn.backward_update(p.g, _dev(D), _dev(X0), 0.01, X_next_dev=x1d)
    p.o.backward_update(D, X0, 0.01)
    S = cn.forward(p.g, x2d)                          # not the announced input: products recomputed
    assert _rel(S.cpu().numpy(), p.o.forward(X2)[0]) <= TOL_F32
    S = cn.forward(p.g, x1d)                          # the stored products were discarded by that call
    assert _rel(S.cpu().numpy(), p.o.forward(X1)[0]) <= TOL_F32
    cn.backward_update(p.g, _dev(D), _dev(X0), 0.01, X_next_dev=x1d)
    p.o.backward_update(D, X0, 0.01)
    S = cn.forward(p.g, x1d)                          # announced input: products from the update sweep
    assert _rel(S.cpu().numpy(), p.o.forward(X1)[0]) <= TOL_F32


@pytest.mark.parametrize("case", [
    # n_out, n_in, m, n, rr, rc, B, one launch for the two checks?
    (1024, 1024, 2, 2, 1, 1, 1, True),
    (2048, 4096, 4, 8, 1, 1, 1, True),
    (1024, 2048, 2, 4, 1, 0, 1, True),     # no parity column: the backward codewords carry the node check alone
    (1024, 1024, 2, 2, 1, 1, 3, False),    # a batch: the two calls one after the other
    (1024, 1024, 2, 2, 2, 2, 1, False),    # two parities: a decoding plan may need the fix kernel
    (96, 64, 2, 2, 1, 1, 1, False),        # column strips do not tile the block-columns: no products taken ahead
])
def test_backward_update_and_the_next_forward_stage_in_one_call(cn, orc, case):
    """codenet_backward_update_forward_next against the oracle's backward + update of iteration t followed by its
    forward stage of iteration t + 1 (fault plan read one iteration on): sums, reports, weights, checksums; and the
    number of launches says whether the two checks shared one."""
    no, ni, m, n, rr, rc, B, paired = case
    W = wl.weights(no, ni, seed=41)
    p = Pair(cn, orc, W, m, n, rr, rc, batch_max=B)
    it_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    rep = cn.new_reports(2)
    prob = min(0.25, 1.5 / max(m + rr, n + rc))
    fg = cn.make_fault(seed=43, layer=1, mode=cn.FAULT_BERNOULLI, p=prob, sigma=10.0, iteration_dev=it_dev)
    fo = orc.make_fault(seed=43, layer=1, mode=orc.FAULT_BERNOULLI, p=prob, sigma=10.0)
    xs = [_dev(wl.gaussian_inputs(B, ni, seed=44, iteration=it)) for it in range(14)]
    seen = set()
    for it in range(13):
        X = wl.gaussian_inputs(B, ni, seed=44, iteration=it)
        X1 = wl.gaussian_inputs(B, ni, seed=44, iteration=it + 1)
        D = wl.gaussian_inputs(B, no, seed=45, iteration=it) / np.float32(B)
        it_dev.fill_(it)
        before = cn.launch_count()
        Cg, Sg = cn.backward_update_forward_next(p.g, _dev(D), xs[it], 0.01, xs[it + 1], fault=fg, fault_next=fg,
                                                 rep_dev=rep[cn.REPORT_BYTES:], rep_next_dev=rep[:cn.REPORT_BYTES])
        launches = cn.launch_count() - before
        Co, rbo = p.o.backward_update(D, X, 0.01, fo, it)
        So, rfo = p.o.forward(X1, fo, it + 1)
        rf, rb = cn.read_reports(rep)
        assert rb.decisions() == rbo.decisions(), ("backward", it)
        assert rf.decisions() == rfo.decisions(), ("next forward", it)
        assert _rel(Cg.cpu().numpy(), Co) <= TOL_F32 and _rel(Sg.cpu().numpy(), So) <= TOL_F32
        for r in (rf, rb):
            if any(r.injected_mask):
                assert r.min_margin_hit > 10.0
            assert r.max_margin_clean < 0.1
            seen.add(r.status)
        # vector encoding, fused sweep, one check kernel -- or the separate calls' launches
        assert (launches == 3) == paired, launches
    assert cn.CORRECTED in seen and cn.FALLBACK in seen
    assert _rel(cn.decode_weights(p.g).cpu().numpy(), p.o.decode_weights()) <= 1e-5
    p.compare_checksums(cn, 1e-5)
    # a stand-alone forward call afterwards starts from scratch and agrees as well
    S = cn.forward(p.g, xs[13])
    assert _rel(S.cpu().numpy(), p.o.forward(wl.gaussian_inputs(B, ni, seed=44, iteration=13))[0]) <= TOL_F32


def test_paired_checks_in_a_network_with_hidden_layers(cn, orc):
    """Three layers with ReLU and the softmax loss, the first with 512-wide blocks (so that its update sweep can take
    the next products), the next input announced before every step: the first layer's backward check and its next
    forward check share a launch, the staged report and the activations reach the next step; decisions, outputs
    and weights as the oracle's."""
    cfg = wl.Config("mlp", [wl.LayerSpec(384, 2048, 4, 4, 1, 1), wl.LayerSpec(256, 384, 4, 4, 1, 1),
                            wl.LayerSpec(10, 256, 4, 4, 1, 1)], 1, 0.01, 40,
                    activation="relu", loss="softmax_ce", inputs="uniform", p=2e-2, seed=5)
    launches = cn.launch_count()
    stats = _run_config(cn, orc, cfg, 40, TOL_F32, 1e-4, lookahead=True)
    with_pairs = cn.launch_count() - launches
    assert stats["corrected"] > 0
    launches = cn.launch_count()
    _run_config(cn, orc, cfg, 40, TOL_F32, 1e-4, lookahead=False)
    assert with_pairs < cn.launch_count() - launches - 39     # a forward sweep and a check launch fewer per step


def test_paired_checks_with_the_loss_folded_into_another_layers_encoding(cn, orc):
    """Two layers, ReLU, mean-squared-error loss, batch 1, the next input announced: the loss partials are left by the
    LAST layer's vector encoding and added up by the paired check of the FIRST layer at the end of the step."""
    cfg = wl.Config("two", [wl.LayerSpec(256, 1024, 2, 2, 1, 1), wl.LayerSpec(128, 256, 2, 2, 1, 1)], 1, 0.01, 30,
                    activation="relu", loss="mse", p=3e-2, seed=7)
    launches = cn.launch_count()
    stats = _run_config(cn, orc, cfg, 30, TOL_F32, 1e-4, lookahead=True)
    with_pairs = cn.launch_count() - launches
    assert stats["corrected"] > 0
    launches = cn.launch_count()
    _run_config(cn, orc, cfg, 30, TOL_F32, 1e-4, lookahead=False)
    assert with_pairs < cn.launch_count() - launches - 29


@pytest.mark.parametrize("coded", [True, False])
def test_layers_that_check_nothing_share_one_launch_for_their_sums(cn, orc, coded):
    """Checks switched off (with and without parity blocks), no faults, the next input announced: the sums of a step's
    backward stage and of the next step's forward stage come from one plain launch, the vector encoding rides on the
    sweep (two launches per step); outputs, loss and weights as the oracle's, eagerly and through a recording."""
    r = 1 if coded else 0
    cfg = wl.Config("off", [wl.LayerSpec(1024, 2048, 2, 4, r, r)], 1, 0.01, 12, fault_mode="none", seed=13)
    pairs, gnet, onet = _build_net(cn, orc, cfg, locate_mode=3)      # CODENET_LOCATE_OFF
    pool = [wl.layer_inputs(cfg, k) for k in range(4)]
    xs = [_dev(x) for x, _ in pool]
    ts = [_dev(t) for _, t in pool]
    losses = torch.zeros(4, device="cuda")
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    torch.cuda.set_stream(side)
    try:
        it = 0
        for k in range(4):                                   # eager steps with the next input announced
            cn.net_set_next_input(gnet, xs[(k + 1) % 4])
            before = cn.launch_count()
            cn.step(gnet, xs[k], ts[k], cfg.lr, loss_dev=losses[:1])
            if k > 0:
                assert cn.launch_count() - before == 2       # sweep (+ encoding), one launch for both sums
            lo, out_o, _ = onet.step(pool[k][0], pool[k][1], cfg.lr, None, it)
            assert _rel(gnet.output(1).cpu().numpy(), out_o) <= TOL_F32, it
            assert abs(float(losses[0].item()) - lo) <= 1e-4 * max(1.0, abs(lo)), it
            it += 1
        graph = cn.net_capture_steps(gnet, xs, ts, cfg.lr, loss_dev=losses, loss_stride=1, X_next_dev=xs[0])
        for rep_ in range(2):
            cn.net_replay(gnet, graph)
            lg = losses.cpu().numpy()
            for k in range(4):
                lo, out_o, _ = onet.step(pool[k][0], pool[k][1], cfg.lr, None, it)
                assert abs(float(lg[k]) - lo) <= 1e-4 * max(1.0, abs(lo)), it
                it += 1
            assert _rel(gnet.output(1).cpu().numpy(), out_o) <= TOL_F32, rep_
        assert _rel(cn.decode_weights(pairs[0].g).cpu().numpy(), pairs[0].o.decode_weights()) <= 1e-4
    finally:
        torch.cuda.synchronize()
        torch.cuda.set_stream(torch.cuda.default_stream())


def test_config2_mlp_relu_softmax(cn, orc):
    """784-1000-1000-10 MLP, 4x4 + 1 + 1 per layer, batch 1; error rate raised so that 200
    iterations see faults in every layer."""
    cfg = wl.config("c2")
    stats = _run_config(cn, orc, cfg, 200, TOL_F32, 1e-4, p=2e-2)
    assert stats["corrected"] > 0


def test_paper_network_scaled(cn, orc):
    """The paper's own experiment shape, 784-1000-1000-10 here (widths / 10), 5 x 4 data grid + 2 + 2
    Gaussian parities per layer, ReLU, softmax cross-entropy, batch 1: non-square grids, block widths
    that are no power of two (196, 250), a head of 2-row blocks."""
    cfg = wl.config("paper", scale=10)
    stats = _run_config(cn, orc, cfg, 40, TOL_F32, 1e-4, p=2e-2, tol_decoded=TOL_DECODED)
    assert stats["detected"] > 0 and stats["corrected"] > 0


@pytest.mark.parametrize("p", [0.0, 1e-2])
def test_config3_scaled(cn, orc, p):
    """8x8 + 1 + 1 grid of config 3 on a 2048x2048 layer."""
    cfg = wl.config("c3", scale=4)
    stats = _run_config(cn, orc, cfg, 40, TOL_F32, 1e-4, p=p)
    if p == 0.0:
        assert stats["detected"] == 0


def test_config5_scaled(cn, orc):
    """8 ReLU layers + 10-way head, 4x4 + 1 + 1, batch 64, widths divided by 16."""
    cfg = wl.config("c5", scale=16)
    stats = _run_config(cn, orc, cfg, 12, TOL_F32, 1e-4, p=1e-2)
    assert stats["detected"] > 0


def test_config4_scaled_bf16_gaussian_code(cn, orc):
    """bfloat16 storage, 8x8 + 2 + 2 Gaussian MDS code, batch 128, on a 1024x1024 layer."""
    cfg = wl.config("c4", scale=16)
    # one bfloat16 rounding that goes the other way is 2^-8 of that element, so the weights are
    # compared in the relative Frobenius norm
    # ... and an output rebuilt by erasure decoding inherits the 2^-9 rounding of the stored parity
    # blocks times the conditioning of the Gaussian erasure system, on both sides alike; the two
    # sides then differ where a stored element rounded the other way
    stats = _run_config(cn, orc, cfg, 10, TOL_LOWP, 2e-3, p=2e-2, weight_norm="fro", tol_decoded=3e-2)
    assert stats["detected"] > 0


def test_bfloat16_blocks_at_batch_1_with_the_encoding_aboard_the_sweep(cn, orc):
    """bfloat16 storage, checksum code, batch 1, mean-squared-error loss, the next input announced: the streaming sweep
    takes the next products, carries the vector encoding and is followed by the paired check (two launches per step)."""
    cfg = wl.Config("b16", [wl.LayerSpec(2048, 2048, 2, 2, 1, 1)], 1, 0.01, 24, bf16=True, p=5e-2, seed=17)
    launches = cn.launch_count()
    stats = _run_config(cn, orc, cfg, 24, TOL_LOWP, 2e-3, weight_norm="fro", lookahead=True)
    assert stats["corrected"] > 0
    # the first step runs its own forward stage (sweep, check), encoding, sweep and pair: 5; the other 23: 2 each,
    # the decoded-weights / report helpers launch nothing that is counted here
    assert cn.launch_count() - launches <= 5 + 2 * 23 + 8


# ---------------------------------------------------------------------------------------------
# tensor-core tiles (batch >= 64)
# ---------------------------------------------------------------------------------------------

def test_config5_scaled_tf32_tensor_core_tiles(cn, orc):
    """8 ReLU layers of 1024x1024 + 10-way head, fp32 blocks multiplied as TF32, batch 64."""
    cfg = wl.config("c5", scale=4)
    # every layer's product is within 2e-3 of the exact one for the inputs it is given (checked per
    # layer in test_tensor_core_update_...); through nine layers the deviations add up to first order
    stats = _run_config(cn, orc, cfg, 10, TOL_LOWP * len(cfg.layers), 1e-4, p=1e-2, math=1)
    assert stats["detected"] > 0


def test_config4_scaled_bf16_tensor_core_tiles(cn, orc):
    """bfloat16 blocks, 8x8 + 2 + 2 Gaussian code, batch 128, 2048x2048: forward / backward products
    and the rank-B update on tcgen05 tiles."""
    cfg = wl.config("c4", scale=8)
    stats = _run_config(cn, orc, cfg, 8, TOL_LOWP, 2e-3, p=2e-2, weight_norm="fro", tol_decoded=3e-2, math=2)
    assert stats["detected"] > 0


@pytest.mark.parametrize("name,math,batch", [("c4", 2, 96), ("c5", 1, 128), ("c4", 2, 64)])
def test_tensor_core_tiles_on_other_batches(cn, orc, name, math, batch):
    """Batch 96 (bfloat16) and batch 128 with fp32 blocks (the operand tiles would not fit beside the 64 KB
    weight tiles) run the backward products and the rank-B update as two tensor-core kernels; batch 64 with
    bfloat16 blocks takes the fused sweep with half-size operand tiles."""
    import dataclasses
    cfg = dataclasses.replace(wl.config(name, scale=8 if name == "c4" else 4), batch=batch)
    if name == "c5":
        cfg = dataclasses.replace(cfg, layers=cfg.layers[:2] + cfg.layers[-1:])
        # weights: delta carries the TF32 deviation of the products (<= 2e-3 per layer), times lr per step
        stats = _run_config(cn, orc, cfg, 6, TOL_LOWP * len(cfg.layers), 3e-4, p=2e-2, math=math)
    else:
        stats = _run_config(cn, orc, cfg, 6, TOL_LOWP, 2e-3, p=2e-2, weight_norm="fro", tol_decoded=3e-2, math=math)
    assert stats["detected"] > 0


def test_config4_scaled_200_iterations_on_tensor_core_tiles(cn, orc):
    """The iteration count configuration 4 names, at 2048 x 2048 (same grid, code, batch and error rate): decisions
    as the oracle's at every checked step, weights inside the bfloat16 bound after all 200."""
    cfg = wl.config("c4", scale=8)
    stats = _run_config(cn, orc, cfg, 200, TOL_LOWP, 2e-3, weight_norm="fro", tol_decoded=3e-2, math=2, check_every=8)
    assert stats["detected"] > 0 and stats["corrected"] > 0


def test_config5_scaled_100_iterations_on_tensor_core_tiles(cn, orc):
    """Configuration 5 at a quarter of its widths (nine layers, TF32 tiles, batch 64), 100 iterations at the largest
    error rate of its sweep.  Every layer's TF32 products deviate by up to 2e-3 and the deviations add up through
    the layers; the weights take lr times the deviation of delta per step."""
    cfg = wl.config("c5", scale=4)
    stats = _run_config(cn, orc, cfg, 100, TOL_LOWP * len(cfg.layers), 1e-3, p=1e-2, math=1, check_every=5)
    assert stats["detected"] > 0


def test_config2_2000_iterations_at_its_own_error_rate(cn, orc):
    """Configuration 2 at the error rate it names (1e-3 per node and phase), 2000 of its iterations.  Decisions are
    the oracle's at every step of the run.  Values: outputs within 1e-5 and weights within 1e-4 at every step until
    the two runs part at a ReLU unit, which must not happen in the first 100 steps (the bar of the configuration).
    Float against double evaluate a pre-activation s = W x a few 1e-7 apart; when an s falls between them, one side
    sees f'(s) = 1 where the other sees 0, that unit's delta is dropped on one side only, and ONE row of one
    layer's weights moves by lr * delta * x on one side only.  The test recognises exactly that signature (one
    layer, one row) at the step where the weights part; any other first difference fails.  From then on the two
    equally valid runs are compared on decisions only."""
    cfg = wl.config("c2")
    pairs, gnet, onet = _build_net(cn, orc, cfg)
    L = len(pairs)
    it_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    fg = [cn.make_fault(seed=cfg.seed, layer=l, mode=1, p=cfg.p, sigma=cfg.sigma, iteration_dev=it_dev) for l in range(L)]
    fo = [orc.make_fault(seed=cfg.seed, layer=l, mode=1, p=cfg.p, sigma=cfg.sigma) for l in range(L)]
    reps = cn.new_reports(2 * L)
    loss_dev = torch.zeros(1, device="cuda")
    together, parted_at, detected = True, None, 0
    for it in range(2000):
        X, T = wl.layer_inputs(cfg, it)
        it_dev.fill_(it)
        cn.step(gnet, _dev(X), torch.tensor(T, device="cuda"), cfg.lr, faults=fg, reps_dev=reps, loss_dev=loss_dev)
        lo, out_o, reps_o = onet.step(X, T, cfg.lr, fo, it)
        rg = cn.read_reports(reps)
        assert [r.decisions() for r in rg] == [r.decisions() for r in reps_o], it
        detected += sum(r.n_detected_cw for r in rg)
        if not together:
            continue
        assert _rel(gnet.output(1).cpu().numpy(), out_o) <= TOL_F32, it
        devs = []
        for pr in pairs:
            wg, wo = cn.decode_weights(pr.g).float().cpu().numpy(), pr.o.decode_weights()
            devs.append(np.max(np.abs(wg - wo), axis=1) / np.max(np.abs(wo)))
        worst = [float(d.max()) for d in devs]
        if max(worst) > 1e-5:
            # the runs part here: one row of one layer, by about lr * delta * x, everything else as before
            layers_off = [l for l in range(L) if worst[l] > 1e-5]
            assert len(layers_off) == 1, (it, worst)
            rows_off = np.flatnonzero(devs[layers_off[0]] > 1e-6)
            assert len(rows_off) == 1 and worst[layers_off[0]] < 1e-2, (it, rows_off, worst)
            together, parted_at = False, it
    assert parted_at is None or parted_at > 100, parted_at
    assert detected > 100


def test_config4_full_size_iteration_against_the_oracle(cn, orc):
    """One whole iteration of configuration 4 at full size (16384 x 16384 bfloat16, batch 128) compared with the
    oracle element by element: decisions, outputs, loss, and every decoded weight."""
    cfg = wl.config("c4")
    stats = _run_config(cn, orc, cfg, 1, TOL_LOWP, 2e-3, p=2e-2, weight_norm="fro", tol_decoded=3e-2, math=2)
    assert stats["detected"] > 0


def test_config5_full_size_layers_against_the_oracle(cn, orc):
    """Two whole iterations of the first two layers and the head of configuration 5 at full size (4096 x 4096,
    batch 64, TF32 tiles) compared with the oracle element by element."""
    import dataclasses
    cfg = wl.config("c5")
    cfg = dataclasses.replace(cfg, layers=cfg.layers[:2] + cfg.layers[-1:])
    stats = _run_config(cn, orc, cfg, 2, TOL_LOWP * len(cfg.layers), 3e-4, p=2e-2, math=1)
    assert stats["detected"] > 0


@pytest.mark.parametrize("bf16,math", [(False, 1), (True, 2)])
def test_tensor_core_update_moves_every_stored_block(cn, orc, bf16, math):
    """One step with a learning rate large enough for bfloat16 storage to see the update: every stored
    block (data, parity rows, parity columns) follows the coded update rule."""
    W = wl.weights(1024, 1024, seed=41, bf16=bf16)
    p = Pair(cn, orc, W, 4, 4, 1, 1, bf16=bf16, batch_max=64, math=math)
    X = wl.gaussian_inputs(64, 1024, seed=42)
    D = wl.gaussian_inputs(64, 1024, seed=43) / np.float32(8)
    Cg = cn.backward_update(p.g, _dev(D), _dev(X), 0.05)
    Co, _ = p.o.backward_update(D, X, 0.05)
    assert _rel(Cg.cpu().numpy(), Co) <= TOL_LOWP
    # the update product is taken in tf32 / bf16: 2^-11 / 2^-9 of the update, far below the weights
    worst = 0.0
    for i in range(p.o.M):
        for j in range(p.o.Nn):
            if p.o.has_node(i, j):
                got = cn.get_block(p.g, i, j).cpu().numpy()
                worst = max(worst, _fro(got, p.o.block(i, j)))
    assert worst <= (3e-3 if bf16 else TOL_LOWP), worst
    moved = _fro(cn.decode_weights(p.g).float().cpu().numpy(), W)
    assert moved > 0.05                                  # the step really changed the weights
    S = cn.forward(p.g, _dev(X))
    assert _rel(S.cpu().numpy(), p.o.forward(X)[0]) <= (2e-2 if bf16 else TOL_LOWP)


# ---------------------------------------------------------------------------------------------
# recorded steps (CUDA graphs)
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("lookahead", [False, True])
def test_recorded_steps_replay_like_plain_steps(cn, orc, lookahead):
    """Two recorded steps over alternating input buffers, replayed for 30 iterations with faults,
    against the oracle stepping normally."""
    cfg = wl.config("c1", scale=2)                    # 512 x 512, 2x2 + 1 + 1, batch 1
    pairs, gnet, onet = _build_net(cn, orc, cfg)
    it_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    fg = [cn.make_fault(seed=3, layer=0, mode=cn.FAULT_EXACTLY_ONE, sigma=10.0, iteration_dev=it_dev)]
    fo = [orc.make_fault(seed=3, layer=0, mode=orc.FAULT_EXACTLY_ONE, sigma=10.0)]
    reps = cn.new_reports(2)
    loss_dev = torch.zeros(1, device="cuda")
    bufs = [torch.zeros((1, 512), device="cuda") for _ in range(2)]
    tbuf = torch.zeros((1, 512), device="cuda")
    inputs = [wl.layer_inputs(cfg, it) for it in range(32)]

    def check(it):
        lo, out_o, reps_o = onet.step(inputs[it][0], inputs[it][1], cfg.lr, fo, it)
        rg = cn.read_reports(reps)
        assert [r.decisions() for r in rg] == [r.decisions() for r in reps_o], it
        assert _rel(gnet.output(1).cpu().numpy(), out_o) <= TOL_F32, it

    side = torch.cuda.Stream()                        # the default stream cannot record a graph
    torch.cuda.synchronize()
    torch.cuda.set_stream(side)
    # iteration 0 runs plainly (and announces buffer 1 as the next input)
    bufs[0].copy_(_dev(inputs[0][0])); bufs[1].copy_(_dev(inputs[1][0])); tbuf.copy_(_dev(inputs[0][1]))
    if lookahead:
        cn.net_set_next_input(gnet, bufs[1])
    cn.step(gnet, bufs[0], tbuf, cfg.lr, faults=fg, reps_dev=reps, loss_dev=loss_dev)
    check(0)
    # record "odd" (input in buffer 1) then "even" (input in buffer 0): the order of the replays
    g_odd = cn.net_capture_step(gnet, bufs[1], tbuf, cfg.lr, faults=fg, reps_dev=reps, loss_dev=loss_dev,
                                X_next_dev=bufs[0] if lookahead else None)
    g_even = cn.net_capture_step(gnet, bufs[0], tbuf, cfg.lr, faults=fg, reps_dev=reps, loss_dev=loss_dev,
                                 X_next_dev=bufs[1] if lookahead else None)
    launches = cn.launch_count()
    it_dev.fill_(1)                                           # recorded steps advance the counter themselves
    for it in range(1, 31):
        tbuf.copy_(_dev(inputs[it][1]))
        bufs[(it + 1) % 2].copy_(_dev(inputs[it + 1][0]))     # the next input, into the buffer not in use
        cn.net_replay(gnet, g_odd if it % 2 else g_even)
        check(it)
    assert cn.launch_count() == launches                      # replays go through the graph, not the launchers
    assert _rel(cn.decode_weights(pairs[0].g).cpu().numpy(), pairs[0].o.decode_weights()) <= 1e-4
    torch.cuda.synchronize()
    torch.cuda.set_stream(torch.cuda.default_stream())


@pytest.mark.parametrize("lookahead", [False, True, "off"])
def test_several_steps_recorded_into_one_graph(cn, orc, lookahead):
    """Five consecutive steps over a pool of five inputs recorded into one graph (each with its own reports and loss
    slot), replayed three times after one plain step.  Inside the recording every step knows its successor's input,
    so the forward stage of steps two to five is done by the step before; with the input after the last step
    announced as well, that holds across the end of a replay too.  Against the oracle stepping normally."""
    cfg = wl.Config("one", [wl.LayerSpec(1024, 2048, 2, 4, 1, 1)], 1, 0.01, 16, p=0.1, seed=9)
    pairs, gnet, onet = _build_net(cn, orc, cfg)
    if lookahead == "off":
        # announced inputs are ignored: every step sweeps the weights for its own forward products
        cn.net_set_lookahead(gnet, False)
        lookahead = False
        expected_launches = 25                        # forward sweep, check, encoding, update sweep, check
    else:
        expected_launches = 10 if lookahead else 13
    it_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    fg = [cn.make_fault(seed=3, layer=0, mode=cn.FAULT_BERNOULLI, p=cfg.p, sigma=10.0, iteration_dev=it_dev)]
    fo = [orc.make_fault(seed=3, layer=0, mode=orc.FAULT_BERNOULLI, p=cfg.p, sigma=10.0)]
    pool = [wl.layer_inputs(cfg, k) for k in range(5)]
    xs = [_dev(x) for x, _ in pool]
    ts = [_dev(t) for _, t in pool]
    reps = cn.new_reports(2 * 5)
    losses = torch.zeros(5, device="cuda")
    side = torch.cuda.Stream()                        # the default stream cannot record a graph
    torch.cuda.synchronize()
    torch.cuda.set_stream(side)
    if lookahead:
        cn.net_set_next_input(gnet, xs[1])
    cn.step(gnet, xs[0], ts[0], cfg.lr, faults=fg, reps_dev=reps[:2 * cn.REPORT_BYTES], loss_dev=losses[:1])
    lo, out_o, reps_o = onet.step(pool[0][0], pool[0][1], cfg.lr, fo, 0)
    assert [r.decisions() for r in cn.read_reports(reps)[:2]] == [r.decisions() for r in reps_o]
    order = [1, 2, 3, 4, 0]
    before = cn.launch_count()
    graph = cn.net_capture_steps(gnet, [xs[k] for k in order], [ts[k] for k in order], cfg.lr, faults=fg,
                                 reps_dev=reps, reps_stride=2, loss_dev=losses, loss_stride=1,
                                 X_next_dev=xs[1] if lookahead else None)
    # two launches (the sweep, which carries the vector encoding, and one check for two stages) for every step whose
    # successor the recording knows: all five with the input after the last one announced; else the first step of a
    # replay also runs its own forward stage (sweep, check) and the last one is encoding, sweep and its own check
    assert cn.launch_count() - before == expected_launches, cn.launch_count() - before
    it_dev.fill_(1)
    seen = set()
    for r in range(3):
        cn.net_replay(gnet, graph)
        rg = cn.read_reports(reps)
        lg = losses.cpu().numpy()
        for s, k in enumerate(order):
            it = 1 + 5 * r + s
            lo, out_o, reps_o = onet.step(pool[k][0], pool[k][1], cfg.lr, fo, it)
            assert [x.decisions() for x in rg[2 * s:2 * s + 2]] == [x.decisions() for x in reps_o], it
            assert abs(float(lg[s]) - lo) <= 1e-4 * max(1.0, abs(lo)), it
            seen.update(x.status for x in rg[2 * s:2 * s + 2])
        assert _rel(gnet.output(1).cpu().numpy(), out_o) <= TOL_F32, r
    assert cn.CORRECTED in seen and cn.FALLBACK in seen
    assert _rel(cn.decode_weights(pairs[0].g).cpu().numpy(), pairs[0].o.decode_weights()) <= 1e-4
    pairs[0].compare_checksums(cn, 1e-5)
    torch.cuda.synchronize()
    torch.cuda.set_stream(torch.cuda.default_stream())


def test_steps_in_a_graph_of_the_callers_own_with_copies_around_them(cn, orc):
    """The caller captures four steps into a CUDA graph of their own, each with the upload of its target and next
    input from pinned host memory (on a second stream) and the download of its reports and loss; the network
    advances the fault plans' iteration counter itself (codenet_net_set_iteration_counter).  Three replays with the
    host buffers refilled in between, against the oracle stepping normally."""
    cfg = wl.Config("one", [wl.LayerSpec(1024, 2048, 2, 4, 1, 1)], 1, 0.01, 16, p=0.1, seed=11)
    pairs, gnet, onet = _build_net(cn, orc, cfg)
    it_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    fg = [cn.make_fault(seed=3, layer=0, mode=cn.FAULT_BERNOULLI, p=cfg.p, sigma=10.0, iteration_dev=it_dev)]
    fo = [orc.make_fault(seed=3, layer=0, mode=orc.FAULT_BERNOULLI, p=cfg.p, sigma=10.0)]
    n_steps, n_in, n_out = 4, 2048, 1024
    inputs = [wl.layer_inputs(cfg, it) for it in range(3 * n_steps + 1)]
    # host side: per step [next input | target]; device side: a ring of four staging buffers
    h_up = [torch.empty(n_in + n_out).pin_memory() for _ in range(n_steps)]
    stage = [torch.zeros(n_in + n_out, device="cuda") for _ in range(4)]
    sx = [b[:n_in].view(1, n_in) for b in stage]
    st = [b[n_in:].view(1, n_out) for b in stage]
    slot = 2 * cn.REPORT_BYTES + 16
    out_dev = torch.zeros(n_steps * slot, dtype=torch.uint8, device="cuda")
    h_out = torch.empty(n_steps * slot, dtype=torch.uint8).pin_memory()
    main, up = torch.cuda.Stream(), torch.cuda.Stream()
    cn.net_set_iteration_counter(gnet, it_dev)
    torch.cuda.synchronize()
    with torch.cuda.stream(main):
        sx[3].copy_(_dev(inputs[0][0]))                      # the input of step 0, as if uploaded for the step before
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=main):
            up.wait_stream(main)
            step_done = []
            for k in range(n_steps):
                if k >= 3:
                    up.wait_event(step_done[k - 3])          # buffer k % 4 held the input of step k - 3
                with torch.cuda.stream(up):
                    stage[k % 4].copy_(h_up[k], non_blocking=True)
                main.wait_stream(up)
                o = out_dev[k * slot:(k + 1) * slot]
                cn.net_set_next_input(gnet, sx[k % 4])
                cn.step(gnet, sx[(k - 1) % 4], st[k % 4], cfg.lr, faults=fg, reps_dev=o[:2 * cn.REPORT_BYTES],
                        loss_dev=o[2 * cn.REPORT_BYTES:2 * cn.REPORT_BYTES + 4].view(torch.float32))
                h_out[k * slot:(k + 1) * slot].copy_(o, non_blocking=True)
                step_done.append(torch.cuda.Event())
                step_done[-1].record(main)
        seen = set()
        for r in range(3):
            for k in range(n_steps):
                it = r * n_steps + k
                h_up[k][:n_in].copy_(torch.tensor(inputs[it + 1][0]).reshape(-1))
                h_up[k][n_in:].copy_(torch.tensor(inputs[it][1]).reshape(-1))
            graph.replay()
            main.synchronize()
            assert int(it_dev.item()) == (r + 1) * n_steps       # the network advanced the counter, once per step
            for k in range(n_steps):
                it = r * n_steps + k
                lo, out_o, reps_o = onet.step(inputs[it][0], inputs[it][1], cfg.lr, fo, it)
                rg = cn.read_reports(h_out[k * slot:k * slot + 2 * cn.REPORT_BYTES])
                assert [x.decisions() for x in rg] == [x.decisions() for x in reps_o], it
                loss = float(h_out[k * slot + 2 * cn.REPORT_BYTES:k * slot + 2 * cn.REPORT_BYTES + 4].view(torch.float32)[0])
                assert abs(loss - lo) <= 1e-4 * max(1.0, abs(lo)), it
                seen.update(x.status for x in rg)
            assert _rel(gnet.output(1).cpu().numpy(), out_o) <= TOL_F32, r
        assert cn.CORRECTED in seen
        assert _rel(cn.decode_weights(pairs[0].g).cpu().numpy(), pairs[0].o.decode_weights()) <= 1e-4
    cn.net_set_iteration_counter(gnet, None)
    torch.cuda.synchronize()


def test_eager_checks_between_replays_of_a_recorded_step(cn, orc):
    """A recorded step, then an odd number of eager checks on the same layer (an evaluation pass with a fault,
    a stand-alone detect / decode), then the recorded step again: every replay must still decide like the
    oracle.  (Each check works in one of two statistics buffers and clears the other; which one is the
    library's own business, whatever the order of eager calls and replays.)"""
    cfg = wl.config("c1", scale=2)
    pairs, gnet, onet = _build_net(cn, orc, cfg)
    pg, po = pairs[0].g, pairs[0].o
    it_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    fg = [cn.make_fault(seed=5, layer=0, mode=cn.FAULT_EXACTLY_ONE, sigma=10.0, iteration_dev=it_dev)]
    fo = [orc.make_fault(seed=5, layer=0, mode=orc.FAULT_EXACTLY_ONE, sigma=10.0)]
    ev_it = torch.full((1,), 1000, dtype=torch.int32, device="cuda")
    fe_g = cn.make_fault(seed=6, layer=0, mode=cn.FAULT_EXACTLY_ONE, sigma=10.0, iteration_dev=ev_it)
    fe_o = orc.make_fault(seed=6, layer=0, mode=orc.FAULT_EXACTLY_ONE, sigma=10.0)
    reps = cn.new_reports(2)
    rep_e = cn.new_reports(1)
    loss_dev = torch.zeros(1, device="cuda")
    xbuf = torch.zeros((1, 512), device="cuda")
    tbuf = torch.zeros((1, 512), device="cuda")
    inputs = [wl.layer_inputs(cfg, it) for it in range(12)]
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    torch.cuda.set_stream(side)
    xbuf.copy_(_dev(inputs[0][0])); tbuf.copy_(_dev(inputs[0][1]))
    cn.step(gnet, xbuf, tbuf, cfg.lr, faults=fg, reps_dev=reps, loss_dev=loss_dev)
    lo, out_o, reps_o = onet.step(inputs[0][0], inputs[0][1], cfg.lr, fo, 0)
    assert [r.decisions() for r in cn.read_reports(reps)] == [r.decisions() for r in reps_o]
    graph = cn.net_capture_step(gnet, xbuf, tbuf, cfg.lr, faults=fg, reps_dev=reps, loss_dev=loss_dev)
    it_dev.fill_(1)
    for it in range(1, 11):
        xbuf.copy_(_dev(inputs[it][0])); tbuf.copy_(_dev(inputs[it][1]))
        cn.net_replay(gnet, graph)
        lo, out_o, reps_o = onet.step(inputs[it][0], inputs[it][1], cfg.lr, fo, it)
        assert [r.decisions() for r in cn.read_reports(reps)] == [r.decisions() for r in reps_o], it
        assert _rel(gnet.output(1).cpu().numpy(), out_o) <= TOL_F32, it
        # an odd number of eager checks between two replays: one, or three
        for k in range(1 if it % 2 else 3):
            xe = wl.gaussian_inputs(1, 512, seed=77, iteration=10 * it + k)
            ev_it.fill_(1000 + 10 * it + k)
            s_g = cn.forward(pg, _dev(xe), fault=fe_g, rep_dev=rep_e)
            s_o, rep_o = po.forward(xe, fe_o, 1000 + 10 * it + k)
            assert cn.read_reports(rep_e)[0].decisions() == rep_o.decisions(), (it, k)
            assert _rel(s_g.cpu().numpy(), s_o) <= TOL_F32, (it, k)
    torch.cuda.synchronize()
    torch.cuda.set_stream(torch.cuda.default_stream())


# ---------------------------------------------------------------------------------------------
# faults in the stored blocks and regeneration of a block from its code
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("gauss", [False, True])
def test_stored_block_faults_and_regeneration(cn, orc, bf16, gauss):
    """The sparse fault of the paper's experiment lands on the same elements with the same bits on both
    sides; the node is located at the next products on both sides; regeneration along the block-column or
    the block-row gives the oracle's block bit for bit (sums in double in the same order)."""
    m, n, rr, rc = 3, 4, 2, 1
    W = wl.weights(96, 160, seed=51, bf16=bf16)
    Pr = wl.gaussian_parity(m, rr, 6, 0) if gauss else None
    Pc = wl.gaussian_parity(n, rc, 6, 1) if gauss else None
    p = Pair(cn, orc, W, m, n, rr, rc, Pr, Pc, bf16=bf16, batch_max=2)
    X = wl.gaussian_inputs(2, 160, seed=52)
    rep = cn.new_reports(1)
    for (i, j, along) in [(1, 2, 0), (0, 0, 1), (3, 1, 0), (2, 4, 1), (4, 3, 0)]:
        cn.corrupt_block(p.g, i, j, 7, 0, 11, 0.01, 5.0)
        n_changed = p.o.corrupt_block(i, j, seed=7, layer=0, iteration=11, density=0.01, amplitude=5.0)
        assert n_changed > 0
        assert np.array_equal(cn.get_block(p.g, i, j).cpu().numpy(), p.o.block(i, j)), (i, j)
        if j < n:   # the block takes part in the feedforward products: located there, output corrected
            S = cn.forward(p.g, _dev(X), rep_dev=rep)
            So, ro = p.o.forward(X, None, 0)
            rg = cn.read_reports(rep)[0]
            assert rg.decisions() == ro.decisions() and rg.flagged_mask[j] == 1 << i
            assert _rel(S.cpu().numpy(), So) <= (TOL_DECODED if gauss and not bf16 else 3e-2 if bf16 else TOL_F32)
        cn.regenerate_block(p.g, i, j, along)
        p.o.regenerate_block(i, j, along)
        assert np.array_equal(cn.get_block(p.g, i, j).cpu().numpy(), p.o.block(i, j)), (i, j, along)
    Wg = cn.decode_weights(p.g).float().cpu().numpy()
    assert np.array_equal(Wg, p.o.decode_weights())
    # a data block solved through a bfloat16-rounded Gaussian parity block inherits that rounding divided by
    # the generator entry (both sides alike); otherwise the rebuilt weights are the original ones
    if not (bf16 and gauss):
        assert _rel(Wg, W) <= (1e-2 if bf16 else 2e-6)
    S = cn.forward(p.g, _dev(X), rep_dev=rep)
    assert cn.read_reports(rep)[0].decisions() == p.o.forward(X, None, 0)[1].decisions()
    # directions without redundancy for the block, and blocks that do not exist
    for (i, j, along) in [(1, 4, 0), (3, 1, 1)]:
        with pytest.raises(cn.CodenetError):
            cn.regenerate_block(p.g, i, j, along)
    with pytest.raises(cn.CodenetError):
        cn.regenerate_block(p.g, 3, 4, 0)
    with pytest.raises(cn.CodenetError):
        cn.corrupt_block(p.g, 4, 4, 0, 0, 0, 0.1, 1.0)


@pytest.mark.parametrize("shape,bf16,B", [(SHAPES[1], False, 1), (SHAPES[3], True, 4), (SHAPES[4], False, 32)])
def test_checkpoint_and_roll_back(cn, orc, shape, bf16, B):
    """Roll-back to the last checkpoint (the paper's answer to an undecodable pattern): the stored state comes
    back bit for bit, and training continues from it as the oracle's does."""
    no, ni, m, n, rr, rc, gauss = shape
    W = wl.weights(no, ni, seed=21, bf16=bf16)
    Pr, Pc = _codes(m, n, rr, rc, gauss)
    p = Pair(cn, orc, W, m, n, rr, rc, Pr, Pc, bf16=bf16, batch_max=B)
    with pytest.raises(Exception):
        cn.checkpoint_restore(p.g)              # nothing saved yet
    tol = TOL_LOWP if bf16 else TOL_F32

    def steps(first, count):
        for it in range(first, first + count):
            X = wl.gaussian_inputs(B, ni, seed=31, iteration=it)
            D = wl.gaussian_inputs(B, no, seed=32, iteration=it) / np.float32(B)
            Cg = cn.backward_update(p.g, _dev(D), _dev(X), 0.02)
            Co, _ = p.o.backward_update(D, X, 0.02)
            assert _rel(Cg.cpu().numpy(), Co) <= tol

    steps(0, 2)
    nodes = [(i, j) for i in range(p.o.M) for j in range(p.o.Nn) if p.o.has_node(i, j)]
    saved = {ij: (cn.get_block(p.g, *ij).clone(), [c.clone() for c in cn.get_checksums(p.g, *ij)]) for ij in nodes}
    cn.checkpoint_save(p.g)
    p.o.checkpoint_save()
    steps(2, 3)
    cn.corrupt_block(p.g, 0, 1, 9, 0, 0, 0.1, 5.0)
    assert any(not torch.equal(cn.get_block(p.g, *ij), saved[ij][0]) for ij in nodes)
    cn.checkpoint_restore(p.g)
    p.o.checkpoint_restore()
    for ij in nodes:
        assert torch.equal(cn.get_block(p.g, *ij), saved[ij][0])
        u, v = cn.get_checksums(p.g, *ij)
        assert torch.equal(u, saved[ij][1][0]) and torch.equal(v, saved[ij][1][1])
    p.compare_blocks(cn, tol)
    steps(2, 3)                                  # the iterations lost to the roll-back, again
    p.compare_blocks(cn, tol)
    p.compare_checksums(cn, tol)
    cn.checkpoint_save(p.g)                      # a second checkpoint reuses the memory of the first
    p.o.checkpoint_save()
    steps(5, 1)
    cn.checkpoint_restore(p.g)
    p.o.checkpoint_restore()
    p.compare_blocks(cn, tol)


def test_regeneration_at_full_size_of_configuration_3(cn, orc):
    """8192x8192 on the 8x8 + 1 + 1 grid: a 1024x1024 block is corrupted, located by the next feedforward
    products, rebuilt from the eight other blocks of its column; the oracle does the same at full size."""
    cfg = wl.config("c3")
    pairs, gnet, onet = _build_net(cn, orc, cfg)
    pr = pairs[0]
    X = wl.gaussian_inputs(1, 8192, seed=61)
    rep = cn.new_reports(1)
    cn.corrupt_block(pr.g, 5, 3, 1, 0, 0, 0.005, 5.0)
    pr.o.corrupt_block(5, 3, seed=1, layer=0, iteration=0, density=0.005, amplitude=5.0)
    S = cn.forward(pr.g, _dev(X), rep_dev=rep)
    So, ro = pr.o.forward(X, None, 0)
    rg = cn.read_reports(rep)[0]
    assert rg.decisions() == ro.decisions() and rg.flagged_mask[3] == 1 << 5 and rg.status == cn.CORRECTED
    assert _rel(S.cpu().numpy(), So) <= TOL_F32
    cn.regenerate_block(pr.g, 5, 3, 0)
    pr.o.regenerate_block(5, 3, 0)
    assert np.array_equal(cn.get_block(pr.g, 5, 3).cpu().numpy(), pr.o.block(5, 3))
    assert cn.check_invariance(pr.g) < 1e-5
    S = cn.forward(pr.g, _dev(X), rep_dev=rep)
    assert cn.read_reports(rep)[0].status == cn.CLEAN


# ---------------------------------------------------------------------------------------------
# full sizes, in the launch configuration bench.py times (recorded steps on a created stream,
# look-ahead for batch 1, tensor-core tiles for the batched configurations)
# ---------------------------------------------------------------------------------------------

def test_config3_full_size_recorded_steps_against_the_oracle(cn, orc):
    """8192x8192 fp32, 8x8 + 1 + 1, batch 1, p = 1e-2: the oracle runs the same 12 iterations at full
    size; every report, output and loss is compared, and the decoded weights at the end."""
    cfg = wl.config("c3")
    pairs, gnet, onet = _build_net(cn, orc, cfg)
    sp = cfg.layers[0]
    it_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    fg = [cn.make_fault(seed=cfg.seed, layer=0, mode=cn.FAULT_BERNOULLI, p=1e-2, sigma=cfg.sigma, iteration_dev=it_dev)]
    fo = [orc.make_fault(seed=cfg.seed, layer=0, mode=orc.FAULT_BERNOULLI, p=1e-2, sigma=cfg.sigma)]
    reps = cn.new_reports(2)
    loss_dev = torch.zeros(1, device="cuda")
    bufs = [torch.zeros((1, sp.n_in), device="cuda") for _ in range(2)]
    tbuf = torch.zeros((1, sp.n_out), device="cuda")
    n_it = 12
    inputs = [wl.layer_inputs(cfg, it) for it in range(n_it + 1)]
    detected = 0

    def check(it):
        nonlocal detected
        lo, out_o, reps_o = onet.step(inputs[it][0], inputs[it][1], cfg.lr, fo, it)
        rg = cn.read_reports(reps)
        assert [r.decisions() for r in rg] == [r.decisions() for r in reps_o], it
        for r in rg:
            detected += r.n_detected_cw
            if any(r.injected_mask):
                assert r.min_margin_hit > 10.0
            assert r.max_margin_clean < 0.1
        assert _rel(gnet.output(1).cpu().numpy(), out_o) <= TOL_F32, it
        assert abs(float(loss_dev.item()) - lo) <= 1e-4 * max(1.0, abs(lo))

    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    torch.cuda.set_stream(side)
    try:
        bufs[0].copy_(_dev(inputs[0][0])); bufs[1].copy_(_dev(inputs[1][0])); tbuf.copy_(_dev(inputs[0][1]))
        cn.net_set_next_input(gnet, bufs[1])
        cn.step(gnet, bufs[0], tbuf, cfg.lr, faults=fg, reps_dev=reps, loss_dev=loss_dev)
        check(0)
        g_odd = cn.net_capture_step(gnet, bufs[1], tbuf, cfg.lr, faults=fg, reps_dev=reps, loss_dev=loss_dev, X_next_dev=bufs[0])
        g_even = cn.net_capture_step(gnet, bufs[0], tbuf, cfg.lr, faults=fg, reps_dev=reps, loss_dev=loss_dev, X_next_dev=bufs[1])
        it_dev.fill_(1)
        for it in range(1, n_it):
            tbuf.copy_(_dev(inputs[it][1]))
            bufs[(it + 1) % 2].copy_(_dev(inputs[it + 1][0]))
            cn.net_replay(gnet, g_odd if it % 2 else g_even)
            check(it)
        assert detected > 0
        assert _rel(cn.decode_weights(pairs[0].g).cpu().numpy(), pairs[0].o.decode_weights()) <= 1e-4
        assert cn.check_invariance(pairs[0].g) < 1e-5
    finally:
        torch.cuda.synchronize()
        torch.cuda.set_stream(torch.cuda.default_stream())


def test_config3_full_size_eight_steps_per_recording(cn, orc):
    """The launch configuration bench.py times: 8192x8192 fp32, 8x8 + 1 + 1, batch 1, a pool of eight inputs, eight
    consecutive steps in one recording (two kernels per step: the sweep, in alternating directions and with the vector
    encoding aboard, and the paired check), replayed thirteen times after one plain step, p = 1e-2.  The oracle runs the
    same 105 iterations at full size: every report and loss of every step, the outputs at the end of each replay, and
    after more than a hundred steps the weights (within 1e-4) and the code invariance."""
    cfg = wl.config("c3")
    pairs, gnet, onet = _build_net(cn, orc, cfg)
    it_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    fg = [cn.make_fault(seed=cfg.seed, layer=0, mode=cn.FAULT_BERNOULLI, p=1e-2, sigma=cfg.sigma, iteration_dev=it_dev)]
    fo = [orc.make_fault(seed=cfg.seed, layer=0, mode=orc.FAULT_BERNOULLI, p=1e-2, sigma=cfg.sigma)]
    pool = [wl.layer_inputs(cfg, k) for k in range(8)]
    xs = [_dev(x) for x, _ in pool]
    ts = [_dev(t) for _, t in pool]
    reps = cn.new_reports(2 * 8)
    losses = torch.zeros(8, device="cuda")
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    torch.cuda.set_stream(side)
    try:
        cn.net_set_next_input(gnet, xs[1])
        cn.step(gnet, xs[0], ts[0], cfg.lr, faults=fg, reps_dev=reps[:2 * cn.REPORT_BYTES], loss_dev=losses[:1])
        lo, out_o, reps_o = onet.step(pool[0][0], pool[0][1], cfg.lr, fo, 0)
        assert [r.decisions() for r in cn.read_reports(reps)[:2]] == [r.decisions() for r in reps_o]
        order = [1, 2, 3, 4, 5, 6, 7, 0]
        before = cn.launch_count()
        graph = cn.net_capture_steps(gnet, [xs[k] for k in order], [ts[k] for k in order], cfg.lr, faults=fg,
                                     reps_dev=reps, reps_stride=2, loss_dev=losses, loss_stride=1, X_next_dev=xs[1])
        assert cn.launch_count() - before == 16     # per step: the sweep (with the encoding aboard) and the paired check
        it_dev.fill_(1)
        detected = 0
        for r in range(13):
            cn.net_replay(gnet, graph)
            rg = cn.read_reports(reps)
            lg = losses.cpu().numpy()
            for s_, k in enumerate(order):
                it = 1 + 8 * r + s_
                lo, out_o, reps_o = onet.step(pool[k][0], pool[k][1], cfg.lr, fo, it)
                assert [x.decisions() for x in rg[2 * s_:2 * s_ + 2]] == [x.decisions() for x in reps_o], it
                assert abs(float(lg[s_]) - lo) <= 1e-4 * max(1.0, abs(lo)), it
                for x in rg[2 * s_:2 * s_ + 2]:
                    detected += x.n_detected_cw
                    if any(x.injected_mask):
                        assert x.min_margin_hit > 10.0
                    assert x.max_margin_clean < 0.1
            assert _rel(gnet.output(1).cpu().numpy(), out_o) <= TOL_F32, r
        assert detected > 0
        assert _rel(cn.decode_weights(pairs[0].g).cpu().numpy(), pairs[0].o.decode_weights()) <= 1e-4
        assert cn.check_invariance(pairs[0].g) < 1e-5
    finally:
        torch.cuda.synchronize()
        torch.cuda.set_stream(torch.cuda.default_stream())


def _sampled_full_size_layer(cn, orc, cfg, math, tol):
    """One layer of a batched configuration at full size, two iterations with faults.  The oracle cannot
    run this size in seconds, so the run is checked on what can be computed one by one: the injection
    masks from the oracle's own hit test, detection of exactly the injected codewords with the
    required margins, sampled entries of W x, W^T delta and of the updated weights from their
    definitions in float64, and the code invariance of the stored blocks after the updates."""
    sp = cfg.layers[0]
    W = wl.weights(sp.n_out, sp.n_in, seed=cfg.seed, layer=0, bf16=cfg.bf16)
    Pr, Pc = (wl.layer_codes(sp, cfg.seed, 0) if sp.gaussian_code else (None, None))
    Wd = torch.tensor(W, device="cuda")
    g = cn.encode_layer(Wd.bfloat16() if cfg.bf16 else Wd, sp.m, sp.n, sp.r_row, sp.r_col, P_row=Pr, P_col=Pc,
                        batch_max=cfg.batch, math=math, check_rows=sp.check_rows, check_cols=sp.check_cols,
                        tau_rel=3e-2)
    B, M, Nn = cfg.batch, sp.m + sp.r_row, sp.n + sp.r_col
    it_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    prob = 2e-2
    fg = cn.make_fault(seed=cfg.seed, layer=0, mode=cn.FAULT_BERNOULLI, p=prob, sigma=cfg.sigma, iteration_dev=it_dev)
    fo = orc.make_fault(seed=cfg.seed, layer=0, mode=orc.FAULT_BERNOULLI, p=prob, sigma=cfg.sigma)
    rep = cn.new_reports(2)
    rng = np.random.default_rng(5)
    rows = rng.integers(0, sp.n_out, 48)
    cols = rng.integers(0, sp.n_in, 48)
    Wr, Wc = W[rows].astype(np.float64), W[:, cols].astype(np.float64)   # the sampled rows and columns only
    lr = cfg.lr
    seen_hit = 0
    for it in range(2):
        X = wl.gaussian_inputs(B, sp.n_in, seed=21, iteration=it)
        D = wl.gaussian_inputs(B, sp.n_out, seed=22, iteration=it) / np.float32(B)
        it_dev.fill_(it)
        S = cn.forward(g, _dev(X), fault=fg, rep_dev=rep[:cn.REPORT_BYTES])
        C = cn.backward_update(g, _dev(D), _dev(X), lr, fault=fg, rep_dev=rep[cn.REPORT_BYTES:])
        rf, rb = cn.read_reports(rep)
        # injection plan: the oracle's hit test, node by node
        for phase, r, n_cw, K in ((0, rf, sp.n, M), (1, rb, sp.m, Nn)):
            for cw in range(n_cw):
                mask = 0
                for k in range(K):
                    i, j = (k, cw) if phase == 0 else (cw, k)
                    if orc.node_hit(fo, phase, it, i * Nn + j, 0, n_cw * K):
                        mask |= 1 << k
                assert r.injected_mask[cw] == mask, (it, phase, cw)
                assert r.flagged_mask[cw] == mask, (it, phase, cw)      # located exactly the hit nodes
                seen_hit += mask != 0
            assert r.status != cn.TIMEOUT
            if any(r.injected_mask):
                assert r.min_margin_hit > 10.0
            assert r.max_margin_clean < 0.1
        # sampled entries from the definitions (float64); corrected or fault-free values either way
        X64, D64 = X.astype(np.float64), D.astype(np.float64)
        Sref = X64 @ Wr.T
        Cref = D64 @ Wc
        Sg, Cg = S.cpu().numpy()[:, rows], C.cpu().numpy()[:, cols]
        # An output rebuilt by erasure decoding carries the storage rounding of the parity blocks times
        # the conditioning of the erasure system (the oracle's value has the same deviation from the exact
        # product; GPU against oracle is compared in the scaled test): those entries get a loose bound.
        b_r, b_c = -(-sp.n_out // sp.m), -(-sp.n_in // sp.n)
        dec_rows = {k for cw in range(sp.n) for k in range(sp.m) if (rf.flagged_mask[cw] >> k) & 1}
        dec_cols = {k for cw in range(sp.m) for k in range(sp.n) if (rb.flagged_mask[cw] >> k) & 1}
        loose = 0.15 if cfg.bf16 else 1e-3
        bf = np.array([loose if (r // b_r) in dec_rows else tol for r in rows])
        bb = np.array([loose if (c // b_c) in dec_cols else tol for c in cols])
        assert np.all(np.max(np.abs(Sg - Sref), axis=0) / np.max(np.abs(Sref)) <= bf), it
        assert np.all(np.max(np.abs(Cg - Cref), axis=0) / np.max(np.abs(Cref)) <= bb), it
        # W += lr * delta^T x on the sampled rows and columns
        Wr += lr * (D64[:, rows].T @ X64)
        Wc += lr * (D64.T @ X64[:, cols])
        if cfg.bf16:   # a data block is stored rounded after every update
            Wr, Wc = wl.bf16_round(Wr).astype(np.float64), wl.bf16_round(Wc).astype(np.float64)
    Wg = cn.decode_weights(g).float().cpu().numpy()
    assert np.linalg.norm(Wg[rows] - Wr) / np.linalg.norm(Wr) <= (4e-3 if cfg.bf16 else 1e-3)
    assert np.linalg.norm(Wg[:, cols] - Wc) / np.linalg.norm(Wc) <= (4e-3 if cfg.bf16 else 1e-3)
    # the parity blocks follow the data blocks up to the operand rounding of the update term (2^-9 bfloat16,
    # 2^-11 TF32) and, with bfloat16 storage, one storage rounding per block
    assert cn.check_invariance(g) < (5e-2 if cfg.bf16 else 1e-3)
    assert seen_hit > 0
    g.free()


def test_config4_full_size_sampled(cn, orc):
    """16384x16384 bfloat16, 8x8 + 2 + 2 Gaussian code, batch 128, tensor-core tiles."""
    _sampled_full_size_layer(cn, orc, wl.config("c4"), 2, TOL_LOWP)


def test_config5_full_size_layer_sampled(cn, orc):
    """One 4096x4096 fp32 layer of configuration 5, 4x4 + 1 + 1, batch 64, TF32 tensor-core tiles."""
    _sampled_full_size_layer(cn, orc, wl.config("c5"), 1, TOL_LOWP)
