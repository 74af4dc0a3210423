"""Pins of the CPU oracle against what the paper (arXiv 2407.04480) and the mathematics fix.

None of these tests touches the CUDA library.  Each names the statement it checks.
"""
import dataclasses
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import loco_definition as defn
from oracle import loco_oracle as orc
from oracle.loco_oracle import OracleConfig

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
RNG = np.random.default_rng(20240704)


def qrange(p):
    return -(2 ** (p - 1)), 2 ** (p - 1) - 1


def run_steps(cfg, grads, k0=1):
    """Run consecutive send steps k0, k0+1, ... on one worker; return the per-step traces and final state."""
    n = grads[0].size
    state = orc.new_state(cfg, n)
    comm = orc.new_comm(cfg, n)
    traces = []
    for i, g in enumerate(grads):
        (_, _), tr = orc.send_step(cfg, g, state, comm, k0 + i, trace=True)
        traces.append(tr)
    return traces, state, comm


# ------------------------------------------------------------------ Eq. 1: the compressor

@pytest.mark.parametrize("p", [2, 4, 8])
def test_code_range(p):
    """Text under Eq. 1: codes lie in [-2^(p-1), 2^(p-1)-1]."""
    x = np.concatenate([RNG.normal(0, 1, 4096), [1e30, -1e30, np.inf, -np.inf, 0.0]]).astype(np.float32)
    q = orc.compressor(x, 3.0, p)
    lo, hi = qrange(p)
    assert q.min() == lo and q.max() == hi
    assert np.all((q >= lo) & (q <= hi))


@pytest.mark.parametrize("p", [2, 4, 8])
@pytest.mark.parametrize("s", [4.0, 2.0 ** 11, 2.0 ** 19, 6.0 * 2 ** 11, 1000.0])
def test_half_step_bound_and_saturation(p, s):
    """Lemma "round": |x - C(x)| <= 1/(2s) inside the range; outside, C(x) is the end of the range
    and the error is |x| minus that end."""
    lo, hi = qrange(p)
    x = (RNG.normal(0, 1.0, 20000) * (hi + 2) / s / 2).astype(np.float32)
    q = orc.compressor(x, s, p).astype(np.float64)
    Cx = q / s
    x64 = x.astype(np.float64)
    # x*s is rounded once to fp32 before the nearest-integer step: allow that half-ulp in the bound
    slack = np.abs(x64) * 2.0 ** -24 + 1e-300
    inside = (x64 * s >= lo - 0.5) & (x64 * s <= hi + 0.5)
    assert np.all(np.abs(x64 - Cx)[inside] <= 0.5 / s + slack[inside])
    above, below = x64 * s > hi + 0.5, x64 * s < lo - 0.5
    assert above.any() and below.any()
    assert np.all(q[above] == hi) and np.all(q[below] == lo)
    assert np.allclose((x64 - Cx)[above], x64[above] - hi / s, rtol=0, atol=1e-12)
    assert np.allclose((Cx - x64)[below], lo / s - x64[below], rtol=0, atol=1e-12)


@pytest.mark.parametrize("p", [2, 4, 8])
def test_brute_force_nearest_code(p):
    """Eq. 1's text: the nearest integer within the range.  Brute force over all 2^p codes; a tie
    between two integers goes to the even one."""
    s = 2.0 ** 7
    lo, hi = qrange(p)
    codes = np.arange(lo, hi + 1, dtype=np.float64)
    ties = (np.arange(lo - 2, hi + 2) + 0.5) / s
    x = np.concatenate([RNG.uniform(lo - 3, hi + 3, 5000) / s, ties, codes / s]).astype(np.float32)
    q = orc.compressor(x, s, p)
    y = x.astype(np.float64) * s                      # exact: s is a power of two
    dist = np.abs(y[:, None] - codes[None, :])
    best = dist.min(axis=1)
    for yi, qi, row, b in zip(y, q, dist, best):
        cands = codes[row == b]
        if len(cands) == 1:
            assert qi == cands[0]
        else:                                         # exact tie inside the range
            assert qi in cands and qi % 2 == 0, (yi, qi, cands)


@pytest.mark.parametrize("p,s", [(4, 2.0 ** 19), (8, 6 * 2.0 ** 19), (4, 37.5), (2, 2.0 ** 17)])
def test_matches_pytorch_default_rounding(p, s):
    """Eq. 1's text calls it the default quantisation in PyTorch: round, then clamp."""
    lo, hi = qrange(p)
    x = (RNG.normal(0, 1, 50000) * 6.0 / s).astype(np.float32)
    x[:200] = ((np.arange(200) - 100) + 0.5) / np.float32(s)
    want = torch.clamp(torch.round(torch.from_numpy(x) * torch.tensor(s, dtype=torch.float32)), lo, hi)
    assert np.array_equal(orc.compressor(x, s, p), want.numpy().astype(np.int32))


@pytest.mark.parametrize("p", [2, 4, 8])
def test_idempotent_on_the_grid(p):
    """C(C(x)) = C(x): a value already on the grid is reproduced (follows from Eq. 1)."""
    s = 2.0 ** 10
    x = (RNG.normal(0, 1, 4096) * 4 / s).astype(np.float32)
    q1 = orc.compressor(x, s, p)
    c1 = orc.decompressor(q1, s)
    q2 = orc.compressor(c1, s, p)
    assert np.array_equal(q1, q2)
    assert np.array_equal(orc.decompressor(q2, s), c1)


def test_round_trip_all_codes():
    """comp(dec(q)) = q for every code, for power-of-two and other scales."""
    for p in (2, 4, 8):
        lo, hi = qrange(p)
        q = np.arange(lo, hi + 1, dtype=np.int32)
        for s in (2.0 ** 19, 2.0 ** 17, 6 * 2.0 ** 19, 3.0, 1e-3):
            assert np.array_equal(orc.compressor(orc.decompressor(q, s), s, p), q)


def test_decompressor_is_division():
    """Eq. 1, second line: float(q) / s (IEEE division, not a rounded reciprocal)."""
    q = np.arange(-128, 128, dtype=np.int32)
    for s in (6 * 2.0 ** 19, 3.0, 7.0):
        want = (q.astype(np.float32) / np.float32(s)).astype(np.float32)
        assert np.array_equal(orc.decompressor(q, s), want)


# ------------------------------------------------------------------ Algorithm 1: worked example

def load_golden(name):
    rec = {}
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, *v = line.split()
        rec[k] = v
    return rec


def test_hand_worked_example():
    """tests/golden/alg1_worked_example.txt: two iterations of Algorithm 1 worked by hand."""
    G = load_golden("alg1_worked_example.txt")
    f = lambda k: np.array([float(v) for v in G[k]], dtype=np.float32)
    cfg = OracleConfig(bits=int(G["p"][0]), s=float(G["s"][0]), s_e=float(G["s_e"][0]),
                       beta=float(G["beta"][0]), reset_period=0, state_fmt=orc.STATE_INT8)
    n = 6
    state, comm = orc.new_state(cfg, n), orc.new_comm(cfg, n)
    comms = []
    for k, tag in ((1, "1"), (2, "2")):
        (flags, sat, ssat), tr = orc.send_step(cfg, f("g" + tag), state, comm, k, trace=True, full_status=True)
        nxt = str(k + 1)
        assert flags == 0 and sat == int(G["sat" + tag][0]) and ssat == int(G["ssat" + tag][0])
        assert np.array_equal(tr["h"], f("h" + tag))
        assert np.array_equal(tr["q"], f("q" + tag).astype(np.int32))
        assert np.array_equal(tr["d"], f("d" + tag))
        assert np.array_equal(tr["e_new"], f("et" + nxt))
        assert np.array_equal(state[:n].view(np.int8), f("e" + nxt).astype(np.int8))
        comms.append(comm.copy())
    assert [int(b) for b in comms[0][:3]] == [int(v, 16) for v in G["packed1"]]
    assert np.array_equal(orc.reduce(cfg, n, comms), f("mean"))


# ------------------------------------------------------------------ Algorithm 1: invariants

def dyadic(n, bits, scale):
    """Values m * scale with |m| < 2^bits: sums and products by powers of two stay exact in fp32."""
    return (RNG.integers(-(2 ** bits), 2 ** bits, n) * scale).astype(np.float32)


@pytest.mark.parametrize("fmt", [orc.STATE_INT8, orc.STATE_FP32, orc.STATE_FP32_Q8COMP])
def test_identity_compression_keeps_zero_error(fmt):
    """If every g*s is an integer inside the range, compression loses nothing: d = g and e~ stays 0."""
    s = 2.0 ** 9
    cfg = OracleConfig(bits=4, s=s, s_e=4 * s, beta=0.3, reset_period=0, state_fmt=fmt)
    grads = [(RNG.integers(-8, 8, 257) / s).astype(np.float32) for _ in range(5)]
    traces, state, _ = run_steps(cfg, grads)
    for g, tr in zip(grads, traces):
        assert np.array_equal(tr["d"], g) and not tr["e_new"].any()
    assert not state.any()


def test_beta_one_is_classic_error_feedback():
    """Eq. 4 versus Eq. 5: with beta = 1 the new error is h - d of this iteration alone, so the
    sum of what was sent equals the sum of the gradients minus the last error."""
    s = 2.0 ** 6
    cfg = OracleConfig(bits=4, s=s, s_e=4 * s, beta=1.0, reset_period=0, state_fmt=orc.STATE_FP32)
    grads = [dyadic(64, 6, 2.0 ** -10) for _ in range(6)]
    traces, state, _ = run_steps(cfg, grads)
    for tr in traces:
        assert np.array_equal(tr["e_new"], tr["h"] - tr["d"])
    sent = np.sum([t["d"].astype(np.float64) for t in traces], axis=0)
    want = np.sum([g.astype(np.float64) for g in grads], axis=0) - state.view(np.float32)[:64]
    assert np.array_equal(sent, want)


@pytest.mark.parametrize("variant", ["state_none", "beta_zero"])
def test_no_feedback_is_plain_quantisation(variant):
    """Ablation row without error feedback: the output is compressor(g) and nothing carries over."""
    s = 2.0 ** 11
    cfg = OracleConfig(bits=4, s=s, s_e=4 * s, beta=0.0, reset_period=0,
                       state_fmt=orc.STATE_NONE if variant == "state_none" else orc.STATE_INT8)
    grads = [(RNG.normal(0, 1e-3, 300)).astype(np.float32) for _ in range(3)]
    traces, state, _ = run_steps(cfg, grads)
    for g, tr in zip(grads, traces):
        assert np.array_equal(tr["q"], orc.compressor(g, s, 4))
    assert not state.any()


@pytest.mark.parametrize("beta", [0.5, 0.25, 0.75])
def test_closed_form_unrolling(beta):
    """Eq. 5 unrolled from e~_0 = 0 without reset: e~_K = beta * sum_i (1-beta)^(K-i) * delta_i."""
    s = 2.0 ** 8
    cfg = OracleConfig(bits=4, s=s, s_e=4 * s, beta=beta, reset_period=0, state_fmt=orc.STATE_FP32)
    K = 4
    grads = [(RNG.normal(0, 2e-2, 8)).astype(np.float32) for _ in range(K)]
    traces, state, _ = run_steps(cfg, grads)
    deltas = [t["delta"].astype(np.float64) for t in traces]
    want = beta * sum((1 - beta) ** (K - 1 - i) * deltas[i] for i in range(K))
    got = state.view(np.float32)[:8].astype(np.float64)
    assert np.allclose(got, want, rtol=1e-6, atol=1e-12)
    assert np.abs(want).max() > 0


@pytest.mark.parametrize("fmt,beta", [(orc.STATE_FP32, 0.5), (orc.STATE_FP32, 0.1),
                                      (orc.STATE_FP32_Q8COMP, 0.5), (orc.STATE_FP32_Q8COMP, 0.25),
                                      (orc.STATE_INT8, 0.5), (orc.STATE_INT8, 1.0)])
def test_lemma_1_identity(fmt, beta):
    """Lemma 1, per element and worker:
         d_k = g_k + (e~_k - e~_{k+1})/beta + e^_k - e~_k,   e^_k = dec(comp(e~_k; s_e, 8); s_e).
    With fp32 storage used as it is, e^ = e~.  With only the 8-bit state stored, e~_k is its image
    e^_k, which leaves d_k - g_k = (e^_k - e~_{k+1})/beta."""
    s = 2.0 ** 9
    s_e = 4 * s
    cfg = OracleConfig(bits=4, s=s, s_e=s_e, beta=beta, reset_period=0, state_fmt=fmt)
    n, K = 96, 6
    grads = [(RNG.normal(0, 6e-3, n)).astype(np.float32) for _ in range(K)]
    state = orc.new_state(cfg, n)
    comm = orc.new_comm(cfg, n)
    seen_nonzero = False
    for k, g in enumerate(grads, start=1):
        before = state.copy()
        (_, _), tr = orc.send_step(cfg, g, state, comm, k, trace=True)
        g64, d64 = g.astype(np.float64), tr["d"].astype(np.float64)
        e_next = tr["e_new"].astype(np.float64)
        if fmt == orc.STATE_INT8:
            e_hat = before[:n].view(np.int8).astype(np.float64) / s_e
            e_prev = e_hat
        else:
            e_prev = before.view(np.float32)[:n].astype(np.float64)
            e_hat = e_prev if fmt == orc.STATE_FP32 else defn.decompressor(defn.compressor(e_prev, s_e, 8), s_e)
        want = g64 + (e_prev - e_next) / beta + e_hat - e_prev
        assert np.allclose(d64, want, rtol=0, atol=4e-7 / beta * 6e-3 + 1e-9)
        seen_nonzero |= bool(np.abs(e_hat).max() > 0)
    assert seen_nonzero


def test_lemma_1_identity_detects_swapped_beta():
    """The identity above is sharp enough to catch Eq. 5 written with beta and 1-beta exchanged
    (the mistake is planted in a copy of the double-precision definition, not in any product code)."""
    s, s_e, beta = 2.0 ** 9, 2.0 ** 11, 0.25
    g = RNG.normal(0, 6e-3, 64)
    e_prev = RNG.normal(0, 1e-3, 64)
    q, d, h, e_next, _, _ = defn.loco_step(g, e_prev, None, 1, s=s, s_e=s_e, beta=beta, T_c=0, state="fp32")
    assert np.allclose(d, g + (e_prev - e_next) / beta, rtol=0, atol=1e-12)
    wrong_next = beta * e_prev + (1 - beta) * (h - d)
    assert not np.allclose(d, g + (e_prev - wrong_next) / beta, rtol=0, atol=1e-6)


def test_errors_do_not_accumulate():
    """Proof of Lemma 2 (and Eq. 6): with fp32 storage the sum telescopes exactly,
         sum_{i<=K} (d_i - g_i) = (e~_0 - e~_K)/beta;
    with the 8-bit state each iteration adds at most one half step 1/(2 s_e) of the state grid."""
    s, beta, n, K = 2.0 ** 9, 0.5, 128, 40
    s_e = 4 * s
    grads = [(RNG.normal(0, 5e-3, n)).astype(np.float32) for _ in range(K)]
    gsum = np.sum([g.astype(np.float64) for g in grads], axis=0)
    # fp32 state: exact telescoping
    cfg = OracleConfig(bits=4, s=s, s_e=s_e, beta=beta, reset_period=0, state_fmt=orc.STATE_FP32)
    traces, state, _ = run_steps(cfg, grads)
    dsum = np.sum([t["d"].astype(np.float64) for t in traces], axis=0)
    assert np.allclose(dsum - gsum, -state.view(np.float32)[:n].astype(np.float64) / beta, rtol=0, atol=1e-7)
    # 8-bit state: bounded drift
    cfg8 = OracleConfig(bits=4, s=s, s_e=s_e, beta=beta, reset_period=0, state_fmt=orc.STATE_INT8)
    traces8, _, _ = run_steps(cfg8, grads)
    dsum8 = np.sum([t["d"].astype(np.float64) for t in traces8], axis=0)
    last = traces8[-1]["e_new"].astype(np.float64)
    assert np.all(np.abs(dsum8 - gsum) <= np.abs(last) / beta + K * 0.5 / s_e / beta + 1e-9)
    # and a plain quantiser without feedback drifts further than that on at least one element
    plain = np.sum([orc.decompressor(orc.compressor(g, s, 4), s).astype(np.float64) for g in grads], axis=0)
    assert np.abs(plain - gsum).max() > np.abs(dsum - gsum).max()


def test_error_bound_after_reset():
    """Lemma "err_bound", first case: the first error after a reset is at most beta/(2s) wherever
    h stayed inside the range, and beta*(|h| - end of range) where it saturated."""
    s, beta = 2.0 ** 9, 0.5
    cfg = OracleConfig(bits=4, s=s, s_e=4 * s, beta=beta, reset_period=4, state_fmt=orc.STATE_FP32)
    n = 512
    grads = [(RNG.normal(0, 8e-3, n)).astype(np.float32) for _ in range(6)]
    state, comm = orc.new_state(cfg, n), orc.new_comm(cfg, n)
    for k, g in enumerate(grads):
        (_, _), tr = orc.send_step(cfg, g, state, comm, k, trace=True)
        if k % 4 == 1:                                   # first iteration after the reset at k % T_c == 0
            h = tr["h"].astype(np.float64)
            assert np.array_equal(tr["h"], g)            # compensation was zero
            inside = (h * s >= -8.5) & (h * s <= 7.5)
            e = np.abs(tr["e_new"].astype(np.float64))
            assert np.all(e[inside] <= beta / (2 * s) + 1e-12)
            assert (~inside).any()
            bound = np.where(h > 0, 7 / s, 8 / s)
            assert np.allclose(e[~inside], beta * (np.abs(h[~inside]) - bound[~inside]), rtol=1e-6, atol=1e-12)


@pytest.mark.parametrize("fmt", [orc.STATE_INT8, orc.STATE_FP32, orc.STATE_FP32_Q8COMP])
def test_reset_rule(fmt):
    """Eq. 7 / Algorithm 1: e_{k+1} = 0 exactly when k % T_c == 0 (the caller's 0-based k); the codes
    of that iteration are still compensated with e_k."""
    s = 2.0 ** 9
    cfg = OracleConfig(bits=4, s=s, s_e=4 * s, beta=0.5, reset_period=3, state_fmt=fmt)
    n = 200
    state, comm = orc.new_state(cfg, n), orc.new_comm(cfg, n)
    for k in range(8):
        g = RNG.normal(0, 6e-3, n).astype(np.float32)
        before_nonzero = bool(state.any())
        (_, _), tr = orc.send_step(cfg, g, state, comm, k, trace=True)
        if k % 3 == 0:
            assert not state.any()
            if before_nonzero:
                assert np.abs(tr["c"]).max() > 0 and np.array_equal(tr["h"], g + tr["c"])
        else:
            assert state.any()
    cfg0 = OracleConfig(bits=4, s=s, s_e=4 * s, beta=0.5, reset_period=0, state_fmt=fmt)
    state = orc.new_state(cfg0, n)
    orc.send_step(cfg0, RNG.normal(0, 6e-3, n).astype(np.float32), state, comm, 0)
    assert state.any()                                   # T_c = 0: never reset


def test_int8_state_matches_definition_on_exact_inputs():
    """On dyadic inputs every fp32 operation is exact, so the fp32 oracle must reproduce the
    double-precision definition bit for bit (codes, state codes, d)."""
    s, s_e, beta = 2.0 ** 6, 2.0 ** 8, 0.5
    cfg = OracleConfig(bits=4, s=s, s_e=s_e, beta=beta, reset_period=5, state_fmt=orc.STATE_INT8)
    n = 300
    state, comm = orc.new_state(cfg, n), orc.new_comm(cfg, n)
    e_code = np.zeros(n)
    for k in range(12):
        g = dyadic(n, 7, 2.0 ** -10)
        (_, _), tr = orc.send_step(cfg, g, state, comm, k, trace=True)
        q, d, h, e_next, _, e_code = defn.loco_step(g, None, e_code, k, s=s, s_e=s_e, beta=beta, T_c=5)
        assert np.array_equal(tr["q"], q) and np.array_equal(tr["d"], d) and np.array_equal(tr["h"], h)
        assert np.array_equal(tr["e_new"], e_next)
        assert np.array_equal(state[:n].view(np.int8), e_code)


# ------------------------------------------------------------------ Eq. 8: the average

def make_comms(cfg, n, N, sigma=2e-3):
    comms, ds = [], []
    for w in range(N):
        g = RNG.normal(0, sigma, n).astype(np.float32)
        if cfg.grad_dtype == orc.BF16:
            g = orc.f32_to_bf16_bits(g)
        state, comm = orc.new_state(cfg, n), orc.new_comm(cfg, n)
        (_, _), tr = orc.send_step(cfg, g, state, comm, 1, trace=True)
        comms.append(comm)
        ds.append(tr["d"])
    return comms, ds


@pytest.mark.parametrize("N", [1, 2, 3, 8, 16])
@pytest.mark.parametrize("mode", [orc.SCALE_FIXED, orc.SCALE_BLOCK_ABSMAX])
def test_average_is_the_mean(N, mode):
    """Eq. 8: (1/N) * sum_n dec(h~^n), computed after dequantisation in high precision."""
    n = 1000
    cfg = OracleConfig(bits=4, scale_mode=mode, block_size=64, s=2.0 ** 10, s_e=2.0 ** 12, num_partitions=1,
                       reset_period=0)
    comms, ds = make_comms(cfg, n, N)
    got = orc.reduce(cfg, n, comms).astype(np.float64)
    want = defn.average(ds)
    assert np.allclose(got, want, rtol=1e-6, atol=1e-9)
    same = orc.reduce(cfg, n, [comms[0]] * N)
    assert np.allclose(same, ds[0], rtol=1e-6, atol=0)      # N identical workers give d back
    if mode == orc.SCALE_FIXED and N in (1, 2, 8, 16):
        assert np.array_equal(same, ds[0])                   # exactly: few-bit codes, 1/N a power of two


def test_average_all_code_pairs():
    """Brute force for N = 2: every pair of 4-bit codes averages to (a + b) / (2 s)."""
    s = 2.0 ** 5
    cfg = OracleConfig(bits=4, s=s, s_e=4 * s, state_fmt=orc.STATE_NONE, reset_period=0)
    pairs = np.array(list(itertools.product(range(-8, 8), repeat=2)), dtype=np.float32)
    n = len(pairs)
    comms = []
    for col in (0, 1):
        comm = orc.new_comm(cfg, n)
        orc.send_step(cfg, (pairs[:, col] / np.float32(s)).astype(np.float32), orc.new_state(cfg, n), comm, 1)
        comms.append(comm)
    got = orc.reduce(cfg, n, comms)
    assert np.array_equal(got, (pairs[:, 0] + pairs[:, 1]) / (2 * s))


def test_partitions_cover_the_vector():
    """Sec. 3.3: the vector is cut into N parts; reducing part j of every worker gives part j of the
    full average, and the parts together give all of it."""
    n, P = 5000, 4
    cfg = OracleConfig(bits=4, s=2.0 ** 10, s_e=2.0 ** 12, num_partitions=P, reset_period=0, out_dtype=orc.BF16)
    comms, ds = make_comms(cfg, n, 3)
    whole = orc.reduce(cfg, n, comms)
    parts = [orc.reduce(cfg, n, comms, first=j, count=1) for j in range(P)]
    assert sum(p.size for p in parts) == n and np.array_equal(np.concatenate(parts), whole)
    cfg1 = OracleConfig(bits=4, s=2.0 ** 10, s_e=2.0 ** 12, num_partitions=1, reset_period=0, out_dtype=orc.BF16)
    flat = []
    for d in ds:                                              # same codes, unpartitioned layout
        comm = orc.new_comm(cfg1, n)
        orc.send_step(OracleConfig(**{**cfg1.__dict__, "state_fmt": orc.STATE_NONE}), d, orc.new_state(cfg1, n), comm, 1)
        flat.append(comm)
    assert np.array_equal(orc.reduce(cfg1, n, flat), whole)
    want = orc.f32_to_bf16_bits(defn.average(ds).astype(np.float32))
    assert np.mean(whole == want) > 0.99                      # bf16 output is the rounded mean


# ------------------------------------------------------------------ storage

def test_storage_sizes():
    """Table 1's text: the error state costs one byte per parameter, the gradient 4 bits on the wire."""
    n = 25_000_000
    cfg = OracleConfig(bits=4, num_partitions=8)
    assert n <= orc.state_bytes(cfg, n) < n + 256
    assert n // 2 <= orc.packed_bytes(cfg, n) <= n // 2 + 8 * (128 + 128)
    assert orc.state_bytes(OracleConfig(state_fmt=orc.STATE_NONE), n) == 0
    assert orc.state_bytes(OracleConfig(state_fmt=orc.STATE_FP32), n) == 4 * n
    blk = OracleConfig(bits=4, scale_mode=orc.SCALE_BLOCK_ABSMAX, block_size=256, num_partitions=8)
    assert orc.packed_bytes(blk, n) >= n // 2 + 4 * (n // 256)
    for cfg_ in (cfg, blk):
        assert sum(orc.partition_elems(cfg_, n, j) for j in range(8)) == n
        assert orc.partition_bytes(cfg_, n) % 128 == 0 and orc.partition_capacity(cfg_, n) % 256 == 0
    assert orc.packed_bytes(cfg, 0) == 0 and orc.state_bytes(cfg, 0) == 0


@pytest.mark.parametrize("p", [2, 4, 8])
def test_packing_all_byte_values(p):
    """Brute force over all 256 byte values: unpack then pack reproduces the byte, fields are two's
    complement, element i sits at bit (i mod 8/p)*p of byte i*p/8 (little end first)."""
    per = 8 // p
    lo, hi = qrange(p)
    for b in range(256):
        q = orc.unpack_codes(np.array([b], np.uint8), per, p)
        assert np.all((q >= lo) & (q <= hi))
        assert orc.pack_codes(q, p)[0] == b
        for i in range(per):
            field = (b >> (i * p)) & (2 ** p - 1)
            assert q[i] == (field - 2 ** p if field >= 2 ** (p - 1) else field)


def test_packing_all_code_tuples_of_a_tiny_block():
    """Brute force: all 16^3 code triples survive pack / unpack through the partitioned layout."""
    cfg = OracleConfig(bits=4, s=1.0, s_e=4.0, state_fmt=orc.STATE_NONE, reset_period=0, num_partitions=1)
    triples = np.array(list(itertools.product(range(-8, 8), repeat=3)), dtype=np.float32).ravel()
    comm = orc.new_comm(cfg, triples.size, fill=0xAA)
    orc.send_step(cfg, triples, orc.new_state(cfg, triples.size), comm, 1)
    codes, _ = orc.comm_views(cfg, triples.size, comm)[0]
    assert np.array_equal(orc.unpack_codes(codes, triples.size, 4), triples.astype(np.int32))
    assert not codes[(triples.size + 1) // 2:].any()          # padding elements carry code 0


# ------------------------------------------------------------------ block-scaled extension, non-finite

def test_block_absmax_properties():
    """Extension without counterpart in the paper: per block, scale = amax/qmax, the largest element
    maps to +-qmax, an all-zero block has scale 0 and codes 0, and Lemma 1's identity still holds."""
    n, B = 1000, 64
    cfg = OracleConfig(bits=4, scale_mode=orc.SCALE_BLOCK_ABSMAX, block_size=B, beta=0.5, reset_period=0,
                       state_fmt=orc.STATE_FP32)
    g = RNG.normal(0, 1e-3, n).astype(np.float32)
    g[128:192] = 0
    state, comm = orc.new_state(cfg, n), orc.new_comm(cfg, n)
    (_, sat), tr = orc.send_step(cfg, g, state, comm, 1, trace=True)
    codes, scales = orc.comm_views(cfg, n, comm)[0]
    assert sat == 0 and scales[2] == 0 and not tr["q"][128:192].any()
    for b in range((n + B - 1) // B):
        blk = slice(b * B, min((b + 1) * B, n))
        amax = np.abs(g[blk]).max()
        assert scales[b] == np.float32(amax) / np.float32(7)
        if amax > 0:
            assert np.abs(tr["q"][blk]).max() == 7 and tr["q"][blk].min() >= -7
            assert np.all(np.abs(tr["delta"][blk]) <= scales[b] / 2 * (1 + 1e-6))
    e_next = state.view(np.float32)[:n].astype(np.float64)
    assert np.allclose(tr["d"].astype(np.float64), g - e_next / 0.5, rtol=0, atol=1e-9)


def test_non_finite_inputs():
    """Reading for inputs the paper's boundedness assumption excludes: NaN -> code 0, +-Inf -> the end
    of the range, the element's error is taken as 0, and a flag is raised."""
    cfg = OracleConfig(bits=4, s=2.0 ** 10, s_e=2.0 ** 12, beta=0.5, reset_period=0, state_fmt=orc.STATE_FP32)
    g = np.array([np.nan, np.inf, -np.inf, 1e-3, 3e38], dtype=np.float32)
    state, comm = orc.new_state(cfg, 5), orc.new_comm(cfg, 5)
    (flags, sat), tr = orc.send_step(cfg, g, state, comm, 1, trace=True)
    assert flags & orc.FLAG_NONFINITE
    assert list(tr["q"]) == [0, 7, -8, 1, 7] and sat == 1
    e = state.view(np.float32)[:5]
    assert e[0] == 0 and e[1] == 0 and e[2] == 0 and np.isfinite(e).all()


# ---------------------------------------------------------------- Adam-family step fused behind Eq. 8

def _codes_to_comm(cfg, qs):
    """A one-partition communication buffer holding the given codes (via the oracle's own packing routine)."""
    n = len(qs)
    comm = orc.new_comm(cfg, n)
    packed = orc.pack_codes(np.asarray(qs, dtype=np.int32), cfg.bits)
    comm[:packed.size] = packed
    return comm


def test_adam_family_hand_worked_example():
    ex = {}
    for line in open(os.path.join(GOLDEN, "adam_family_worked_example.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, *vals = line.split()
        ex[k] = [float(x) for x in vals]
    cfg = orc.OracleConfig(bits=int(ex["p"][0]), s=ex["s"][0], state_fmt=orc.STATE_NONE, grad_dtype=orc.F32, out_dtype=orc.F32)
    comms = [_codes_to_comm(cfg, [int(q) for q in ex["qa"]]), _codes_to_comm(cfg, [int(q) for q in ex["qb"]])]
    m, v, th = (np.array(ex[k], dtype=np.float32) for k in ("m0", "v0", "theta0"))
    g = orc.reduce_adam(cfg, 4, comms, m, v, th, lr=ex["eta"][0], beta1=ex["beta1"][0], beta2=ex["beta2"][0],
                        delta=ex["delta"][0], want_grad=True)
    assert g.tolist() == ex["g"] and m.tolist() == ex["m1"] and v.tolist() == ex["v1"] and th.tolist() == ex["theta1"]


def test_adam_family_sign_update_special_case():
    """beta1 = beta2 = 1, delta = 0: m = g, v = g^2, so theta moves by eta * sign(g) wherever g != 0 (up to the
    rounding of the square, the root, the quotient and the product: a few ulp of eta)."""
    rng = np.random.default_rng(3)
    n = 4096
    cfg = orc.OracleConfig(bits=4, s=2.0 ** 6, state_fmt=orc.STATE_NONE, grad_dtype=orc.F32, out_dtype=orc.F32)
    comms = [_codes_to_comm(cfg, rng.integers(-8, 8, n)) for _ in range(3)]
    g = orc.reduce(cfg, n, comms)
    m, v = rng.normal(size=n).astype(np.float32), rng.random(n).astype(np.float32)
    th0 = rng.normal(size=n).astype(np.float32)
    th = th0.copy()
    orc.reduce_adam(cfg, n, comms, m, v, th, lr=0.125, beta1=1.0, beta2=1.0, delta=0.0)
    nz = g != 0
    assert nz.sum() > n // 2
    assert np.array_equal(m, g) and np.array_equal(v, g * g)
    step = (th0.astype(np.float64) - th.astype(np.float64))
    assert np.allclose(step[nz], 0.125 * np.sign(g[nz]), rtol=0, atol=1e-6)
    assert np.array_equal(th[~nz], th0[~nz]) or np.isnan(th[~nz]).all()      # g = 0: 0/0, the update is undefined there


def test_adam_family_constant_gradient_closed_form():
    """From m = v = 0 under a constant gradient: m_k = (1 - (1-b1)^k) g, v_k = (1 - (1-b2)^k) g^2."""
    n, K, b1, b2 = 64, 6, 0.1, 0.01
    cfg = orc.OracleConfig(bits=8, s=2.0 ** 4, state_fmt=orc.STATE_NONE, grad_dtype=orc.F32, out_dtype=orc.F32)
    comms = [_codes_to_comm(cfg, np.arange(-32, 32))]
    g = orc.reduce(cfg, n, comms).astype(np.float64)
    m, v, th = np.zeros(n, np.float32), np.zeros(n, np.float32), np.ones(n, np.float32)
    th64 = np.ones(n)
    for k in range(1, K + 1):
        orc.reduce_adam(cfg, n, comms, m, v, th, lr=1e-3, beta1=b1, beta2=b2, delta=1e-8)
        mk, vk = (1 - (1 - b1) ** k) * g, (1 - (1 - b2) ** k) * g * g
        th64 = th64 - 1e-3 / np.sqrt(vk + 1e-8) * mk
        assert np.allclose(m, mk, rtol=1e-5, atol=1e-9) and np.allclose(v, vk, rtol=1e-5, atol=1e-12)
    assert np.allclose(th, th64, rtol=1e-5, atol=1e-7)


def test_adam_family_matches_float64_definition_and_unfused_path():
    """Random moments and codes: the fused step equals Eq. 8 followed by the float64 formulas; a swapped beta, a
    missing square or delta outside the root would all break the tolerance."""
    rng = np.random.default_rng(11)
    n = 5000
    for mode in (orc.SCALE_FIXED, orc.SCALE_BLOCK_ABSMAX):
        cfg = orc.OracleConfig(bits=4, scale_mode=mode, block_size=64, s=2.0 ** 10, s_e=2.0 ** 12, state_fmt=orc.STATE_NONE,
                               grad_dtype=orc.F32, out_dtype=orc.BF16, num_partitions=3)
        comms = []
        for w in range(4):
            comm = orc.new_comm(cfg, n)
            orc.send_step(cfg, rng.normal(0, 2e-3, n).astype(np.float32), orc.new_state(cfg, n), comm, 1)
            comms.append(comm)
        cfg32 = dataclasses.replace(cfg, out_dtype=orc.F32)
        g = orc.reduce(cfg32, n, comms).astype(np.float64)
        m0, v0, th0 = rng.normal(0, 1e-3, n).astype(np.float32), (rng.random(n) * 1e-6).astype(np.float32), rng.normal(size=n).astype(np.float32)
        m, v, th = m0.copy(), v0.copy(), th0.copy()
        gb = orc.reduce_adam(cfg, n, comms, m, v, th, lr=1e-2, beta1=0.1, beta2=0.05, delta=1e-10, want_grad=True)
        assert np.array_equal(gb, orc.reduce(cfg, n, comms)), "the optional gradient output is Eq. 8 in the output type"
        wm, wv, wth = defn.adam_family_step(g, m0, v0, th0, lr=1e-2, beta1=0.1, beta2=0.05, delta=1e-10)
        assert np.allclose(m, wm, rtol=1e-5, atol=1e-9) and np.allclose(v, wv, rtol=1e-5, atol=1e-13)
        assert np.allclose(th, wth, rtol=1e-5, atol=1e-6)
        # the planted mistakes are far outside those tolerances
        bm, bv, bth = defn.adam_family_step(g, m0, v0, th0, lr=1e-2, beta1=0.9, beta2=0.05, delta=1e-10)
        assert not np.allclose(m, bm, rtol=1e-3, atol=1e-7)
        # part by part gives the same as all parts at once
        m2, v2, th2 = m0.copy(), v0.copy(), th0.copy()
        pos = 0
        for j in range(3):
            cnt = orc.partition_elems(cfg, n, j)
            orc.reduce_adam(cfg, n, comms, m2[pos:pos + cnt], v2[pos:pos + cnt], th2[pos:pos + cnt], lr=1e-2, beta1=0.1,
                            beta2=0.05, delta=1e-10, first=j, count=1)
            pos += cnt
        assert np.array_equal(m2, m) and np.array_equal(v2, v) and np.array_equal(th2, th)


def test_adam_family_zero_gradient_decays_the_moments():
    n = 256
    cfg = orc.OracleConfig(bits=4, s=2.0 ** 8, state_fmt=orc.STATE_NONE, grad_dtype=orc.F32, out_dtype=orc.F32)
    comms = [orc.new_comm(cfg, n), orc.new_comm(cfg, n)]          # all codes 0
    m, v, th = np.full(n, 0.5, np.float32), np.full(n, 4.0, np.float32), np.zeros(n, np.float32)
    orc.reduce_adam(cfg, n, comms, m, v, th, lr=1.0, beta1=0.5, beta2=0.75, delta=0.0)
    assert (m == 0.25).all() and (v == 1.0).all() and (th == -0.25).all()


# ---------------------------------------------------------------- element-wise clipping of the local gradient

@pytest.mark.parametrize("mode", [orc.SCALE_FIXED, orc.SCALE_BLOCK_ABSMAX])
def test_clipping_equals_clipping_the_input_first(mode):
    """send(clip = c, g) must be send(clip = 0, clamp(g, -c, c)) byte for byte over several iterations; a very large
    threshold changes nothing; +-Inf becomes +-c and raises no flag; NaN is still flagged."""
    rng = np.random.default_rng(8)
    n, c = 3000, 2e-3
    kw = dict(bits=4, scale_mode=mode, block_size=64, s=2.0 ** 10, s_e=2.0 ** 12, beta=0.5, reset_period=0,
              state_fmt=orc.STATE_INT8, grad_dtype=orc.F32, out_dtype=orc.F32, num_partitions=2)
    a, b, big = orc.OracleConfig(clip=c, **kw), orc.OracleConfig(**kw), orc.OracleConfig(clip=1e30, **kw)
    sa, sb, sg = (orc.new_state(a, n) for _ in range(3))
    ca, cb, cg = (orc.new_comm(a, n) for _ in range(3))
    changed = 0
    for k in range(1, 4):
        g = rng.normal(0, 2e-3, n).astype(np.float32)
        g[5], g[6] = np.inf, -np.inf
        gc = np.clip(g, -c, c).astype(np.float32)
        changed += int((gc != g).sum())
        fa = orc.send_step(a, g, sa, ca, k)
        fb = orc.send_step(b, gc, sb, cb, k)
        assert fa == fb and fa[0] == 0
        assert np.array_equal(ca, cb) and np.array_equal(sa, sb)
        g2 = g.copy()
        g2[5], g2[6] = 1.0, -1.0
        orc.send_step(big, g2, sg, cg, k)
    assert changed > 100
    sref, cref = orc.new_state(b, n), orc.new_comm(b, n)
    rng = np.random.default_rng(8)
    for k in range(1, 4):
        g = rng.normal(0, 2e-3, n).astype(np.float32)
        g[5], g[6] = 1.0, -1.0
        orc.send_step(b, g, sref, cref, k)
    assert np.array_equal(cg, cref) and np.array_equal(sg, sref), "a threshold nothing reaches must change nothing"
    g = rng.normal(0, 2e-3, n).astype(np.float32)
    g[7] = np.nan
    flags, _ = orc.send_step(a, g, sa, ca, 9)
    assert flags & orc.FLAG_NONFINITE


# ---------------------------------------------------------------- stochastic rounding on a Philox stream (extension)

def test_philox_known_answer_vectors():
    """The three known-answer vectors published with the generator (Random123 kat_vectors, philox4x32 10 rounds)."""
    kat = [((0, 0, 0, 0), (0, 0), (0x6627e8d5, 0xe169c58d, 0xbc57ac4c, 0x9b00dbd8)),
           ((0xffffffff,) * 4, (0xffffffff,) * 2, (0x408f276d, 0x41c83b0e, 0xa20bc7c6, 0x6d5451fd)),
           ((0x243f6a88, 0x85a308d3, 0x13198a2e, 0x03707344), (0xa4093822, 0x299f31d0), (0xd16cfe09, 0x94fdcceb, 0x5001e420, 0x24126ea1))]
    for ctr, key, want in kat:
        assert tuple(int(x) for x in orc.philox4x32_10(ctr, key)) == want


def test_stochastic_rounding_properties():
    """q is floor or ceil of h x s (inside the range), integers are never moved, the mean over many draws is h x s, the
    stream depends on (element, iteration, seed) only, and the added numbers are the 256 cell centres (b + 1/2) / 256,
    equally likely, one byte of a Philox block of 16 per element."""
    n, s = 1 << 14, 4.0
    kw = dict(bits=8, s=s, s_e=16.0, beta=0.5, reset_period=0, state_fmt=orc.STATE_NONE, grad_dtype=orc.F32, out_dtype=orc.F32)
    cfg = orc.OracleConfig(rounding=1, seed=12345, **kw)
    rng = np.random.default_rng(5)
    h = rng.uniform(-20, 20, n).astype(np.float32) / np.float32(s)
    h[:64] = np.arange(-32, 32, dtype=np.float32) / np.float32(s)            # exact integers after scaling
    y = (h * np.float32(s)).astype(np.float64)
    draws = []
    for k in range(1, 201):
        comm = orc.new_comm(cfg, n)
        orc.send_step(cfg, h, orc.new_state(cfg, n), comm, k)
        q = orc.unpack_codes(comm, n, 8)
        assert ((q == np.floor(y)) | (q == np.ceil(y))).all()
        assert (q[:64] == np.arange(-32, 32)).all()
        draws.append(q)
    mean = np.mean(draws, axis=0)
    frac = y - np.floor(y)
    # binomial standard error of 200 draws is at most 0.036; 5 sigma
    assert np.abs(mean - y).max() < 0.18 and abs(float(np.mean(mean - y))) < 2e-3
    # same (seed, element, iteration) -> same code; another seed or iteration -> another stream
    comm2 = orc.new_comm(cfg, n)
    orc.send_step(cfg, h, orc.new_state(cfg, n), comm2, 200)
    assert np.array_equal(orc.unpack_codes(comm2, n, 8), draws[-1])
    other = orc.OracleConfig(rounding=1, seed=12346, **kw)
    comm3 = orc.new_comm(other, n)
    orc.send_step(other, h, orc.new_state(other, n), comm3, 200)
    assert (orc.unpack_codes(comm3, n, 8) != draws[-1]).mean() > 0.2
    us = np.array([orc.sr_uniform(cfg, i, 7) for i in range(1 << 16)])
    assert us.min() > 0.0 and us.max() < 1.0 and abs(us.mean() - 0.5) < 0.005
    cells = us * 256 - 0.5
    assert np.array_equal(cells, np.round(cells))                       # cell centres only
    counts = np.bincount(cells.astype(np.int64), minlength=256)
    assert counts.min() > 176 and counts.max() < 336                    # 256 expected per cell, 5 sigma
    # element i takes byte (i mod 4) of word ((i mod 16) / 4) of the block's Philox output
    for i in (0, 5, 15, 16, 1000003):
        blk = i >> 4
        words = orc.philox4x32_10((blk & 0xffffffff, blk >> 32, 7, 0), (12345, 0))
        b = (int(words[(i >> 2) & 3]) >> (8 * (i & 3))) & 0xff
        assert orc.sr_uniform(cfg, i, 7) == (b + 0.5) / 256
    # the position inside a bucket matters, not the bucket's partitioning
    cfgp = orc.OracleConfig(rounding=1, seed=12345, num_partitions=4, **kw)
    commp = orc.new_comm(cfgp, n)
    orc.send_step(cfgp, h, orc.new_state(cfgp, n), commp, 200)
    qp = np.concatenate([orc.unpack_codes(c, orc.partition_elems(cfgp, n, j), 8) for j, (c, _) in enumerate(orc.comm_views(cfgp, n, commp))])
    assert np.array_equal(qp, draws[-1])


# ---------------------------------------------------------------- Eq. 7's clamp: saturated 8-bit error codes

def test_state_clamp_hand_worked_example():
    """tests/golden/eq7_clamp_worked_example.txt: error codes whose nearest integer leaves [-128, 127] are clamped
    (Eq. 7 compresses with the 8-bit compressor of Eq. 1) and counted; the ties 127.5 and -128.5 fall on either side."""
    G = load_golden("eq7_clamp_worked_example.txt")
    f = lambda k: np.array([float(v) for v in G[k]], dtype=np.float32)
    for fmt in (orc.STATE_INT8, orc.STATE_FP32_Q8COMP):
        cfg = OracleConfig(bits=int(G["p"][0]), s=float(G["s"][0]), s_e=float(G["s_e"][0]), beta=float(G["beta"][0]),
                           reset_period=0, state_fmt=fmt)
        state, comm = orc.new_state(cfg, 6), orc.new_comm(cfg, 6)
        (flags, sat, ssat), tr = orc.send_step(cfg, f("g1"), state, comm, 1, trace=True, full_status=True)
        assert flags == 0 and sat == int(G["sat1"][0])
        assert np.array_equal(tr["q"], f("q1").astype(np.int32)) and np.array_equal(tr["d"], f("d1"))
        assert np.array_equal(tr["e_new"], f("et2"))
        if fmt == orc.STATE_INT8:
            assert ssat == int(G["ssat1"][0])
            assert np.array_equal(state[:6].view(np.int8), f("e2").astype(np.int8))
        else:
            # the fp32 error is kept; its 8-bit image is formed (and its clamp counted) when it is next used
            assert ssat == 0
            (_, _, ssat2), tr2 = orc.send_step(cfg, np.zeros(6, np.float32), state, comm, 2, trace=True, full_status=True)
            assert ssat2 == int(G["ssat1"][0])
            assert np.array_equal(tr2["c"], f("e2") / np.float32(16))


# ---------------------------------------------------------------- block-scaled 8-bit error state (extension)

@pytest.mark.parametrize("B", [32, 256, 1024])
@pytest.mark.parametrize("p", [4, 8])
def test_block_scaled_int8_state(B, p):
    """The 8-bit error state with one scale per block (no counterpart in the paper; Eq. 7's 8-bit compression with the
    global s_e replaced by 127 / amax of the block).  What the mathematics fixes: the stored scale is fl(amax / 127),
    the largest code of a non-zero block is 127 in magnitude, |e~ - e x scale| <= scale / 2, a zero block and a
    reset give scale 0 and codes 0, the next iteration compensates with e x scale, and Lemma 1's identity holds in
    its 8-bit form d - g = (e^_k - e~_{k+1}) / beta with e^_k = e_k x scale_k."""
    n = 5 * B + B // 2 + 3                       # five whole blocks, one ragged
    beta = 0.5
    cfg = OracleConfig(bits=p, scale_mode=orc.SCALE_BLOCK_ABSMAX, block_size=B, beta=beta, reset_period=3,
                       state_fmt=orc.STATE_INT8)
    nblk = (n + B - 1) // B
    state, comm = orc.new_state(cfg, n), orc.new_comm(cfg, n)
    codes_v, scales_v = orc.state_views(cfg, n, state)
    prev_codes, prev_scales = codes_v.copy(), scales_v.copy()
    assert not prev_codes.any() and not prev_scales.any()
    for k in range(1, 7):                        # k = 3 and k = 6 reset
        g = RNG.normal(0, 1e-3, n).astype(np.float32)
        g[2 * B:3 * B] = 0                       # block 2 never carries anything
        (_, _), tr = orc.send_step(cfg, g, state, comm, k, trace=True)
        # step 1 compensated with the stored image of the previous error: one product per element
        want_c = prev_codes.astype(np.float32) * np.repeat(prev_scales, B)[:n]
        assert np.array_equal(tr["c"], want_c)
        assert np.array_equal(tr["h"], g + want_c)
        # Lemma 1, 8-bit form
        lhs = tr["d"].astype(np.float64) - g.astype(np.float64)
        rhs = (tr["c"].astype(np.float64) - tr["e_new"].astype(np.float64)) / beta
        assert np.allclose(lhs, rhs, rtol=0, atol=1e-9)
        if k % 3 == 0:
            assert not codes_v.any() and not scales_v.any()
        else:
            for b in range(nblk):
                blk = slice(b * B, min((b + 1) * B, n))
                en = tr["e_new"][blk]
                amax = np.abs(en).max()
                assert scales_v[b].view(np.uint32) == (np.float32(amax) / np.float32(127)).view(np.uint32)
                if amax == 0:
                    assert scales_v[b] == 0 and not codes_v[blk].any()
                    continue
                e = codes_v[blk].astype(np.float64)
                assert np.abs(e).max() == 127
                # en x fl(127 / amax) is rounded once before the nearest-integer step: a few ulps of slack
                assert np.all(np.abs(en.astype(np.float64) - e * float(scales_v[b])) <= float(scales_v[b]) * (0.5 + 1e-4))
            assert scales_v[2] == 0 and not codes_v[2 * B:3 * B].any()
        prev_codes, prev_scales = codes_v.copy(), scales_v.copy()


def test_block_scaled_int8_state_detects_a_wrong_divisor():
    """The pin above has teeth: codes formed with 128 / amax (a plausible slip) against the stored scale amax / 127
    break the half-step bound."""
    en = RNG.normal(0, 1e-3, 256).astype(np.float32)
    amax = np.abs(en).max()
    scale = float(np.float32(amax) / np.float32(127))
    wrong = np.rint(en * (np.float32(128) / amax)).clip(-128, 127).astype(np.float64)
    right = np.rint(en * (np.float32(127) / amax)).clip(-128, 127).astype(np.float64)
    assert np.all(np.abs(en - right * scale) <= scale * (0.5 + 1e-4))
    assert np.any(np.abs(en - wrong * scale) > scale * (0.5 + 1e-4))


# ---------------------------------------------------------------- bf16 conversions

def _torch_bf16_bits(x: np.ndarray) -> np.ndarray:
    return torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def test_bf16_conversions_against_an_independent_conversion():
    """bf16 is the upper half of binary32; conversion to it rounds to nearest, ties to even.  Checked against PyTorch's
    own conversion on ties, +-0, denormals, the largest finite values, +-Inf, NaN and a million random bit patterns."""
    special = np.array([0x00000000, 0x80000000, 0x00000001, 0x80000001, 0x00008000, 0x00018000, 0x00007fff, 0x0000ffff,
                        0x3f808000, 0x3f818000, 0x3f807fff, 0x3f808001, 0x3f817fff, 0x3f818001,      # ties and their neighbours
                        0x7f7fffff, 0xff7fffff, 0x7f7f7fff, 0x7f7f8000, 0x7f7f8001,                  # largest finite: rounds to Inf
                        0x7f800000, 0xff800000, 0x007fffff, 0x00800000, 0x807fffff], dtype=np.uint32)
    rnd = RNG.integers(0, 2 ** 32, 1_000_000, dtype=np.uint64).astype(np.uint32)
    words = np.concatenate([special, rnd])
    x = words.view(np.float32)
    got = orc.f32_to_bf16_bits(x)
    want = _torch_bf16_bits(x)
    nan = np.isnan(x)
    assert np.array_equal(got[~nan], want[~nan])
    # a NaN stays a NaN (its payload is not part of the contract)
    assert np.all((got[nan] & 0x7f80) == 0x7f80) and np.all((got[nan] & 0x007f) != 0)
    # ties-to-even spelled out: 1 + 2^-8 -> 1 (even), 1 + 3 * 2^-8 -> 1 + 2^-6
    assert list(orc.f32_to_bf16_bits(np.array([0x3f808000, 0x3f818000], np.uint32).view(np.float32))) == [0x3f80, 0x3f82]
    # widening is exact and inverts the narrowing on every bf16 value
    allb = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    wide = orc.bf16_bits_to_f32(allb)
    assert np.array_equal(wide.view(np.uint32), allb.astype(np.uint32) << 16)
    fin = ~np.isnan(wide)
    assert np.array_equal(orc.f32_to_bf16_bits(wide[fin]), allb[fin])
    assert np.array_equal(wide[fin], torch.from_numpy(allb[fin].view(np.int16)).view(torch.bfloat16).float().numpy())


def test_bf16_gradient_is_the_widened_value_and_bf16_output_is_the_rounded_mean():
    """A bf16 gradient enters Algorithm 1 as the fp32 number it denotes; a bf16 output is the fp32 result of Eq. 8
    rounded once (checked with PyTorch's conversion, not the oracle's)."""
    n = 4099
    kw = dict(bits=4, s=2.0 ** 11, s_e=2.0 ** 13, beta=0.5, reset_period=0, num_partitions=3)
    cb, cf = OracleConfig(grad_dtype=orc.BF16, **kw), OracleConfig(grad_dtype=orc.F32, **kw)
    sb, sf = orc.new_state(cb, n), orc.new_state(cf, n)
    comms_b, comms_f = [], []
    for k in range(1, 4):
        gb = _torch_bf16_bits(RNG.normal(0, 1e-3, n).astype(np.float32))
        gf = torch.from_numpy(gb.view(np.int16)).view(torch.bfloat16).float().numpy()
        mb, mf = orc.new_comm(cb, n), orc.new_comm(cf, n)
        assert orc.send_step(cb, gb, sb, mb, k) == orc.send_step(cf, gf, sf, mf, k)
        assert np.array_equal(mb, mf) and np.array_equal(sb, sf)
        comms_b.append(mb)
        comms_f.append(mf)
    o32 = orc.reduce(cf, n, comms_f)
    o16 = orc.reduce(OracleConfig(grad_dtype=orc.F32, out_dtype=orc.BF16, **kw), n, comms_f)
    assert np.array_equal(o16, _torch_bf16_bits(o32))


# ---------------------------------------------------------------- 1-bit LoCo (sign code; named in the paper, not defined)

def test_one_bit_code_is_the_sign():
    """Reading for bits = 1: q = -1 if h < 0 else +1 (so +-0 -> +1), wire bit 1 for -1, d = q / s, eight codes per
    byte with element i at bit i mod 8; Eq. 8 then averages +-1/s."""
    s = 8.0
    cfg = OracleConfig(bits=1, s=s, s_e=4 * s, beta=1.0, reset_period=0, state_fmt=orc.STATE_FP32)
    g = np.array([0.5, -0.5, 0.0, -0.0, 1e-30, -1e-30, 3.0, -7.0, 0.125, -0.125], dtype=np.float32)
    state, comm = orc.new_state(cfg, g.size), orc.new_comm(cfg, g.size, fill=0xEE)
    (flags, sat), tr = orc.send_step(cfg, g, state, comm, 1, trace=True)
    assert flags == 0 and sat == 0
    assert list(tr["q"]) == [1, -1, 1, 1, 1, -1, 1, -1, 1, -1]
    assert np.array_equal(tr["d"], tr["q"].astype(np.float32) / np.float32(s))
    assert comm[0] == 0b10100010 and comm[1] == 0b00000010        # bits 1, 5, 7 and bit 9
    # beta = 1: classic error feedback, e~ = h - sign(h) / s
    assert np.array_equal(state.view(np.float32)[:g.size], g - tr["d"])
    # idempotent: the dequantised vector compresses to the same codes
    comm2 = orc.new_comm(cfg, g.size)
    (_, _), tr2 = orc.send_step(cfg, tr["d"], orc.new_state(cfg, g.size), comm2, 1, trace=True)
    assert np.array_equal(tr2["q"], tr["q"]) and np.array_equal(tr2["d"], tr["d"])
    # Eq. 8 over 3 workers holding q, q and -q: (q + q - q) / (3 s)
    gneg = np.where(tr["q"] > 0, -1.0, 1.0).astype(np.float32)
    comm3 = orc.new_comm(cfg, g.size)
    orc.send_step(cfg, gneg, orc.new_state(cfg, g.size), comm3, 1)
    got = orc.reduce(cfg, g.size, [comm, comm, comm3])
    want = ((tr["d"] + tr["d"]) - tr["d"]) / np.float32(3)
    assert np.array_equal(got, want)


def test_one_bit_packing_all_byte_values():
    """Brute force over all 256 bytes: bit i of a byte is element i, 1 meaning -1."""
    for b in range(256):
        q = orc.unpack_codes(np.array([b], np.uint8), 8, 1)
        assert list(q) == [(-1 if (b >> i) & 1 else 1) for i in range(8)]
        assert orc.pack_codes(q, 1)[0] == b


def test_one_bit_block_scale_is_the_pairwise_mean_of_magnitudes():
    """With block scales the magnitude sent for a block is the mean of |h| -- the value that minimises the squared
    error sum (h - q mu)^2 of a sign code -- formed by pairwise summation in fp32 over the block's positions."""
    B = 32
    cfg = OracleConfig(bits=1, scale_mode=orc.SCALE_BLOCK_ABSMAX, block_size=B, beta=0.5, reset_period=0,
                       state_fmt=orc.STATE_FP32)
    # (a) the order of the sum, on values where it shows: sequential summation would lose the three 2^-24
    g = np.zeros(2 * B + 5, dtype=np.float32)
    g[0], g[1], g[2], g[3] = 1.0, -(2.0 ** -24), 2.0 ** -24, -(2.0 ** -24)
    g[B:2 * B] = np.arange(1, B + 1, dtype=np.float32) * np.where(np.arange(B) % 2, -1, 1)   # 1, -2, 3, ...: exact sum 528
    g[2 * B:] = [4.0, -1.0, 0.5, -0.25, 0.25]                                                # ragged block: 6 / 5
    state, comm = orc.new_state(cfg, g.size), orc.new_comm(cfg, g.size)
    (_, _), tr = orc.send_step(cfg, g, state, comm, 1, trace=True)
    _, scales = orc.comm_views(cfg, g.size, comm)[0]
    # (1 + 2^-24) rounds to 1 (tie to even); (2^-24 + 2^-24) = 2^-23; 1 + 2^-23 is representable; / 32 is exact
    assert scales[0] == np.float32((1.0 + 2.0 ** -23) / 32)
    assert scales[1] == np.float32(528.0 / 32) and scales[2] == np.float32(6.0) / np.float32(5.0)
    assert np.array_equal(tr["d"], np.where(g < 0, -1, 1).astype(np.float32) * np.repeat(scales, B)[:g.size])
    # (b) optimality, brute force on a tiny block: no magnitude on a fine grid beats the one sent
    h = RNG.normal(0, 1e-3, B).astype(np.float32)
    comm = orc.new_comm(cfg, B)
    orc.send_step(cfg, h, orc.new_state(cfg, B), comm, 1)
    mu = float(orc.comm_views(cfg, B, comm)[0][1][0])
    a = np.abs(h.astype(np.float64))
    loss = lambda m: float(((a - m) ** 2).sum())
    grid = np.linspace(0.0, 2 * a.max(), 4001)
    assert all(loss(mu) <= loss(m) + 1e-18 for m in grid)
    assert abs(mu - a.mean()) <= 6 * 2.0 ** -24 * a.mean()         # log2(32) + 1 roundings
    # (c) pairwise summation is exact whenever no partial sum needs rounding, and within log2(B) ulps otherwise
    d = dyadic(1024, 10, 2.0 ** -20)
    assert orc.pairwise_sum(np.abs(d)) == float(np.abs(d.astype(np.float64)).sum())
    r = np.abs(RNG.normal(0, 1, 4096)).astype(np.float32)
    assert abs(orc.pairwise_sum(r) - float(r.astype(np.float64).sum())) <= 12 * 2.0 ** -24 * float(r.sum())


@pytest.mark.parametrize("mode,fmt", [(orc.SCALE_FIXED, orc.STATE_FP32), (orc.SCALE_FIXED, orc.STATE_INT8),
                                      (orc.SCALE_BLOCK_ABSMAX, orc.STATE_FP32), (orc.SCALE_BLOCK_ABSMAX, orc.STATE_INT8)])
def test_one_bit_keeps_lemma_1_identity(mode, fmt):
    """Lemma 1's identity d - g = (e^_k - e~_{k+1}) / beta does not depend on the compressor: it holds for the sign code."""
    n, beta = 777, 0.25
    cfg = OracleConfig(bits=1, scale_mode=mode, block_size=64, s=2.0 ** 9, s_e=2.0 ** 13, beta=beta, reset_period=0,
                       state_fmt=fmt)
    state, comm = orc.new_state(cfg, n), orc.new_comm(cfg, n)
    for k in range(1, 5):
        g = RNG.normal(0, 1e-3, n).astype(np.float32)
        (_, _), tr = orc.send_step(cfg, g, state, comm, k, trace=True)
        assert set(np.unique(tr["q"])) <= {-1, 1}
        lhs = tr["d"].astype(np.float64) - g.astype(np.float64)
        rhs = (tr["c"].astype(np.float64) - tr["e_new"].astype(np.float64)) / beta
        assert np.allclose(lhs, rhs, rtol=0, atol=1e-9)
    with pytest.raises(ValueError):
        orc.send_step(dataclasses.replace(cfg, rounding=1), g, state, comm, 1)     # a sign code has nothing to round


def test_one_bit_non_finite_inputs():
    cfg = OracleConfig(bits=1, s=2.0 ** 10, s_e=2.0 ** 12, beta=0.5, reset_period=0, state_fmt=orc.STATE_FP32)
    g = np.array([np.nan, np.inf, -np.inf, 1e-3], dtype=np.float32)
    state, comm = orc.new_state(cfg, 4), orc.new_comm(cfg, 4)
    (flags, sat), tr = orc.send_step(cfg, g, state, comm, 1, trace=True)
    assert flags & orc.FLAG_NONFINITE and sat == 0
    assert list(tr["q"]) == [1, 1, -1, 1]
    e = state.view(np.float32)[:4]
    assert e[0] == 0 and e[1] == 0 and e[2] == 0 and np.isfinite(e).all()
