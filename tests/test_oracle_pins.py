"""Pins for the float64 CPU oracle: every check here compares the oracle with something that is
NOT the oracle -- a closed form, an identity the equations imply, a brute-force sum, a library
routine, a hand-worked rational example, or a finite difference.  CPU only.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
LN = math.log


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 -> bf16 with torch and return the bit patterns (uint16)."""
    t = torch.from_numpy(np.asarray(x, np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def offsets(sizes):
    return np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)


# --------------------------------------------------------------------------------------------
# step 1: log-sum-exp and the sampled token's log-probability
# --------------------------------------------------------------------------------------------

@pytest.mark.parametrize("V", [1, 2, 7, 4096])
@pytest.mark.parametrize("const", [0.0, -3.5, 11.0])
def test_lse_closed_form_equal_logits(oracle, V, const):
    """All logits equal to c: lse = c + ln V, log pi = -ln V for every token."""
    z = np.full((3, V), const, np.float32)
    y = np.array([0, V - 1, V // 2], np.int32)
    o = oracle.token_logp(z, V, y)
    np.testing.assert_allclose(o["lse"], const + LN(V), rtol=0, atol=1e-13 * max(1, abs(const) + LN(V)))
    np.testing.assert_allclose(o["token_logp"], -LN(V), rtol=0, atol=2e-14 * max(1.0, LN(V)))


def test_lse_two_logit_closed_form(oracle):
    """V = 2: log pi(0) = -log(1 + e^{b-a}) (the logistic function)."""
    a, b = 1.25, -0.5
    z = np.array([[a, b], [a, b]], np.float32)
    o = oracle.token_logp(z, 2, np.array([0, 1], np.int32))
    assert o["token_logp"][0] == pytest.approx(-math.log1p(math.exp(b - a)), abs=1e-15)
    assert o["token_logp"][1] == pytest.approx(-math.log1p(math.exp(a - b)), abs=1e-15)


@pytest.mark.parametrize("as_bf16", [False, True])
def test_lse_with_minus_infinity_logits_closed_form(oracle, as_bf16):
    """A masked part of the vocabulary (-inf logits): with k finite logits all equal to c and the rest -inf,
    lse = c + ln k, log pi = -ln k on the finite ones, and the gradient is exactly 0 on the masked ones
    and g (1/k - 1[v = y]) elsewhere."""
    V, k, c = 64, 5, 1.5
    z = np.full((3, V), -np.inf, np.float32)
    cols = [[0, 1, 2, 3, 4], [59, 60, 61, 62, 63], [7, 20, 33, 46, 63]]
    for r in range(3):
        z[r, cols[r]] = c
    y = np.array([2, 63, 33], np.int32)
    bits = torch.from_numpy(z).to(torch.bfloat16).view(torch.int16).numpy().view("uint16") if as_bf16 else z
    o = oracle.token_logp(bits, V, y)
    np.testing.assert_allclose(o["lse"], c + LN(k), rtol=0, atol=1e-15)
    np.testing.assert_allclose(o["token_logp"], -LN(k), rtol=0, atol=1e-15)
    g = np.array([0.25, -0.5, 2.0])
    dz = oracle.dlogits_rows(bits, V, 1, y, o["row_ok"], o["lse"], g, np.arange(3, dtype=np.int64))
    for r in range(3):
        ref = np.zeros(V)
        ref[cols[r]] = g[r] / k
        ref[y[r]] -= g[r]
        np.testing.assert_allclose(dz[r], ref, rtol=0, atol=1e-15)
        assert np.all(dz[r][np.isinf(z[r])] == 0.0)


def test_lse_brute_force_fsum(oracle):
    """Naive log(sum(exp z)) with an exactly rounded sum (math.fsum) on tiny rows."""
    rng = np.random.default_rng(5)
    z = rng.normal(0, 3, (16, 37)).astype(np.float32)
    y = rng.integers(0, 37, 16).astype(np.int32)
    o = oracle.token_logp(z, 37, y)
    for r in range(16):
        ref = math.log(math.fsum(math.exp(float(v)) for v in z[r]))
        assert o["lse"][r] == pytest.approx(ref, abs=1e-13)
        assert o["token_logp"][r] == pytest.approx(float(z[r, y[r]]) - ref, abs=1e-13)


def test_lse_matches_library_logsumexp(oracle):
    rng = np.random.default_rng(6)
    z = rng.normal(0, 2, (64, 4096)).astype(np.float32)
    y = rng.integers(0, 4096, 64).astype(np.int32)
    o = oracle.token_logp(z, 4096, y)
    ref = torch.logsumexp(torch.from_numpy(z).double(), dim=1).numpy()
    np.testing.assert_allclose(o["lse"], ref, rtol=0, atol=1e-12)
    lp = torch.log_softmax(torch.from_numpy(z).double(), dim=1).numpy()[np.arange(64), y]
    np.testing.assert_allclose(o["token_logp"], lp, rtol=0, atol=1e-12)


def test_lse_shift_invariance_and_large_values(oracle):
    """log pi is unchanged by adding a constant to a row, also where naive exp would overflow."""
    rng = np.random.default_rng(7)
    base = (rng.integers(-64, 64, (4, 50)) / 8.0).astype(np.float32)  # exactly representable
    y = rng.integers(0, 50, 4).astype(np.int32)
    a = oracle.token_logp(base, 50, y)
    for shift in (1024.0, -2048.0, 700.0):
        b = oracle.token_logp(base + np.float32(shift), 50, y)
        np.testing.assert_allclose(b["token_logp"], a["token_logp"], rtol=0, atol=1e-12)
        np.testing.assert_allclose(b["lse"], a["lse"] + shift, rtol=0, atol=1e-9)


def test_bf16_bits_are_decoded_exactly(oracle):
    """0x3F80 = 1.0, 0xC000 = -2.0, 0x4049 = 3.140625: lse over those three values."""
    bits = np.array([[0x3F80, 0xC000, 0x4049]], np.uint16)
    o = oracle.token_logp(bits, 3, np.array([2], np.int32))
    ref = math.log(math.exp(1.0) + math.exp(-2.0) + math.exp(3.140625))
    assert o["lse"][0] == pytest.approx(ref, abs=1e-14)
    assert o["token_logp"][0] == pytest.approx(3.140625 - ref, abs=1e-14)


def test_row_stride_and_column_limit(oracle):
    """Only the first `vocab` entries of a row count; the row stride may be larger."""
    rng = np.random.default_rng(8)
    z = rng.normal(0, 1, (5, 24)).astype(np.float32)
    z[:, 16:] = 50.0  # padding columns that must be ignored
    y = rng.integers(0, 16, 5).astype(np.int32)
    o = oracle.token_logp(z, 16, y)
    ref = torch.logsumexp(torch.from_numpy(z[:, :16].copy()).double(), 1).numpy()
    np.testing.assert_allclose(o["lse"], ref, atol=1e-13)


def test_masked_and_bad_token_rows(oracle):
    z = np.zeros((6, 8), np.float32)
    y = np.array([0, 1, 8, -1, 3, 7], np.int32)
    m = np.array([1, 0, 1, 1, 1, 0], np.uint8)
    o = oracle.token_logp(z, 8, y, m)
    assert o["row_ok"].tolist() == [1, 0, 0, 0, 1, 0]
    assert o["n_bad_token"] == 2
    assert o["token_logp"][1] == 0.0 and o["token_logp"][2] == 0.0
    assert o["token_logp"][0] == pytest.approx(-LN(8))


def test_seq_reduce_by_hand(oracle):
    """s_n and S_n are sums over unmasked tokens only (generation-level accumulation)."""
    lp = np.array([-1.0, -2.0, -4.0, -0.5, -0.25, -8.0])
    mu = np.array([-1.5, -2.0, -1.0, -0.5, -1.25, -3.0], np.float32)
    ok = np.array([1, 1, 0, 0, 1, 1], np.uint8)
    s, S, cnt = oracle.seq_reduce(2, 3, lp, mu, ok)
    assert s.tolist() == [0.5, 1.0 - 5.0]
    assert S.tolist() == [-3.0, -8.25]
    assert cnt.tolist() == [2, 2]


# --------------------------------------------------------------------------------------------
# steps 3-4: group advantage (Eq. 2, Eq. 4, Eq. 5, leave-one-out)
# --------------------------------------------------------------------------------------------

def _frac_list(s):
    return [Fraction(x) for x in s.split()]


def _golden_adv_cases():
    cases = []
    with open(os.path.join(GOLDEN, "group_advantage_cases.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            parts = [p.strip() for p in line.split("|")]
            cases.append(parts)
    assert len(cases) >= 7
    return cases


@pytest.mark.parametrize("case", _golden_adv_cases(), ids=lambda c: c[0])
def test_group_advantage_hand_worked(oracle, case):
    name, eq, sizes, R, w, eta, mode, c_exp, a_exp = case
    sizes = [int(x) for x in sizes.split()]
    R = np.array([float(x) for x in _frac_list(R)], np.float32)
    eta = math.inf if eta == "inf" else float(eta)
    flags = oracle.FLAG_LEAVE_ONE_OUT if mode == "loo" else 0
    c_exp = np.array([float(x) for x in _frac_list(c_exp)])
    a_exp = np.array([float(x) for x in _frac_list(a_exp)])
    go = offsets(sizes)
    if w == "-":
        o = oracle.group_advantage(R, None, go, eta, flags)
        np.testing.assert_array_equal(o["clipped_w"], c_exp)
        np.testing.assert_allclose(o["adv64"], a_exp, rtol=0, atol=1e-15)
        return
    wv = np.array([float(x) for x in _frac_list(w)])
    # (a) weights handed over directly
    o = oracle.group_advantage(R, wv, go, eta, flags | oracle.FLAG_ADV_INPUT_IS_WEIGHT)
    np.testing.assert_array_equal(o["clipped_w"], c_exp)
    np.testing.assert_allclose(o["adv64"], a_exp, rtol=0, atol=4e-16 * max(1, np.abs(a_exp).max()))
    np.testing.assert_array_equal(o["adv32"], a_exp.astype(np.float32))
    # (b) as log-ratios s_n = log w_n (the form the loss uses)
    o = oracle.group_advantage(R, np.log(wv), go, eta, flags)
    np.testing.assert_allclose(o["adv64"], a_exp, rtol=0, atol=1e-14)
    # the rejected reading of Eq. 5 (max instead of min) must NOT reproduce these numbers
    if eq == "Eq.5" and name != "tie_at_cap":
        c_max = np.maximum(wv, eta)
        assert not np.allclose(c_max, c_exp)


def test_eq2_sums_to_zero_and_is_exact_for_binary_rewards(oracle):
    rng = np.random.default_rng(11)
    sizes = [8, 8, 1, 5, 16, 3]
    N = sum(sizes)
    R = (rng.random(N) < 0.4).astype(np.float32)
    o = oracle.group_advantage(R, None, offsets(sizes), 2.0)
    go = offsets(sizes)
    for k, nk in enumerate(sizes):
        seg = slice(go[k], go[k + 1])
        ones = int(R[seg].sum())
        # exact rational: R - ones/nk
        ref = np.array([float(Fraction(int(r)) - Fraction(ones, nk)) for r in R[seg]])
        np.testing.assert_allclose(o["adv64"][seg], ref, rtol=0, atol=1e-16)
        assert abs(o["adv64"][seg].sum()) < 1e-14
    assert o["adv64"][16] == 0.0  # a group of one has zero advantage on-policy


def test_eq5_identities(oracle):
    rng = np.random.default_rng(12)
    sizes = [8, 4, 6, 2]
    go = offsets(sizes)
    N = sum(sizes)
    R = rng.normal(0, 1, N).astype(np.float32)
    s = rng.normal(0, 1.0, N)
    eta = 2.0
    o = oracle.group_advantage(R, s, go, eta)
    w = np.exp(s)
    np.testing.assert_allclose(o["weight"], w, rtol=1e-15)
    np.testing.assert_array_equal(o["clipped_w"], np.minimum(w, eta))
    assert (w > eta).any() and (w < eta).any()
    c = np.minimum(w, eta)
    for k in range(len(sizes)):
        seg = slice(go[k], go[k + 1])
        # sum over the group of A_n = sum (1 - c_n) R_n
        assert o["adv64"][seg].sum() == pytest.approx(((1 - c[seg]) * R[seg]).sum(), abs=1e-13)
    # eta -> inf reproduces the unclipped estimate (Eq. 4)
    o_inf = oracle.group_advantage(R, s, go, math.inf)
    for k in range(len(sizes)):
        seg = slice(go[k], go[k + 1])
        ref = R[seg].astype(np.float64) - (w[seg] * R[seg]).sum() / sizes[k]
        np.testing.assert_allclose(o_inf["adv64"][seg], ref, atol=1e-13)
    # eta below every weight: A_n = R_n - eta * mean(R)
    lo = float(w.min()) * 0.5
    o_lo = oracle.group_advantage(R, s, go, lo)
    for k in range(len(sizes)):
        seg = slice(go[k], go[k + 1])
        ref = R[seg].astype(np.float64) - lo * R[seg].astype(np.float64).mean()
        np.testing.assert_allclose(o_lo["adv64"][seg], ref, atol=1e-13)
    # linear in the rewards (rewards chosen exactly representable so that R1 + 2 R2 is exact)
    R1 = (rng.integers(-8, 8, N) / 4).astype(np.float32)
    R2 = (rng.integers(-8, 8, N) / 4).astype(np.float32)
    a1 = oracle.group_advantage(R1, s, go, eta)["adv64"]
    a2 = oracle.group_advantage(R2, s, go, eta)["adv64"]
    a12 = oracle.group_advantage(R1 + 2 * R2, s, go, eta)["adv64"]
    np.testing.assert_allclose(a12, a1 + 2 * a2, atol=1e-13)
    # on-policy weights reduce Eq. 5 to Eq. 2
    a_on = oracle.group_advantage(R, np.zeros(N), go, eta)["adv64"]
    a_eq2 = oracle.group_advantage(R, None, go, eta)["adv64"]
    np.testing.assert_array_equal(a_on, a_eq2)


def test_leave_one_out_relations(oracle):
    rng = np.random.default_rng(13)
    sizes = [8, 3, 1]
    go = offsets(sizes)
    N = sum(sizes)
    R = rng.normal(0, 1, N).astype(np.float32)
    s = rng.normal(0, 0.7, N)
    eta = 2.0
    c = np.minimum(np.exp(s), eta)
    loo = oracle.group_advantage(R, s, go, eta, oracle.FLAG_LEAVE_ONE_OUT)["adv64"]
    lit = oracle.group_advantage(R, s, go, eta, oracle.FLAG_LEAVE_ONE_OUT
                                 | oracle.FLAG_LOO_LITERAL_DIVISOR)["adv64"]
    for k, nk in enumerate(sizes):
        for n in range(go[k], go[k + 1]):
            tot = (c[go[k]:go[k + 1]] * R[go[k]:go[k + 1]]).sum() - c[n] * R[n]
            assert lit[n] == pytest.approx(R[n] - tot / nk, abs=1e-13)
            if nk > 1:
                assert loo[n] == pytest.approx(R[n] - tot / (nk - 1), abs=1e-13)
            else:
                assert loo[n] == R[n]
    # on-policy: leave-one-out advantage = N_k/(N_k-1) times the Eq. 2 advantage
    on = oracle.group_advantage(R, None, go, eta)["adv64"]
    on_loo = oracle.group_advantage(R, None, go, eta, oracle.FLAG_LEAVE_ONE_OUT)["adv64"]
    np.testing.assert_allclose(on_loo[:8], on[:8] * 8 / 7, atol=1e-13)
    np.testing.assert_allclose(on_loo[8:11], on[8:11] * 3 / 2, atol=1e-13)


def test_bad_group_offsets_are_rejected(oracle):
    R = np.zeros(4, np.float32)
    for go in ([1, 4], [0, 3], [0, 3, 2, 4]):
        with pytest.raises(ValueError):
            oracle.group_advantage(R, None, np.array(go, np.int32), 2.0)
    o = oracle.group_advantage(np.ones(4, np.float32), None, np.array([0, 2, 2, 4], np.int32), 2.0)
    np.testing.assert_array_equal(o["adv64"], np.zeros(4))  # an empty group is skipped


# --------------------------------------------------------------------------------------------
# the whole path (steps 1-6)
# --------------------------------------------------------------------------------------------

def _read_kv(path):
    kv = {}
    with open(path) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#") and "=" in line:
                k, v = line.split("=", 1)
                kv[k.strip()] = np.array([float(Fraction(x)) for x in v.split()])
    return kv


@pytest.mark.parametrize("literal", [False, True])
def test_two_token_case_worked_by_hand(oracle, literal):
    kv = _read_kv(os.path.join(GOLDEN, "pg_loss_two_token_case.txt"))
    z = np.array([[LN(3), 0.0], [LN(3), 0.0]], np.float32)
    y = np.array([0, 1], np.int32)
    mu = np.array([LN(0.25), LN(0.5)], np.float32)
    R = np.array([0, 1], np.float32)
    flags = oracle.FLAG_OUTER_UNCLIPPED if literal else 0
    o = oracle.pg_loss(z, 2, 1, 2, y, None, mu, R, np.array([0, 2], np.int32), 2.0, flags,
                       want_dlogits=True)
    tol = 3e-7  # float32 rounding of ln 3, ln(1/4), ln(1/2) in the inputs
    np.testing.assert_allclose(np.exp(o["token_logp"]), [0.75, 0.25], atol=tol)
    np.testing.assert_allclose(o["weight"], kv["weights"], atol=tol)
    np.testing.assert_allclose(o["clipped_w"], kv["clipped"], atol=tol)
    np.testing.assert_allclose(o["adv64"], kv["adv"], atol=tol)
    key = "literal" if literal else "default"
    np.testing.assert_allclose(o["coef"], kv["coef_" + key], atol=tol)
    np.testing.assert_allclose(o["dlogits"].ravel(), kv["dlogits_" + key], atol=tol)
    g = kv["coef_" + key]
    loss = -(g[0] * LN(0.75) + g[1] * LN(0.25))
    assert o["loss"] == pytest.approx(loss, abs=tol)
    assert o["n_clipped"] == 1


def _small_problem(seed=0, N=6, L=5, V=11, sizes=(4, 2), sigma=0.4, dtype="f32", masked=True):
    rng = np.random.default_rng(seed)
    T = N * L
    z = (rng.integers(-40, 40, (T, V)) / 8.0).astype(np.float32)  # multiples of 1/8: exact in bf16 too
    y = rng.integers(0, V, T).astype(np.int32)
    m = np.ones(T, np.uint8)
    if masked:
        m[rng.random(T) < 0.25] = 0
        m[L:2 * L] = 0  # one generation with no token at all
    R = rng.normal(0, 1, N).astype(np.float32)
    logits = bf16_bits(z) if dtype == "bf16" else z
    return dict(z=z, logits=logits, y=y, m=m, R=R, go=offsets(sizes), N=N, L=L, V=V,
                rng=rng, sigma=sigma)


def _independent_pipeline(z64, y, m, mu, R, go, eta, outer_unclipped=False, norm_tokens=False):
    """A second implementation, written differently on purpose: vectorised numpy/torch library
    calls (log_softmax, reduceat) instead of the oracle's loops."""
    T, V = z64.shape
    N = R.shape[0]
    L = T // N
    logp_all = torch.log_softmax(torch.from_numpy(z64), dim=1).numpy()
    lp = logp_all[np.arange(T), y] * m
    s = ((lp - mu.astype(np.float64)) * m).reshape(N, L).sum(1)
    S = lp.reshape(N, L).sum(1)
    w = np.exp(s)
    c = np.minimum(w, eta)
    sizes = np.diff(go)
    b = np.add.reduceat(c * R, go[:-1]) / sizes
    A = R - np.repeat(b, sizes)
    Z = m.sum() if norm_tokens else N
    g = (w if outer_unclipped else c) * A / Z
    loss = -(g * S).sum()
    onehot = np.zeros((T, V))
    onehot[np.arange(T), y] = 1
    dz = np.repeat(g, L)[:, None] * m[:, None] * (np.exp(logp_all) - onehot)
    return dict(loss=loss, dz=dz, A=A, g=g, s=s, S=S, w=w, c=c, lp=lp)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("flags", [0, 1, 2, 3])
def test_whole_path_against_independent_numpy(oracle, dtype, flags):
    p = _small_problem(seed=21, dtype=dtype)
    z64 = p["z"].astype(np.float64)  # multiples of 1/8 are exact in bf16, so both dtypes see the same values
    mu = (np.zeros(p["N"] * p["L"]) + p["rng"].normal(-2.0, 0.6, p["N"] * p["L"])).astype(np.float32)
    o = oracle.pg_loss(p["logits"], p["N"], p["L"], p["V"], p["y"], p["m"], mu, p["R"], p["go"],
                       2.0, flags, want_dlogits=True)
    ref = _independent_pipeline(z64, p["y"], p["m"].astype(np.float64), mu, p["R"].astype(np.float64),
                                p["go"], 2.0, outer_unclipped=bool(flags & 1), norm_tokens=bool(flags & 2))
    np.testing.assert_allclose(o["token_logp"], ref["lp"], atol=1e-13)
    np.testing.assert_allclose(o["seq_log_ratio"], ref["s"], atol=1e-12)
    np.testing.assert_allclose(o["seq_logp"], ref["S"], atol=1e-12)
    np.testing.assert_allclose(o["weight"], ref["w"], rtol=1e-12)
    np.testing.assert_allclose(o["adv64"], ref["A"], atol=1e-12)
    np.testing.assert_allclose(o["coef"], ref["g"], atol=1e-12, rtol=1e-12)
    assert o["loss"] == pytest.approx(ref["loss"], rel=1e-12, abs=1e-12)
    np.testing.assert_allclose(o["dlogits"], ref["dz"], atol=1e-12, rtol=1e-11)
    assert o["n_tokens"] == int(p["m"].sum())
    assert (ref["w"] > 2.0).any(), "the case should exercise clipping"


def test_on_policy_reduces_to_eq1_eq2(oracle):
    """With log mu = log pi_theta every weight is 1 and the estimator is Eq. 1 with Eq. 2 advantages,
    coded here directly: loss = -(1/N) sum_n A_n sum_t log pi, A_n = R_n - mean_group(R)."""
    p = _small_problem(seed=22, masked=True)
    N, L, V = p["N"], p["L"], p["V"]
    lp = oracle.token_logp(p["logits"], V, p["y"], p["m"])["token_logp"]
    # float32 storage of log mu: make log pi representable by construction instead: feed float32(lp)
    mu = lp.astype(np.float32)
    o = oracle.pg_loss(p["logits"], N, L, V, p["y"], p["m"], mu, p["R"], p["go"], 2.0, 0,
                       want_dlogits=True)
    np.testing.assert_allclose(o["weight"], 1.0, atol=1e-5)  # float32 rounding of mu only
    # exact on-policy: rebuild with weights forced to one through the Eq. 2 path
    A = oracle.group_advantage(p["R"], None, p["go"], 2.0)["adv64"]
    S = (lp * p["m"]).reshape(N, L).sum(1)
    loss_eq1 = -(A * S).sum() / N
    assert o["loss"] == pytest.approx(loss_eq1, rel=2e-5)
    sm = torch.softmax(torch.from_numpy(p["z"].astype(np.float64)), 1).numpy()
    onehot = np.eye(V)[p["y"]]
    dz = (np.repeat(A, L) / N)[:, None] * p["m"][:, None] * (sm - onehot)
    np.testing.assert_allclose(o["dlogits"], dz, atol=2e-6)
    assert o["n_clipped"] == 0
    assert abs(o["mean_log_cw"]) < 1e-5


def test_dlogits_row_sums_and_exact_zeros(oracle):
    p = _small_problem(seed=23)
    N, L, V = p["N"], p["L"], p["V"]
    mu = p["rng"].normal(-2.4, 0.3, N * L).astype(np.float32)
    R = p["R"].copy()
    R[4:6] = 0.0  # group 2 all-zero rewards: advantage and gradient exactly zero (no std division)
    o = oracle.pg_loss(p["logits"], N, L, V, p["y"], p["m"], mu, R, p["go"], 2.0, 0, want_dlogits=True)
    np.testing.assert_allclose(o["dlogits"].sum(1), 0.0, atol=1e-15)
    assert np.all(o["dlogits"][p["m"] == 0] == 0.0)
    assert np.all(o["adv64"][4:6] == 0.0)
    assert np.all(o["dlogits"][4 * L:] == 0.0)
    assert o["seq_tokens"][1] == 0 and o["weight"][1] == 1.0  # empty generation: w = 1
    # all-one rewards off-policy: A_n = 1 - mean(c), generally non-zero
    R2 = R.copy()
    R2[4:6] = 1.0
    o2 = oracle.pg_loss(p["logits"], N, L, V, p["y"], p["m"], mu, R2, p["go"], 2.0, 0)
    np.testing.assert_allclose(o2["adv64"][4:6], 1.0 - o2["clipped_w"][4:6].mean(), atol=1e-14)


def _fd_problem():
    rng = np.random.default_rng(31)
    N, L, V = 4, 3, 5
    T = N * L
    z = (rng.integers(-16, 16, (T, V)) / 4.0).astype(np.float32)
    y = rng.integers(0, V, T).astype(np.int32)
    m = np.ones(T, np.uint8)
    m[5] = 0
    R = rng.normal(0, 1, N).astype(np.float32)
    mu = rng.normal(-1.6, 0.2, T).astype(np.float32)
    return N, L, V, T, z, y, m, R, mu, np.array([0, 2, 4], np.int32)


def test_finite_difference_frozen_coefficient(oracle):
    """(i) d/dz of -sum_n g_n S_n(z) with g frozen at the base point (Algorithm 1: the advantage is
    computed first, then the gradient of Eq. 3)."""
    N, L, V, T, z, y, m, R, mu, go = _fd_problem()
    base = oracle.pg_loss(z, N, L, V, y, m, mu, R, go, 2.0, 0, want_dlogits=True)
    g = base["coef"]
    h = 2.0 ** -9

    def surrogate(zz):
        o = oracle.token_logp(zz, V, y, m)
        S = (o["token_logp"] * m).reshape(N, L).sum(1)
        return -(g * S).sum()

    fd = np.zeros((T, V))
    for r in range(T):
        for v in range(V):
            zp, zm = z.copy(), z.copy()
            zp[r, v] += h
            zm[r, v] -= h
            fd[r, v] = (surrogate(zp) - surrogate(zm)) / (2 * h)
    np.testing.assert_allclose(base["dlogits"], fd, atol=2e-6)


def test_finite_difference_of_importance_weighted_objective(oracle):
    """(ii) Eq. 3 itself: with the outer weight as printed and no clipping, the ascent direction is
    the derivative of (1/N) sum_n A_n pi_theta(y_n)/mu(y_n) with only A frozen, because
    grad pi / mu = w grad log pi."""
    N, L, V, T, z, y, m, R, mu, go = _fd_problem()
    flags = oracle.FLAG_OUTER_UNCLIPPED
    base = oracle.pg_loss(z, N, L, V, y, m, mu, R, go, math.inf, flags, want_dlogits=True)
    A = base["adv64"]
    h = 2.0 ** -9

    def neg_objective(zz):
        o = oracle.token_logp(zz, V, y, m)
        s, _, _ = oracle.seq_reduce(N, L, o["token_logp"], mu, o["row_ok"])
        return -(A * np.exp(s)).sum() / N

    fd = np.zeros((T, V))
    for r in range(T):
        for v in range(V):
            zp, zm = z.copy(), z.copy()
            zp[r, v] += h
            zm[r, v] -= h
            fd[r, v] = (neg_objective(zp) - neg_objective(zm)) / (2 * h)
    np.testing.assert_allclose(base["dlogits"], fd, atol=5e-6)


def test_clip_statistics(oracle):
    p = _small_problem(seed=24, masked=False)
    N, L, V = p["N"], p["L"], p["V"]
    lp = oracle.token_logp(p["logits"], V, p["y"], p["m"])["token_logp"]
    mu = (lp + p["rng"].normal(0, 0.8, N * L)).astype(np.float32)
    o_inf = oracle.pg_loss(p["logits"], N, L, V, p["y"], p["m"], mu, p["R"], p["go"], math.inf, 0)
    assert o_inf["n_clipped"] == 0
    o = oracle.pg_loss(p["logits"], N, L, V, p["y"], p["m"], mu, p["R"], p["go"], 2.0, 0)
    assert o["n_clipped"] == int((o["weight"] > 2.0).sum()) > 0
    lc = np.minimum(o["seq_log_ratio"], LN(2.0))
    assert o["mean_log_cw"] == pytest.approx(lc.mean(), abs=1e-14)
    assert o["mean_abs_log_cw"] == pytest.approx(np.abs(lc).mean(), abs=1e-14)
    np.testing.assert_allclose(np.log(o["clipped_w"]), lc, atol=1e-13)


def test_overflowing_weight_is_capped(oracle):
    """exp(s_n) = +inf must still clip to eta (IEEE min), not poison the group."""
    R = np.array([1, 0], np.float32)
    o = oracle.group_advantage(R, np.array([800.0, -800.0]), np.array([0, 2], np.int32), 2.0)
    assert o["clipped_w"].tolist() == [2.0, 0.0]
    assert o["adv64"].tolist() == [0.0, -1.0]


def test_result_independent_of_thread_count(oracle):
    p = _small_problem(seed=25, N=8, L=16, V=300, sizes=(4, 4))
    mu = p["rng"].normal(-5, 0.3, 8 * 16).astype(np.float32)
    outs = []
    for nt in (1, 4):
        oracle.set_threads(nt)
        outs.append(oracle.pg_loss(p["logits"], 8, 16, 300, p["y"], p["m"], mu, p["R"], p["go"], 2.0, 0,
                                   want_dlogits=True))
    oracle.set_threads(oracle.max_threads())
    assert outs[0]["loss"] == outs[1]["loss"]
    np.testing.assert_array_equal(outs[0]["dlogits"], outs[1]["dlogits"])
    np.testing.assert_array_equal(outs[0]["lse"], outs[1]["lse"])


def test_dlogits_rows_matches_dense_and_chunk_base(oracle):
    p = _small_problem(seed=26)
    N, L, V = p["N"], p["L"], p["V"]
    mu = p["rng"].normal(-2.4, 0.3, N * L).astype(np.float32)
    o = oracle.pg_loss(p["logits"], N, L, V, p["y"], p["m"], mu, p["R"], p["go"], 2.0, 0, want_dlogits=True)
    rows = np.array([0, 7, 13, 29], np.int64)
    d = oracle.dlogits_rows(p["logits"], V, L, p["y"], o["row_ok"], o["lse"], o["coef"], rows)
    np.testing.assert_array_equal(d, o["dlogits"][rows])
    d2 = oracle.dlogits_rows(p["logits"][10:], V, L, p["y"], o["row_ok"], o["lse"], o["coef"],
                             np.array([13, 29], np.int64), row_base=10)
    np.testing.assert_array_equal(d2, o["dlogits"][[13, 29]])


# --------------------------------------------------------------------------------------------
# fused-head form
# --------------------------------------------------------------------------------------------

def test_head_functions_against_matmul_and_fd(oracle):
    rng = np.random.default_rng(41)
    T, D, V = 6, 4, 9
    h_bits = bf16_bits(rng.normal(0, 1, (T, D)))
    w_bits = bf16_bits(rng.normal(0, 0.5, (D, V)))
    h, W = bf16_to_f64(h_bits), bf16_to_f64(w_bits)
    z = oracle.head_logits(h_bits, w_bits)
    np.testing.assert_allclose(z, h @ W, atol=1e-14)
    rows = np.array([4, 1], np.int64)
    np.testing.assert_array_equal(oracle.head_logits(h_bits, w_bits, rows), z[rows])
    y = rng.integers(0, V, T).astype(np.int32)
    lse, lp = oracle.token_logp_f64(z, y)
    ref = torch.log_softmax(torch.from_numpy(h @ W), 1).numpy()
    np.testing.assert_allclose(lp, ref[np.arange(T), y], atol=1e-14)
    g = rng.normal(0, 1, T)
    dz = oracle.dlogits_f64_inplace(z.copy(), y, lse, g)
    np.testing.assert_allclose(dz, g[:, None] * (np.exp(ref) - np.eye(V)[y]), atol=1e-14)
    dh = oracle.head_dhidden(dz, w_bits)
    np.testing.assert_allclose(dh, dz @ W.T, atol=1e-14)
    dW = np.zeros((D, V))
    oracle.head_dweight_accum(dW, dz[:3], h_bits, np.arange(3))
    oracle.head_dweight_accum(dW, dz[3:], h_bits, np.arange(3, 6))
    np.testing.assert_allclose(dW, h.T @ dz, atol=1e-14)

    # finite differences of the surrogate -sum_r g_r log pi(y_r) w.r.t. h and W (float64, frozen g)
    def surrogate(hh, WW):
        lsm = torch.log_softmax(torch.from_numpy(hh @ WW), 1).numpy()
        return -(g * lsm[np.arange(T), y]).sum()

    eps = 1e-6
    fd_h = np.zeros_like(h)
    for i in range(T):
        for d in range(D):
            hp, hm = h.copy(), h.copy()
            hp[i, d] += eps
            hm[i, d] -= eps
            fd_h[i, d] = (surrogate(hp, W) - surrogate(hm, W)) / (2 * eps)
    np.testing.assert_allclose(dh, fd_h, atol=1e-8)
    fd_W = np.zeros_like(W)
    for d in range(D):
        for v in range(V):
            Wp, Wm = W.copy(), W.copy()
            Wp[d, v] += eps
            Wm[d, v] -= eps
            fd_W[d, v] = (surrogate(h, Wp) - surrogate(h, Wm)) / (2 * eps)
    np.testing.assert_allclose(dW, fd_W, atol=1e-8)


def test_head_logits_dgemm_is_the_same_product(oracle):
    """The library-matmul form of z = h W against (i) a case whose every product and partial sum is
    an exact small integer, so any summation order gives the same bits, and (ii) the plain loops on
    random bf16 inputs, where the two may differ by summation order only."""
    h_int = np.array([[1, -2, 3], [0, 4, -1]], np.float64)
    W_int = np.array([[2, 0, -1, 5], [1, 1, 3, -2], [-4, 2, 0, 1]], np.float64)
    z = oracle.head_logits_dgemm(bf16_bits(h_int), oracle.decode_bf16(bf16_bits(W_int)))
    np.testing.assert_array_equal(z, [[-12, 4, -7, 12], [8, 2, 12, -9]])
    np.testing.assert_array_equal(oracle.head_logits(bf16_bits(h_int), bf16_bits(W_int)), z)

    rng = np.random.default_rng(43)
    T, D, V = 37, 96, 301
    h_bits = bf16_bits(rng.normal(0, 1, (T, D)))
    w_bits = bf16_bits(rng.normal(0, 0.02, (D, V)))
    np.testing.assert_array_equal(oracle.decode_bf16(w_bits), bf16_to_f64(w_bits))
    plain = oracle.head_logits(h_bits, w_bits)
    fast = oracle.head_logits_dgemm(h_bits, oracle.decode_bf16(w_bits))
    mag = np.abs(bf16_to_f64(h_bits)) @ np.abs(bf16_to_f64(w_bits))
    assert (np.abs(fast - plain) <= 4 * D * 2.0 ** -53 * mag).all()
    rows = np.array([30, 2, 2, 17], np.int64)
    np.testing.assert_array_equal(oracle.head_logits_dgemm(h_bits, oracle.decode_bf16(w_bits), rows), fast[rows])


# --------------------------------------------------------------------------------------------
# structural properties of the whole path (none of them is the oracle's own formula restated)
# --------------------------------------------------------------------------------------------

def _run(oracle, p, mu, logits=None, R=None, flags=0, eta=2.0, go=None, m=None):
    return oracle.pg_loss(p["logits"] if logits is None else logits, p["N"], p["L"], p["V"], p["y"],
                          p["m"] if m is None else m, mu, p["R"] if R is None else R,
                          p["go"] if go is None else go, eta, flags, want_dlogits=True)


def test_masked_rows_are_never_read(oracle):
    """Whatever a masked row holds -- here NaN -- the result does not change, and its gradient is zero."""
    p = _small_problem(seed=31)
    mu = (-3.0 + 0.3 * p["rng"].normal(size=p["N"] * p["L"])).astype(np.float32)
    a = _run(oracle, p, mu)
    poisoned = p["logits"].copy()
    poisoned[p["m"] == 0] = np.nan
    b = _run(oracle, p, mu, logits=poisoned)
    assert a["loss"] == b["loss"]
    np.testing.assert_array_equal(a["dlogits"], b["dlogits"])
    assert np.all(b["dlogits"][p["m"] == 0] == 0.0)


def test_per_row_shift_of_the_logits_changes_nothing(oracle):
    """softmax is invariant under adding a constant to a row: loss, weights and gradient stay put."""
    p = _small_problem(seed=32)
    mu = (-3.0 + 0.3 * p["rng"].normal(size=p["N"] * p["L"])).astype(np.float32)
    a = _run(oracle, p, mu)
    shift = (p["rng"].integers(-16, 16, (p["N"] * p["L"], 1)) / 4.0).astype(np.float32)  # exact in float32
    b = _run(oracle, p, mu, logits=p["logits"] + shift)
    assert b["loss"] == pytest.approx(a["loss"], rel=1e-12)
    np.testing.assert_allclose(b["dlogits"], a["dlogits"], atol=1e-14)
    np.testing.assert_allclose(b["weight"], a["weight"], rtol=1e-12)


def test_permuting_generations_inside_a_group_permutes_the_result(oracle):
    p = _small_problem(seed=33, N=6, sizes=(4, 2))
    N, L, V = p["N"], p["L"], p["V"]
    mu = (-3.0 + 0.3 * p["rng"].normal(size=N * L)).astype(np.float32)
    a = _run(oracle, p, mu)
    perm = np.array([2, 0, 3, 1, 5, 4])            # stays inside the groups {0..3} and {4, 5}
    rows = (perm[:, None] * L + np.arange(L)[None, :]).reshape(-1)
    q = dict(p, logits=p["logits"][rows], y=p["y"][rows], m=p["m"][rows], R=p["R"][perm])
    b = _run(oracle, q, mu[rows])
    assert b["loss"] == pytest.approx(a["loss"], rel=1e-12, abs=1e-15)
    np.testing.assert_allclose(b["adv64"], a["adv64"][perm], atol=1e-15)
    np.testing.assert_allclose(b["dlogits"], a["dlogits"][rows], atol=1e-15)


def test_token_normaliser_only_rescales(oracle):
    """Z = N versus Z = number of tokens: same direction, loss and gradient scaled by N / tokens."""
    p = _small_problem(seed=34)
    mu = (-3.0 + 0.3 * p["rng"].normal(size=p["N"] * p["L"])).astype(np.float32)
    a = _run(oracle, p, mu, flags=0)
    b = _run(oracle, p, mu, flags=2)
    k = p["N"] / a["n_tokens"]
    assert b["loss"] == pytest.approx(a["loss"] * k, rel=1e-12)
    np.testing.assert_allclose(b["dlogits"], a["dlogits"] * k, rtol=1e-12, atol=1e-18)
    np.testing.assert_array_equal(b["adv64"], a["adv64"])


def test_rewards_shifted_by_a_constant_on_policy(oracle):
    """Eq. 2 subtracts the group mean, so adding a constant to every reward of a group changes nothing
    when all weights are one (it does off-policy, through the weighted baseline of Eq. 5)."""
    p = _small_problem(seed=35, masked=False)
    lp = oracle.token_logp(p["logits"], p["V"], p["y"], p["m"])["token_logp"]
    A0 = oracle.group_advantage(p["R"], None, p["go"], 2.0)["adv64"]
    A1 = oracle.group_advantage((p["R"] + np.float32(2.5)).astype(np.float32), None, p["go"], 2.0)["adv64"]
    np.testing.assert_allclose(A1, A0, atol=1e-6)      # float32 rewards: the shift itself rounds
    s = p["rng"].normal(0, 0.5, p["N"])
    B0 = oracle.group_advantage(p["R"], s, p["go"], 2.0)["adv64"]
    B1 = oracle.group_advantage((p["R"] + np.float32(2.5)).astype(np.float32), s, p["go"], 2.0)["adv64"]
    c = np.minimum(np.exp(s), 2.0)
    # off-policy the advantage moves by 2.5 (1 - mean_group(c))
    go = p["go"]
    expect = np.concatenate([np.full(go[k + 1] - go[k], 2.5 * (1.0 - c[go[k]:go[k + 1]].mean())) for k in range(len(go) - 1)])
    np.testing.assert_allclose(B1 - B0, expect, atol=1e-6)
    assert lp.shape[0] == p["N"] * p["L"]
