"""CPU tests of the product's host side: the shared library loads and exports
every symbol the header declares; the host-only design functions (bit allocation,
code construction) agree with the float64 oracle and with the paper's constraints;
argument validation rejects bad plans without touching a GPU."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2605_15890_b200 as agc
from oracle import design as od

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "agc.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = set(re.findall(r"\b(agc_[a-z_0-9]+)\s*\(", header))
    assert {"agc_plan_create", "agc_encode_quantize", "agc_decode", "agc_bit_allocate"} <= names
    lib = ctypes.CDLL(agc.library_path())
    for nm in sorted(names):
        assert hasattr(lib, nm), nm
    assert agc.agc_version() >= 100
    assert agc.agc_strerror(-5).startswith("code violates")


@pytest.mark.parametrize("n,zres,dim", [(4, 12, 512), (10, 10, 128), (10, 50, 4096), (16, 32, 512),
                                        (50, 50, 512), (32, 64, 512)])
def test_allocators_against_oracle(n, zres, dim):
    rng = np.random.default_rng(n * 7 + zres)
    p = rng.uniform(0.02, 0.6, n)
    z_tot = 2 * n + zres
    bits_dp, F_dp = agc.agc_bit_allocate_dp(p, z_tot, b_max=8, phi_dim=dim)
    bits_o, F_o = od.bit_allocate_dp(p, z_tot, dim, b_max=8)
    assert abs(F_dp - F_o) <= 1e-10 * abs(F_o)
    assert bits_dp.sum() == z_tot and bits_dp.min() >= 2 and bits_dp.max() <= 8
    assert abs(od.allocation_value(p, bits_dp.astype(int) - 2, dim) - F_dp) <= 1e-10 * F_dp
    bits_a, F_a = agc.agc_bit_allocate(p, z_tot, b_max=8, phi_dim=dim)
    bits_ao, F_ao = od.bit_allocate_low_complexity(p, z_tot, dim, b_max=8)
    assert bits_a.sum() == z_tot and bits_a.min() >= 2 and bits_a.max() <= 8
    assert abs(od.allocation_value(p, bits_a.astype(int) - 2, dim) - F_a) <= 1e-10 * F_a
    assert F_a <= F_dp * (1 + 1e-12) and F_a >= 0.99 * F_dp
    assert abs(F_a - F_ao) <= 1e-9 * abs(F_ao)


def test_allocator_uncapped_and_errors():
    p = np.array([0.05, 0.3, 0.5])
    bits, F = agc.agc_bit_allocate(p, 30, b_max=0, phi_dim=100000.0)
    bits_o, F_o = od.bit_allocate_dp(p, 30, 100000.0)
    assert bits.sum() == 30 and F >= 0.99 * F_o
    with pytest.raises(agc.AgcError) as e:
        agc.agc_bit_allocate(p, 5)
    assert e.value.code == -8
    with pytest.raises(agc.AgcError) as e:
        agc.agc_bit_allocate(np.array([0.1, 1.0]), 8)
    assert e.value.code == -3
    with pytest.raises(agc.AgcError):
        agc.agc_bit_allocate(p, 100, b_max=8)  # 3 workers cannot hold 100 bits under the cap


@pytest.mark.parametrize("n,k", [(4, 4), (16, 16), (32, 32), (10, 25), (100, 100)])
def test_interval_code_against_oracle(n, k):
    rng = np.random.default_rng(n + k)
    p = rng.uniform(0.02, 0.6, n)
    bits = rng.integers(2, 9, n).astype(np.uint8)
    rp, ci, a, w, Y = agc.agc_code_build(n, k, p, bits, 512.0)
    A = od.csr_to_dense(rp, ci, a.astype(np.float64), k)
    Yo = od.optimal_row_sums(p, bits, k, 512)
    assert np.abs(Y - Yo).max() < 1e-9
    assert np.abs(A - od.interval_alpha(Yo, k)).max() < 1e-6
    assert len(ci) <= n + k - 1
    assert od.unbiasedness_residual(A, w.astype(np.float64), p) < 1e-5
    for i in range(n):
        assert (np.diff(ci[rp[i]:rp[i + 1]]) > 0).all()


@pytest.mark.parametrize("n,s", [(4, 2), (8, 3), (16, 3), (32, 4), (100, 5)])
def test_support_code_is_optimal_on_cyclic_supports(n, s):
    rng = np.random.default_rng(n * 10 + s)
    p = rng.uniform(0.02, 0.6, n)
    bits = rng.integers(2, 9, n).astype(np.uint8)
    sup = od.cyclic_support(n, n, s)
    srp = np.arange(0, n * s + 1, s, dtype=np.int32)
    sci = np.array(sum(sup, []), np.int32)
    rp, ci, a, w, Y = agc.agc_code_build(n, n, p, bits, 512.0, mode=agc.AGC_CODE_SUPPORT,
                                         sup_row_ptr=srp, sup_col_idx=sci)
    A = od.csr_to_dense(rp, ci, a.astype(np.float64), n)
    c = od.c_coeff(p, bits, 512)
    col_err, excess, neg = od.support_kkt_gap(A, c, sup)
    assert col_err < 1e-6 and excess < 1e-5 and neg >= 0
    assert od.unbiasedness_residual(A, w.astype(np.float64), p) < 1e-5
    val = od.structure_objective(A, c)
    assert val >= od.optimal_objective(c, n) * (1 - 1e-6)
    if n <= 16:
        _, ref = od.support_restricted_alpha_reference(c, sup, n)
        assert abs(val - ref) <= 1e-5 * ref


def test_plan_validation_rejects_bad_input_before_any_gpu_work():
    rp = np.array([0, 1, 2], np.int32)
    ci = np.array([0, 1], np.int32)
    a = np.ones(2, np.float32)
    p = np.array([0.2, 0.5], np.float32)
    w = (1 / (1 - p)).astype(np.float32)
    bad = [
        (dict(bits=[1, 4]), -2),
        (dict(bits=[4, 9]), -2),
        (dict(p=np.array([0.2, 1.0], np.float32)), -3),
        (dict(w=np.array([1.0, 1.0], np.float32)), -5),
        (dict(bucket=100), -1),
        (dict(ci=np.array([0, 2], np.int32)), -1),
        (dict(d=0), -1),
    ]
    for kw, code in bad:
        args = dict(rp=rp, ci=ci, a=a, w=w, p=p, bits=[4, 4], bucket=512, d=1000)
        args.update(kw)
        with pytest.raises(agc.AgcError) as e:
            agc.agc_plan_create(2, 2, args["d"], args["rp"], args["ci"], args["a"], args["w"], args["p"],
                                args["bits"], args["bucket"], 0, 0)
        assert e.value.code == code, kw


def test_two_track_vector_against_oracle():
    """v* of Sec. V-E from the library against the float64 oracle (itself pinned as the
    minimiser of Eq. twodec)."""
    rng = np.random.default_rng(12)
    for n, k in [(4, 4), (7, 12), (16, 16)]:
        p = rng.uniform(0.02, 0.5, n)
        bits = rng.integers(2, 9, n).astype(np.uint8)
        alpha = od.interval_alpha(od.optimal_row_sums(p, bits, k, 256), k)
        rp, ci, vals = od.alpha_to_csr(alpha)
        A = np.zeros((n, k))
        for i in range(n):
            A[i, ci[rp[i]:rp[i + 1]]] = vals[rp[i]:rp[i + 1]].astype(np.float32)
        for lam in (0.5, 1.0, 4.0):
            v = agc.agc_two_track_vector(n, k, p, bits, 256.0, rp, vals.astype(np.float32), lam=lam)
            want = od.two_track_decoder(A, p, bits, 256, lam=lam)
            assert np.allclose(v, want, rtol=2e-6, atol=0)


def test_eta_balance_and_its_use_in_the_design_calls():
    """Sec. V-B: the suggested eta against the oracle; with it the allocator and the code builder
    of the library still agree with the oracle's (eta enters phi everywhere)."""
    rng = np.random.default_rng(6)
    n, k, dim, z_tot = 10, 10, 512, 40
    p = rng.uniform(0.05, 0.5, n)
    eta = agc.agc_eta_balance(p, z_tot, float(dim))
    assert np.isclose(eta, od.eta_balance(p, z_tot, dim), rtol=1e-12)
    assert np.isclose(eta * od.phi(z_tot // n, dim), p.mean(), rtol=1e-12)
    bits, F = agc.agc_bit_allocate(p, z_tot, b_max=8, phi_dim=float(dim), eta=eta)
    obits, oF = od.bit_allocate_low_complexity(p, z_tot, dim, b_max=8, eta=eta)
    assert bits.sum() == z_tot and np.isclose(F, oF, rtol=1e-9)
    rp, ci, a, w, Y = agc.agc_code_build(n, k, p, bits, float(dim), eta=eta)
    assert np.allclose(Y, od.optimal_row_sums(p, bits, k, dim, eta=eta), rtol=1e-9)


@pytest.mark.parametrize("n", [10, 50])
def test_allocator_under_the_papers_delay_model(n):
    """The setting of the paper's allocator figure: p_i from the shifted-exponential delay model
    (psi ~ U(0.1, 2), deadline 1.1), residual budgets n and 5n. The library's Algorithm 1 stays
    within 1 % of its own exact DP and never below the equal split."""
    from synth import configs as cfgs
    p = np.minimum(cfgs.shifted_exponential_probs(n, seed=n), 0.95)
    for zres in (n, 5 * n):
        bits, F = agc.agc_bit_allocate(p, 2 * n + zres, b_max=0, phi_dim=512.0)
        _, F_dp = agc.agc_bit_allocate_dp(p, 2 * n + zres, b_max=0, phi_dim=512.0)
        assert bits.sum() == 2 * n + zres and (bits >= 2).all()
        assert F_dp * (1 + 1e-12) >= F >= 0.99 * F_dp
        base, rem = divmod(zres, n)
        order = np.argsort(p, kind="stable")
        r_eq = np.zeros(n, int)
        r_eq[order] = base + (np.arange(n) < rem)
        assert F >= od.allocation_value(p, r_eq, 512) * (1 - 1e-12)


def test_comparison_allocators_against_oracle_and_orderings():
    """The library's greedy / continuous-relaxation heuristics and its upper bound against the
    oracle's (same readings, float64), and the orderings of the allocator comparison of Sec. VI on
    the shifted-exponential model at n = 10 and 50."""
    from paper_2605_15890_b200 import allocator_study
    rng = np.random.default_rng(51)
    for trial in range(6):
        n = int(rng.integers(3, 14))
        zres = int(rng.integers(1, 4 * n))
        p = rng.uniform(0.02, 0.9, n)
        dim = float(rng.choice([8, 512, 4096]))
        z_tot = 2 * n + zres
        bg, Fg = agc.agc_bit_allocate_heuristic(agc.AGC_ALLOC_GREEDY, p, z_tot, b_max=0, phi_dim=dim)
        obg, oFg = od.bit_allocate_greedy(p, z_tot, dim)
        assert (bg == obg).all() and np.isclose(Fg, oFg, rtol=1e-12)
        br, Fr = agc.agc_bit_allocate_heuristic(agc.AGC_ALLOC_RELAXATION, p, z_tot, b_max=0, phi_dim=dim)
        obr, oFr = od.bit_allocate_relaxation(p, z_tot, dim)
        assert br.sum() == z_tot and np.isclose(Fr, oFr, rtol=1e-9)
        assert np.isclose(agc.agc_allocation_upper_bound(p, z_tot, b_max=0, phi_dim=dim),
                          od.allocation_upper_bound(p, z_tot, dim), rtol=1e-12)
    for with_eta in (False, True):
        for r in allocator_study.study(ns=(10, 50), multiples=(1, 3, 5), seeds=3, with_eta=with_eta):
            assert r["alg1_min_ratio"] >= 0.99 and r["alg1"] <= r["dp"] * (1 + 1e-12)
            assert r["greedy"] <= r["dp"] * (1 + 1e-12) and r["relaxation"] <= r["dp"] * (1 + 1e-12)
            assert r["bound"] >= r["dp"] * (1 - 1e-12)
