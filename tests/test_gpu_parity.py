"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the
same seeded inputs. Packed codes, scales and the single-realisation decode must be
bit-exact; the collapsed multi-realisation update must agree to 1e-5 relative."""
import os

import numpy as np
import pytest

from oracle import design as od
from oracle import roundpath as orp
from synth import configs as cfgs
from tests import _codes

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def agc():
    import paper_2605_15890_b200 as m
    return m


@pytest.fixture(scope="module")
def torch():
    import torch as t
    return t


def run_both(agc, torch, G_host, code, p, bits, B, seed, rnd, masks, flags=0, d=None, lr=None, beta0=None,
             ld_pad=0):
    """Encode + decode on the GPU and with the oracle; returns both result sets."""
    from paper_2605_15890_b200.session import Session
    rp, ci, a, w = code
    k = G_host.shape[0]
    d = G_host.shape[1] if d is None else d
    n = len(bits)
    if any(b == 1 for b in bits):
        flags |= agc.AGC_FLAG_ALLOW_1BIT
    ses = Session(n, k, d, rp, ci, a, w, p, bits, bucket=B, seed=seed, flags=flags | agc.AGC_FLAG_NO_UNBIASED_CHECK)
    ld = ((d + 3) // 4) * 4 + ld_pad
    G = torch.zeros((k, ld), dtype=torch.float32, device="cuda")
    G[:, :d] = torch.from_numpy(np.ascontiguousarray(G_host[:, :d]))
    if ld > d:
        G[:, d:] = 7.0  # padding the kernel must never read as data
    ses.codes.fill_(-1)
    ses.scales.fill_(-1.0)
    ses.encode(G, rnd)
    masks = np.atleast_2d(masks).astype(np.uint8)
    R = masks.shape[0]
    m_dev = torch.from_numpy(masks).cuda()
    ghat = torch.full((R, d), -3.0, dtype=torch.float32, device="cuda")
    ses.decode(m_dev, ghat=ghat)
    out = dict(codes=ses.codes_host(), scales=ses.scales_host(), ghat=ghat.cpu().numpy(),
               status=int(ses.status.item()), tma=ses.uses_tma)
    if beta0 is not None:
        b1 = torch.from_numpy(beta0.copy()).cuda()
        ses.decode(m_dev, lr=lr, ghat=ghat, beta=b1)      # sequential definition
        out["beta_seq"] = b1.cpu().numpy()
        b2 = torch.from_numpy(beta0.copy()).cuda()
        ses.decode(m_dev, lr=lr, beta=b2)                  # collapsed when R > 1
        out["beta_fused"] = b2.cpu().numpy()
    torch.cuda.synchronize()
    ses.close()
    Gd = np.ascontiguousarray(G_host[:, :d])
    if B == 0:        # one norm per worker
        oc, osc, ost, _ = orp.encode_quantize_global(rp, ci, a, bits, seed, rnd, Gd, d=d)
        dec_scales, dec_B, osc = orp.expand_global_scales(osc, d), 512, osc.reshape(n, 1)
    elif B > 512:     # buckets of several pack blocks
        oc, osc, ost, _ = orp.encode_quantize_grouped(rp, ci, a, bits, B, seed, rnd, Gd, d=d)
        dec_scales, dec_B = orp.expand_grouped_scales(osc, d, B), 512
    else:
        oc, osc, ost, _ = orp.encode_quantize(rp, ci, a, bits, B, seed, rnd, Gd, d=d)
        dec_scales, dec_B = osc, B
    og, ob = orp.decode(d, bits, dec_B, w, masks, oc, dec_scales, lr=lr, beta=beta0)
    ref = dict(codes=oc, scales=osc, ghat=og, status=ost, beta=ob)
    return out, ref


def assert_exact(out, ref):
    assert out["scales"].shape == ref["scales"].shape
    assert (out["scales"].view(np.uint32) == ref["scales"].view(np.uint32)).all()
    assert out["codes"].shape == ref["codes"].shape
    bad = np.nonzero(out["codes"] != ref["codes"])[0]
    assert bad.size == 0, f"{bad.size} code words differ, first at {bad[:5]}"
    assert (out["ghat"].view(np.uint32) == ref["ghat"].view(np.uint32)).all()
    assert (out["status"] & 1) == (ref["status"] & 1)
    assert out["status"] & 4 == 0


def test_config1_all_rounds_bit_exact(agc, torch):
    """n=k=4, cyclic s=2, d=10,000 (not a multiple of the block), b=(2,3,4,8), 100 rounds
    each with a fresh Bernoulli straggler mask."""
    wl = cfgs.config1()
    code = _codes.cyclic_code(wl.p, wl.bits, wl.k, wl.s, 512)
    masks = cfgs.straggler_masks(wl)
    for t in range(wl.rounds):
        G = cfgs.partials_numpy(wl, t)
        out, ref = run_both(agc, torch, G, code, wl.p, wl.bits, 512, wl.seed, t, masks[t, 0])
        assert_exact(out, ref)
        assert out["tma"]


@pytest.mark.parametrize("d", [1, 3, 127, 128, 129, 511, 512, 513, 1000, 4097, 70001])
@pytest.mark.parametrize("B", [128, 256, 512])
@pytest.mark.parametrize("direct", [False, True, "ring"])
def test_ragged_sizes_all_bit_widths(agc, torch, d, B, direct):
    rng = np.random.default_rng(d * 7 + B)
    n = k = 8
    bits = np.arange(1, 9, dtype=np.uint8)
    p = rng.uniform(0.05, 0.5, n)
    code = _codes.cyclic_code(p, bits, k, 3, B)
    G = (rng.standard_normal((k, d)) * 10.0 ** rng.uniform(-3, 2, (k, 1))).astype(np.float32)
    masks = (rng.random((2, n)) > 0.3).astype(np.uint8)
    # three routes: staged encoder + the short-vector decoder (these lengths are below one pack
    # block per SM), both direct-load kernels, staged encoder + staged (ring) decoder
    flags = agc.AGC_FLAG_FORCE_DIRECT if direct is True else agc.AGC_FLAG_NO_ROW_DECODE if direct == "ring" else 0
    out, ref = run_both(agc, torch, G, code, p, bits, B, 1234 + d, 5, masks, flags=flags, ld_pad=4 if d % 2 else 0,
                        beta0=rng.standard_normal(d).astype(np.float32), lr=np.array([0.01, 0.02], np.float32))
    assert_exact(out, ref)
    assert (out["beta_seq"].view(np.uint32) == ref["beta"].view(np.uint32)).all()
    assert np.abs(out["beta_fused"] - ref["beta"]).max() <= 1e-5 * np.abs(ref["beta"]).max()
    assert out["tma"] == (direct is not True)


@pytest.mark.parametrize("kind", ["identity", "interval", "s1", "s_eq_k", "wide_rows", "many_groups", "many_workers", "scattered", "thousands"])
def test_code_structures(agc, torch, kind):
    rng = np.random.default_rng(["identity", "interval", "s1", "s_eq_k", "wide_rows", "many_groups", "many_workers", "scattered", "thousands"].index(kind))
    d = 3000
    if kind == "identity":
        n = k = 5
        bits = np.array([2, 8, 3, 5, 4], np.uint8)
        p = np.zeros(n)
        code = _codes.identity_code(n)
    elif kind == "interval":
        n, k = 7, 12
        bits = rng.integers(2, 9, n).astype(np.uint8)
        p = rng.uniform(0.05, 0.5, n)
        code = _codes.interval_code(p, bits, k, 512)
    elif kind == "s1":
        n = k = 6
        bits = rng.integers(2, 9, n).astype(np.uint8)
        p = rng.uniform(0.05, 0.5, n)
        code = _codes.cyclic_code(p, bits, k, 1, 512)
    elif kind == "s_eq_k":
        n = k = 6
        bits = rng.integers(2, 9, n).astype(np.uint8)
        p = rng.uniform(0.05, 0.5, n)
        code = _codes.cyclic_code(p, bits, k, k, 512)
    elif kind == "wide_rows":      # a support wider than a staged tile: direct kernel
        n = k = 45
        bits = rng.integers(2, 9, n).astype(np.uint8)
        p = rng.uniform(0.05, 0.5, n)
        code = _codes.cyclic_code(p, bits, k, 40, 512)
    elif kind == "thousands":      # more workers than the staged kernels' tables hold: both fall back
        n = k = 2100
        d = 700
        bits = rng.integers(1, 9, n).astype(np.uint8)
        p = rng.uniform(0.01, 0.5, n)
        code = _codes.cyclic_code(p, bits, k, 2, 512)
    elif kind == "scattered":      # supports scattered over the partitions (not banded): clustered groups
        n, k = 60, 90
        bits = rng.integers(1, 9, n).astype(np.uint8)
        p = rng.uniform(0.01, 0.5, n)
        alpha = np.zeros((n, k))
        for j in range(k):
            holders = rng.choice(n, size=3, replace=False)
            alpha[holders, j] = rng.uniform(0.2, 1.0, 3)
        alpha /= alpha.sum(0, keepdims=True)
        rp_, ci_, vals_ = od.alpha_to_csr(alpha)
        _, w_ = od.physical_coefficients(alpha, p)
        code = (rp_, ci_, vals_.astype(np.float32), w_.astype(np.float32))
    elif kind == "many_workers":   # hundreds of workers: many groups in both kernels
        n = k = 300
        bits = rng.integers(1, 9, n).astype(np.uint8)
        p = rng.uniform(0.01, 0.6, n)
        code = _codes.cyclic_code(p, bits, k, 2, 512)
    else:                          # many worker groups per block in the staged kernel
        n = k = 100
        bits = rng.integers(1, 9, n).astype(np.uint8)
        p = rng.uniform(0.01, 0.6, n)
        code = _codes.cyclic_code(p, bits, k, 5, 512)
    G = rng.standard_normal((k, d)).astype(np.float32)
    masks = (rng.random((1, n)) >= p).astype(np.uint8)
    out, ref = run_both(agc, torch, G, code, p, bits, 512, 77, 3, masks)
    assert_exact(out, ref)
    assert out["tma"] == (kind not in ("wide_rows", "thousands"))
    assert G.shape[0] == k


@pytest.mark.parametrize("case", range(int(os.environ.get("AGC_SWEEP_CASES", "16"))))   # more cases for a longer sweep
def test_seeded_random_shapes_codes_and_masks(agc, torch, case):
    """Random worker / partition counts, sparse supports, widths, bucket sizes, lengths (a few
    blocks up to several hundred: every tile height of the decoder), heavy-tailed values, 64-bit
    seeds and round numbers, several realisations with the fused update."""
    rng = np.random.default_rng(9000 + case)
    n = int(rng.integers(1, 70))
    k = int(rng.integers(1, 50))
    B = int(rng.choice([128, 256, 512, 512, 1024, 2048, 4096, 0]))
    d = int(rng.choice([rng.integers(1, 3000), rng.integers(3000, 80_000), rng.integers(80_000, 400_000)]))
    if n * d > 6_000_000:
        d = 6_000_000 // n
    bits = rng.integers(1, 9, n).astype(np.uint8)
    p = rng.uniform(0.0, 0.7, n)
    rp = [0]
    ci, a = [], []
    for i in range(n):
        cols = np.sort(rng.choice(k, size=int(rng.integers(1, min(k, 6) + 1)), replace=False))
        ci.extend(cols.tolist())
        a.extend((rng.standard_normal(cols.size) * 10.0 ** rng.uniform(-2, 1)).tolist())
        rp.append(len(ci))
    code = (np.array(rp, np.int32), np.array(ci, np.int32), np.array(a, np.float32),
            (rng.standard_normal(n) * 2).astype(np.float32))
    G = (rng.standard_t(3, (k, d)) * 10.0 ** rng.uniform(-4, 3, (k, 1))).astype(np.float32)
    if case % 4 == 0:
        G[rng.integers(0, k), : min(d, 600)] = 0.0          # stretches of zeros inside a row
    R = int(rng.integers(1, 5))
    if case % 3 == 0 and n * d <= 400_000:
        R = int(rng.integers(8, 70))                        # g_hat of all realisations in one pass
    masks = (rng.random((R, n)) >= p).astype(np.uint8)
    lr = rng.uniform(1e-3, 1e-1, R).astype(np.float32)
    beta0 = rng.standard_normal(d).astype(np.float32)
    seed = int(rng.integers(0, 2**63)) * 2 + 1
    rnd = int(rng.integers(0, 2**63))
    # short vectors: every other case keeps the staged decoder instead of the warp-per-row kernel
    flags = agc.AGC_FLAG_NO_ROW_DECODE if case % 2 else 0
    out, ref = run_both(agc, torch, G, code, p, bits, B, seed, rnd, masks, lr=lr, beta0=beta0,
                        ld_pad=int(rng.choice([0, 4, 36])), flags=flags)
    assert_exact(out, ref)
    assert (out["beta_seq"].view(np.uint32) == ref["beta"].view(np.uint32)).all()
    scale = max(np.abs(ref["beta"]).max(), 1e-30)
    assert np.abs(out["beta_fused"] - ref["beta"]).max() / scale <= 1e-5


def test_straggler_extremes_and_batched_decode(agc, torch):
    """All stragglers (g_hat = 0), none, single survivors; R realisations with per-
    realisation outputs, the sequential update and the collapsed update."""
    rng = np.random.default_rng(11)
    n = k = 8
    d = 5000
    bits = np.array([1, 2, 3, 4, 5, 6, 7, 8], np.uint8)
    p = rng.uniform(0.05, 0.5, n)
    code = _codes.cyclic_code(p, bits, k, 2, 256)
    G = rng.standard_normal((k, d)).astype(np.float32)
    masks = np.concatenate([np.zeros((1, n)), np.ones((1, n)), np.eye(n), rng.random((6, n)) > 0.4]).astype(np.uint8)
    R = masks.shape[0]
    lr = rng.uniform(0.001, 0.01, R).astype(np.float32)
    beta0 = rng.standard_normal(d).astype(np.float32)
    out, ref = run_both(agc, torch, G, code, p, bits, 256, 3, 9, masks, lr=lr, beta0=beta0)
    assert_exact(out, ref)
    assert (out["ghat"][0] == 0).all()
    assert (out["beta_seq"].view(np.uint32) == ref["beta"].view(np.uint32)).all()
    rel = np.abs(out["beta_fused"] - ref["beta"]).max() / np.abs(ref["beta"]).max()
    assert rel <= 1e-5
    # R = 1 fused update is the definition itself
    out1, ref1 = run_both(agc, torch, G, code, p, bits, 256, 3, 9, masks[12:13], lr=lr[:1], beta0=beta0)
    assert (out1["beta_fused"].view(np.uint32) == ref1["beta"].view(np.uint32)).all()


def test_nonfinite_and_zero_buckets(agc, torch):
    rng = np.random.default_rng(2)
    n = k = 4
    d = 2048
    bits = np.array([1, 2, 5, 8], np.uint8)
    p = np.full(n, 0.2)
    code = _codes.cyclic_code(p, bits, k, 2, 512)
    G = rng.standard_normal((k, d)).astype(np.float32)
    G[:, 512:1024] = 0.0
    G[1, 1500] = np.inf
    G[2, 100] = np.nan
    out, ref = run_both(agc, torch, G, code, p, bits, 512, 1, 0, np.ones((1, n)))
    assert ref["status"] & 1 and out["status"] & 1
    assert (out["scales"].view(np.uint32) == ref["scales"].view(np.uint32)).all()
    assert (out["codes"] == ref["codes"]).all()
    both_nan = np.isnan(out["ghat"]) & np.isnan(ref["ghat"])
    assert ((out["ghat"].view(np.uint32) == ref["ghat"].view(np.uint32)) | both_nan).all()


@pytest.mark.parametrize("B", [128, 256, 512, 2048, 0])
@pytest.mark.parametrize("direct", [False, True])
def test_buckets_with_tiny_sums_of_squares(agc, torch, B, direct):
    """Sums of squares across the whole exponent range: ordinary, between the smallest normal
    number and 2^-102 (the encoder's general square root and division), below the smallest normal
    (flushed), huge. Blocks differ in magnitude, so every path occurs in one message."""
    rng = np.random.default_rng(31 + B)
    n = k = 6
    d = 16 * 512 + 77
    bits = np.array([1, 2, 3, 4, 6, 8], np.uint8)
    p = np.full(n, 0.1)
    code = _codes.cyclic_code(p, bits, k, 2, 512)
    G = rng.standard_normal((k, d)).astype(np.float32)
    mags = [1.0, 1e-15, 3e-17, 1e-18, 2e-19, 1e-20, 1e-22, 1e17, 3e-16, 7e-17, 1e-17, 5e-18, 4e-19, 1e-19, 1e5, 1e-25, 1.0]
    for q, m in enumerate(mags):
        G[:, q * 512:(q + 1) * 512] *= np.float32(m)
    G[:, 3 * 512 + 128:3 * 512 + 256] = 0.0      # a flushed 128-bucket next to tiny ones
    out, ref = run_both(agc, torch, G, code, p, bits, B, 3, 1, np.ones((1, n)),
                        flags=agc.AGC_FLAG_FORCE_DIRECT if direct else 0)
    assert out["status"] == 0 and ref["status"] == 0
    assert (out["scales"].view(np.uint32) == ref["scales"].view(np.uint32)).all()
    if B in (128, 256, 512):
        tiny = (ref["scales"] > 0) & (ref["scales"] < 2.0 ** -51)
        assert tiny.any() and (ref["scales"] == 0).any()
    assert (out["codes"] == ref["codes"]).all()
    assert (out["ghat"].view(np.uint32) == ref["ghat"].view(np.uint32)).all()


@pytest.mark.parametrize("B,direct", [(512, False), (128, False), (512, True), (0, False), (2048, False)])
def test_workers_without_entries_send_the_zero_vector(agc, torch, B, direct):
    """A worker whose row of A is empty encodes f_i = 0: zero codes, scale 0, in every mode
    (the unbiasedness check is off: the other workers carry the partitions)."""
    rng = np.random.default_rng(5 + B)
    n, k, d = 7, 5, 3 * 512 + 100
    bits = np.array([3, 1, 8, 2, 5, 4, 6], np.uint8)
    p = np.full(n, 0.2)
    sup = [[0, 1], [], [2], [], [1, 3, 4], [0], []]
    rp = np.zeros(n + 1, np.int32)
    ci, a = [], []
    for i, cols in enumerate(sup):
        ci += cols
        a += list(rng.uniform(0.3, 1.5, len(cols)))
        rp[i + 1] = len(ci)
    code = (rp, np.array(ci, np.int32), np.array(a, np.float32), rng.uniform(0.5, 1.5, n).astype(np.float32))
    G = rng.standard_normal((k, d)).astype(np.float32)
    masks = np.ones((2, n), np.uint8)
    masks[1, 2] = 0
    out, ref = run_both(agc, torch, G, code, p, bits, B, 21, 2, masks,
                        flags=agc.AGC_FLAG_FORCE_DIRECT if direct else 0)
    assert_exact(out, ref)
    assert (ref["scales"][[1, 3, 6]] == 0).all()


@pytest.mark.parametrize("B", [128, 512])
def test_decode_coefficients_across_the_exponent_range(agc, torch, B):
    """Decoding coefficients w_i S / L from the subnormal range up to 1e30: the decoder scales a
    coefficient by a power of two where the code sits in its word, which is exact only inside
    the normal range; smaller coefficients must take its general path and give the same bits
    as the oracle's plain fma chain."""
    rng = np.random.default_rng(17 + B)
    n = k = 8
    d = 5 * 512 + 33
    bits = np.array([2, 3, 4, 5, 6, 7, 8, 2], np.uint8)
    p = np.full(n, 0.1)
    rp, ci, a, _ = _codes.cyclic_code(p, bits, k, 2, B)
    G = rng.standard_normal((k, d)).astype(np.float32)
    for w in ([1e-30, 1e-33, 1e-36, 1e-38, 1e-41, 1e-44, 1.0, 1e-35], [1e30, 1.0, 1e-20, 3e-34, 0.0, -1e-37, -2.5, 1e-39]):
        w = np.array(w, np.float32)
        out, ref = run_both(agc, torch, G, (rp, ci, a, w), p, bits, B, 3, 1, np.ones((1, n)),
                            flags=agc.AGC_FLAG_NO_UNBIASED_CHECK)
        assert_exact(out, ref)
    # tiny values as well: scales near 2^-60 with ordinary weights
    out, ref = run_both(agc, torch, G * np.float32(1e-19), (rp, ci, a, np.ones(n, np.float32)), p, bits, B, 3, 1,
                        np.ones((1, n)), flags=agc.AGC_FLAG_NO_UNBIASED_CHECK)
    assert_exact(out, ref)
    out, ref = run_both(agc, torch, G * np.float32(1e-19), (rp, ci, a, np.full(n, 1e-15, np.float32)), p, bits, B, 3, 1,
                        np.ones((1, n)), flags=agc.AGC_FLAG_NO_UNBIASED_CHECK)
    assert_exact(out, ref)


def test_same_round_same_bits_other_round_other_bits(agc, torch):
    wl = cfgs.config1()
    code = _codes.cyclic_code(wl.p, wl.bits, wl.k, wl.s, 512)
    G = cfgs.partials_numpy(wl, 0)
    a, _ = run_both(agc, torch, G, code, wl.p, wl.bits, 512, 5, 7, np.ones((1, 4)))
    b, _ = run_both(agc, torch, G, code, wl.p, wl.bits, 512, 5, 7, np.ones((1, 4)))
    c, _ = run_both(agc, torch, G, code, wl.p, wl.bits, 512, 5, 8, np.ones((1, 4)))
    assert (a["codes"] == b["codes"]).all() and (a["codes"] != c["codes"]).any()


def test_config2_rounds_bit_exact(agc, torch):
    """n=k=16, s=3, d=2^20, per-partition scales log-uniform in [1e-3, 1], bits from the
    allocator under Z_tot = 64."""
    wl = cfgs.config2()
    bits, _ = od.bit_allocate_low_complexity(wl.p, wl.z_tot, 512, b_max=8)
    code = _codes.cyclic_code(wl.p, bits, wl.k, wl.s, 512)
    masks = cfgs.straggler_masks(wl, rounds=2)
    for t in range(2):
        G = cfgs.partials_numpy(wl, t)
        out, ref = run_both(agc, torch, G, code, wl.p, bits, 512, wl.seed, t, masks[t, 0])
        assert_exact(out, ref)


def test_host_buffer_round(agc, torch):
    from paper_2605_15890_b200.session import Session
    wl = cfgs.config1()
    rp, ci, a, w = _codes.cyclic_code(wl.p, wl.bits, wl.k, wl.s, 512)
    ses = Session(wl.n, wl.k, wl.d, rp, ci, a, w, wl.p, wl.bits, bucket=512, seed=3)
    G = torch.from_numpy(cfgs.partials_numpy(wl, 0)).pin_memory()
    mask = torch.tensor([1, 0, 1, 1], dtype=torch.uint8).pin_memory()
    ghat = torch.empty(wl.d, dtype=torch.float32).pin_memory()
    for rnd in (0, 1):
        st = agc.agc_round_host(ses.plan, G, wl.d, rnd, mask, ghat)
        assert st == 0
        oc, osc, _, _ = orp.encode_quantize(rp, ci, a, wl.bits, 512, 3, rnd, G.numpy())
        og, _ = orp.decode(wl.d, wl.bits, 512, w, mask.numpy()[None], oc, osc)
        assert (ghat.numpy().view(np.uint32) == og[0].view(np.uint32)).all()
    ses.close()


def test_shards_with_block_offsets_reproduce_the_whole_vector(agc, torch):
    """The multi-GPU recipe on one GPU: two plans over pack-block-aligned halves, each told
    its first block, give the corresponding slices of the whole vector's codes and scales."""
    from paper_2605_15890_b200 import sharding
    from paper_2605_15890_b200.session import Session
    rng = np.random.default_rng(8)
    n = k = 6
    d = 512 * 9 + 77
    B = 128
    bits = np.array([2, 3, 4, 5, 7, 8], np.uint8)
    p = rng.uniform(0.05, 0.5, n)
    rp, ci, a, w = _codes.cyclic_code(p, bits, k, 3, B)
    G_host = rng.standard_normal((k, d)).astype(np.float32)
    oc, osc, _, _ = orp.encode_quantize(rp, ci, a, bits, B, 31, 2, G_host)
    off = orp.worker_word_offsets(d, bits)
    for rank in range(2):
        lo, hi = sharding.coordinate_range(d, rank, 2)
        ds = hi - lo
        ses = Session(n, k, ds, rp, ci, a, w, p, bits, bucket=B, seed=31)
        ses.set_first_block(sharding.first_block(d, rank, 2))
        ld = (ds + 3) // 4 * 4
        G = torch.zeros((k, ld), dtype=torch.float32, device="cuda")
        G[:, :ds] = torch.from_numpy(np.ascontiguousarray(G_host[:, lo:hi]))
        ses.encode(G, 2)
        torch.cuda.synchronize()
        codes, scales = ses.codes_host(), ses.scales_host()
        nblk_s = (ds + 511) // 512
        q0 = lo // 512
        for i in range(n):
            b = int(bits[i])
            w_lo, w_hi = ses.worker_words(i)
            assert w_hi - w_lo == nblk_s * 16 * b
            want = oc[off[i] + q0 * 16 * b: off[i] + (q0 + nblk_s) * 16 * b]
            assert (codes[w_lo:w_hi] == want).all()
        nb_s = scales.shape[1]
        assert (scales.view(np.uint32) == osc[:, lo // B: lo // B + nb_s].view(np.uint32)).all()
        ses.close()


@pytest.mark.parametrize("d,shards,direct", [(512 * 11 + 37, 3, False), (600_001, 2, False), (512 * 11 + 37, 2, True)])
def test_global_norm_over_shards_equals_the_whole_vector(agc, torch, d, shards, direct):
    """One norm per worker over a vector held as `shards` plans (one GPU here, one per GPU in
    use): first pass per shard, the library's combine of the shards' sums, second pass with the
    whole vector's sums and the shard's block offset. With power-of-two shard sizes the
    codes and scales equal the oracle's unsplit global-norm encoding bit for bit; a plain
    agc_encode_quantize on an offset global-norm plan is refused."""
    from paper_2605_15890_b200 import sharding
    from paper_2605_15890_b200.session import Session
    rng = np.random.default_rng(d)
    n, k = 5, 6
    bits = np.array([2, 3, 8, 1, 6], np.uint8)
    p = rng.uniform(0.05, 0.4, n)
    rp, ci, a, w = _codes.cyclic_code(p, bits, k, 3, 512)
    G_host = (rng.standard_normal((k, d)) * 10.0 ** rng.uniform(-2, 2, (k, 1))).astype(np.float32)
    oc, osc, ost, _ = orp.encode_quantize_global(rp, ci, a, bits, 31, 7, G_host)
    off = orp.worker_word_offsets(d, bits)
    flags = agc.AGC_FLAG_ALLOW_1BIT | (agc.AGC_FLAG_FORCE_DIRECT if direct else 0)
    parts = []
    for r in range(shards):
        lo, hi = sharding.power_of_two_range(d, r, shards)
        assert hi > lo
        ses = Session(n, k, hi - lo, rp, ci, a, w, p, bits, bucket=0, seed=31, flags=flags)
        ses.set_first_block(lo // 512)
        ld = (hi - lo + 3) // 4 * 4
        Gd = torch.zeros((k, ld), dtype=torch.float32, device="cuda")
        Gd[:, :hi - lo] = torch.from_numpy(G_host[:, lo:hi])
        sums = torch.empty(n, dtype=torch.float32, device="cuda")
        agc.agc_encode_norm_sums(ses.plan, Gd, ld, sums)
        parts.append(dict(lo=lo, hi=hi, ses=ses, G=Gd, ld=ld, sums=sums))
    if shards > 1:
        with pytest.raises(agc.AgcError):
            parts[1]["ses"].encode(parts[1]["G"], 7)
    torch.cuda.synchronize()
    whole = agc.agc_combine_norm_sums(np.stack([pt["sums"].cpu().numpy() for pt in parts]))
    assert (whole.view(np.uint32) == orp.global_sumsq(rp, ci, a, G_host).view(np.uint32)).all()
    whole_dev = torch.from_numpy(whole).cuda()
    for pt in parts:
        ses = pt["ses"]
        ses.codes.fill_(-1)
        agc.agc_encode_quantize_with_norms(ses.plan, pt["G"], pt["ld"], 7, whole_dev, ses.codes, ses.scales, ses.status)
        torch.cuda.synchronize()
        assert int(ses.status.item()) == 0 and ost == 0
        assert (ses.scales.cpu().numpy().view(np.uint32) == osc.view(np.uint32)).all()
        got = ses.codes_host()
        roff = orp.worker_word_offsets(pt["hi"] - pt["lo"], bits)
        q0, nq = pt["lo"] // 512, (pt["hi"] - pt["lo"] + 511) // 512
        for i in range(n):
            b = int(bits[i])
            want = oc[off[i] + q0 * 16 * b: off[i] + (q0 + nq) * 16 * b]
            assert (got[roff[i]:roff[i + 1]] == want).all(), (pt["lo"], i)
        ses.close()


def test_config5_shape_one_bit_workers_and_64_realisations(agc, torch):
    """cfg5's structure at a size the oracle finishes: n=k=100, s=5, Student-t(3) values,
    bits 1..8, 64 realisations decoded per encode with the update fused."""
    wl = cfgs.config5(d=40_000 + 13)
    code = _codes.cyclic_code(wl.p, wl.bits, wl.k, wl.s, 512)
    G = cfgs.partials_numpy(wl, 0)
    masks = cfgs.straggler_masks(wl, rounds=1)[0]
    rng = np.random.default_rng(1)
    lr = rng.uniform(1e-4, 1e-3, wl.realizations).astype(np.float32)
    beta0 = rng.standard_normal(wl.d).astype(np.float32)
    out, ref = run_both(agc, torch, G, code, wl.p, wl.bits, 512, wl.seed, 0, masks, lr=lr, beta0=beta0)
    assert_exact(out, ref)
    assert (out["beta_seq"].view(np.uint32) == ref["beta"].view(np.uint32)).all()
    rel = np.abs(out["beta_fused"] - ref["beta"]).max() / np.abs(ref["beta"]).max()
    assert rel <= 1e-5


@pytest.mark.parametrize("builder", ["bench", "oracle"])
def test_config3_full_size_sampled_blocks(agc, torch, builder):
    """The benchmark's own configuration (d = 25,557,032, bits from the allocator, bucket 512,
    the launch shape bench.py times): pack blocks sampled across the vector - first, last
    (ragged), segment boundaries, random ones - are recomputed one by one by the oracle from
    the same inputs and compared bit for bit: codes, scales, decode and fused update.
    builder = bench: the very bits and weights bench.py times (the library's Algorithm 1 and
    its solve on the cyclic support, zero coefficients dropped); oracle: bits from the
    oracle's Algorithm 1 and the column-normalised weights (all s entries per worker)."""
    from paper_2605_15890_b200.session import Session
    wl = cfgs.config3()
    B = 512
    if builder == "bench":
        import bench
        (rp, ci, a, w), bits = bench.build_code(agc, wl, B, "cyclic")
        assert len(ci) < wl.n * wl.s           # the solve drove some coefficients to zero
    else:
        bits, _ = od.bit_allocate_low_complexity(wl.p, wl.z_tot, B, b_max=8)
        bits = np.asarray(bits, np.uint8)
        rp, ci, a, w = _codes.cyclic_code(wl.p, bits, wl.k, wl.s, B)
    ses = Session(wl.n, wl.k, wl.d, rp, ci, a, w, wl.p, bits, bucket=B, seed=wl.seed)
    assert ses.uses_tma
    ld = (wl.d + 3) // 4 * 4
    G = cfgs.partials_torch(wl, "cuda:0", ld=ld)
    mask = cfgs.straggler_masks(wl, rounds=1)[0]
    m_dev = torch.from_numpy(mask).cuda()
    ghat = torch.empty((1, wl.d), dtype=torch.float32, device="cuda")
    gen = torch.Generator(device="cuda")
    gen.manual_seed(77)
    beta0 = torch.empty(wl.d, dtype=torch.float32, device="cuda").normal_(generator=gen)
    beta = beta0.clone()
    lr = np.array([0.05], np.float32)
    rnd = 11
    ses.encode(G, rnd)
    ses.decode(m_dev, lr=lr, ghat=ghat, beta=beta)
    torch.cuda.synchronize()
    assert int(ses.status.item()) == 0
    nblk = (wl.d + 511) // 512
    starts, _, _ = cfgs.segment_table(wl)
    rng = np.random.default_rng(3)
    sample = {0, 1, nblk - 2, nblk - 1} | {int(s_) // 512 for s_ in starts[1:40]} | \
        {int(x) for x in rng.integers(0, nblk, 200)}
    off = orp.worker_word_offsets(wl.d, bits)
    codes = ses.codes
    for q in sorted(sample):
        m0, m1 = q * 512, min((q + 1) * 512, wl.d)
        blk = np.zeros((wl.k, 512), np.float32)
        blk[:, :m1 - m0] = G[:, m0:m1].cpu().numpy()
        oc, osc, st, _ = orp.encode_block(rp, ci, a, bits, B, wl.seed, rnd, q, blk)
        assert st == 0
        wb = 0
        for i in range(wl.n):
            b = int(bits[i])
            lo = int(off[i]) + q * 16 * b
            got = codes[lo:lo + 16 * b].cpu().numpy().view(np.uint32)
            assert (got == oc[wb:wb + 16 * b]).all(), (q, i)
            wb += 16 * b
        got_s = ses.scales.view(wl.n, -1)[:, q].cpu().numpy()
        assert (got_s.view(np.uint32) == osc[:, 0].view(np.uint32)).all(), q
        og = orp.decode_block(bits, B, w, mask[0], oc, osc)
        gg = ghat[0, m0:m1].cpu().numpy()
        assert (gg.view(np.uint32) == og[:m1 - m0].view(np.uint32)).all(), q
        ob = np.float32(beta0[m0:m1].cpu().numpy())
        want_b = (ob.astype(np.float64) - np.float64(lr[0]) * og[:m1 - m0].astype(np.float64))
        # fused update is one fp32 fma: compare against the correctly rounded value
        assert (beta[m0:m1].cpu().numpy() == want_b.astype(np.float32)).all(), q
    ses.close()


def test_encoder_division_is_correctly_rounded_everywhere(agc):
    """The encoder's branch-free L 2^15 / S against the IEEE quotient for all eight
    numerators and every float S in [2^-63, 2^64)."""
    assert agc.agc_selftest_division() == 0


def test_encoder_square_root_is_correctly_rounded_everywhere(agc):
    """The encoder's branch-free square root against the IEEE one for every normal float."""
    assert agc.agc_selftest_sqrt() == 0


def test_config4_least_squares_descent_in_lock_step(agc, torch):
    """cfg4: least squares with 2^20 rows x 4,096 features split into 64 partitions, n = 64
    workers, s = 2, bits 2..6; 500 rounds of gradient descent with the fused decode + update.
    The partial gradients X_j^T (X_j w - y_j) come from torch (harness only). Every round the
    oracle repeats encode, decode and update from the SAME partials and parameters: the
    parameters after the round must agree bit for bit, so the two loss curves coincide; the
    loss itself must fall from its start towards the noise floor."""
    from paper_2605_15890_b200.session import Session
    wl = cfgs.config4()
    rows = wl.extra["rows"]
    free, _ = torch.cuda.mem_get_info()
    while rows * wl.d * 4 * 1.3 > free and rows > 65536:
        rows //= 2                      # smaller boxes: fewer rows, same coding path
    X, y, _ = cfgs.least_squares_problem(wl, "cuda:0", rows=rows)
    B = 512
    rp, ci, a, w = _codes.cyclic_code(wl.p, wl.bits, wl.k, wl.s, B)
    ses = Session(wl.n, wl.k, wl.d, rp, ci, a, w, wl.p, wl.bits, bucket=B, seed=wl.seed)
    masks = cfgs.straggler_masks(wl)
    m_dev = torch.from_numpy(masks).cuda()
    lr = np.array([0.5 / rows], np.float32)
    beta = torch.zeros(wl.d, dtype=torch.float32, device="cuda")
    Xb = X.view(wl.k, rows // wl.k, wl.d)
    losses = []
    for t in range(wl.rounds):
        r = X @ beta - y
        losses.append(0.5 * float((r.double() ** 2).sum()))
        G = torch.bmm(Xb.transpose(1, 2), r.view(wl.k, rows // wl.k, 1)).squeeze(2).contiguous()
        beta_before = beta.cpu().numpy()
        ses.encode(G, t)
        ses.decode(m_dev[t], lr=lr, beta=beta)
        G_host = G.cpu().numpy()
        oc, osc, st, _ = orp.encode_quantize(rp, ci, a, wl.bits, B, wl.seed, t, G_host)
        _, ob = orp.decode(wl.d, wl.bits, B, w, masks[t], oc, osc, lr=lr, beta=beta_before, want_ghat=False)
        got = beta.cpu().numpy()
        assert (got.view(np.uint32) == ob.view(np.uint32)).all(), f"round {t}"
    assert int(ses.status.item()) == 0
    ses.close()
    assert losses[-1] < 0.05 * losses[0]
    assert min(losses) == min(losses[-50:]) or losses[-1] < 1.5 * min(losses)


@pytest.mark.parametrize("B,d", [(512, 5000), (128, 70_001)])
def test_two_track_decode_and_adam_steps(agc, torch, B, d):
    """Sec. V-E: the same messages decoded with w (first moment) and with v* (second moment)
    in one pass, fused with the Adam step; three rounds against the oracle, bit for bit."""
    from paper_2605_15890_b200.session import Session
    rng = np.random.default_rng(B + d)
    n = k = 12
    bits = rng.integers(1, 9, n).astype(np.uint8)
    p = rng.uniform(0.05, 0.5, n)
    rp, ci, a, w = _codes.cyclic_code(p, bits, k, 3, B)
    v = agc.agc_two_track_vector(n, k, p, bits, float(B), rp, a)
    ses = Session(n, k, d, rp, ci, a, w, p, bits, bucket=B, seed=5, flags=agc.AGC_FLAG_ALLOW_1BIT)
    ld = (d + 3) // 4 * 4
    lr, b1, b2, eps = 1e-2, 0.9, 0.999, 1e-8
    beta0 = rng.standard_normal(d).astype(np.float32)
    beta = torch.from_numpy(beta0.copy()).cuda()
    m = torch.zeros(d, dtype=torch.float32, device="cuda")
    u = torch.zeros(d, dtype=torch.float32, device="cuda")
    gw = torch.empty(d, dtype=torch.float32, device="cuda")
    gv = torch.empty(d, dtype=torch.float32, device="cuda")
    ob, om, ou = beta0.copy(), np.zeros(d, np.float32), np.zeros(d, np.float32)
    for t in range(1, 4):
        G_host = (rng.standard_normal((k, d)) * 10.0 ** rng.uniform(-2, 1)).astype(np.float32)
        G = torch.zeros((k, ld), dtype=torch.float32, device="cuda")
        G[:, :d] = torch.from_numpy(G_host)
        mask = (rng.random(n) >= p).astype(np.uint8)
        ses.encode(G, t)
        agc.agc_decode_two_track(ses.plan, ses.codes, ses.scales, torch.from_numpy(mask).cuda(), v, gw, gv, beta, m, u,
                                 adam=(lr, b1, b2, eps, t), status_dev=ses.status)
        torch.cuda.synchronize()
        oc, osc, _, _ = orp.encode_quantize(rp, ci, a, bits, B, 5, t, G_host)
        ogw, _ = orp.decode(d, bits, B, w, mask[None], oc, osc)
        ogv, _ = orp.decode(d, bits, B, v, mask[None], oc, osc)
        ob, om, ou = orp.adam_two_track(ogw[0], ogv[0], lr, b1, b2, eps, t, ob, om, ou)
        assert (gw.cpu().numpy().view(np.uint32) == ogw[0].view(np.uint32)).all()
        assert (gv.cpu().numpy().view(np.uint32) == ogv[0].view(np.uint32)).all()
        assert (m.cpu().numpy().view(np.uint32) == om.view(np.uint32)).all()
        assert (u.cpu().numpy().view(np.uint32) == ou.view(np.uint32)).all()
        assert (beta.cpu().numpy().view(np.uint32) == ob.view(np.uint32)).all()
    assert int(ses.status.item()) == 0
    ses.close()


@pytest.mark.parametrize("d,direct", [(300, False), (5000, False), (5000, True), (600_001, False)])
def test_global_norm_two_pass_encode_and_decode(agc, torch, d, direct):
    """The paper's main formulation (one l2 norm per worker, bucket = 0): two-pass encode
    against the oracle's global-norm encoder, bit for bit, then decode and fused update. The
    largest case spans several 1024-block chunks of the norm reduction; one worker is zero."""
    from paper_2605_15890_b200.session import Session
    rng = np.random.default_rng(d)
    n = k = 6
    bits = np.array([1, 2, 3, 4, 6, 8], np.uint8)
    p = rng.uniform(0.05, 0.4, n)
    rp, ci, a, w = _codes.identity_code(n)
    w = (1.0 / (1.0 - p)).astype(np.float32)
    G_host = (rng.standard_normal((k, d)) * 10.0 ** rng.uniform(-2, 2, (k, 1))).astype(np.float32)
    G_host[3] = 0.0
    flags = agc.AGC_FLAG_ALLOW_1BIT | (agc.AGC_FLAG_FORCE_DIRECT if direct else 0)
    ses = Session(n, k, d, rp, ci, a, w, p, bits, bucket=0, seed=17, flags=flags)
    ld = (d + 3) // 4 * 4
    G = torch.zeros((k, ld), dtype=torch.float32, device="cuda")
    G[:, :d] = torch.from_numpy(G_host)
    ses.codes.fill_(-1)
    ses.scales.fill_(-1.0)
    mask = np.array([1, 1, 0, 1, 1, 1], np.uint8)
    lr = np.array([0.01], np.float32)
    beta0 = rng.standard_normal(d).astype(np.float32)
    beta = torch.from_numpy(beta0.copy()).cuda()
    ghat = torch.empty((1, d), dtype=torch.float32, device="cuda")
    for rnd in (0, 1):
        ses.encode(G, rnd)
    ses.decode(torch.from_numpy(mask).cuda(), lr=lr, ghat=ghat, beta=beta)
    torch.cuda.synchronize()
    assert int(ses.status.item()) == 0 and ses.uses_tma == (not direct)
    oc, osc, st, _ = orp.encode_quantize_global(rp, ci, a, bits, 17, 1, G_host)
    assert st == 0 and osc[3] == 0.0
    assert (ses.scales_host()[:, 0].view(np.uint32) == osc.view(np.uint32)).all()
    bad = np.nonzero(ses.codes_host() != oc)[0]
    assert bad.size == 0, f"{bad.size} code words differ, first at {bad[:5]}"
    og, ob = orp.decode(d, bits, 512, w, mask[None], oc, orp.expand_global_scales(osc, d), lr=lr, beta=beta0)
    assert (ghat.cpu().numpy().view(np.uint32) == og.view(np.uint32)).all()
    assert (beta.cpu().numpy().view(np.uint32) == ob.view(np.uint32)).all()
    if not direct:
        # the two-track decoder reads the same single scale per worker
        v2 = (0.5 * w).astype(np.float32)
        gw = torch.empty(d, dtype=torch.float32, device="cuda")
        gv = torch.empty(d, dtype=torch.float32, device="cuda")
        agc.agc_decode_two_track(ses.plan, ses.codes, ses.scales, torch.from_numpy(mask).cuda(), v2, gw, gv,
                                 status_dev=ses.status)
        ogv, _ = orp.decode(d, bits, 512, v2, mask[None], oc, orp.expand_global_scales(osc, d))
        assert (gw.cpu().numpy().view(np.uint32) == og[0].view(np.uint32)).all()
        assert (gv.cpu().numpy().view(np.uint32) == ogv[0].view(np.uint32)).all()
    ses.close()


@pytest.mark.parametrize("R,B,d,n", [(8, 512, 5000, 12), (16, 256, 70_001, 9), (17, 128, 1300, 40), (33, 512, 513, 70),
                                     (64, 512, 200_000, 20), (65, 256, 4097, 33), (130, 128, 3, 5), (48, 0, 40_000, 6),
                                     (9, 512, 1500, 300), (8, 256, 600, 2048)])
def test_g_hat_of_many_realisations_in_one_pass(agc, torch, R, B, d, n):
    """From 8 realisations on, g_hat of every realisation comes from one pass over the messages
    (chunks of 64 realisations). Every row must equal the oracle's realisation-by-realisation
    decode bit for bit; rows with no survivor and workers nobody received are in the masks."""
    from paper_2605_15890_b200.session import Session
    rng = np.random.default_rng(R * 1000 + n)
    k = n
    bits = rng.integers(1, 9, n).astype(np.uint8)
    p = rng.uniform(0.05, 0.6, n)
    masks = (rng.random((R, n)) >= p).astype(np.uint8)
    masks[R // 2] = 0                       # a realisation in which every worker straggles
    masks[:, n // 3] = 0                    # a worker that no realisation receives
    masks[R - 1] = 1
    masks[R - 1, n // 3] = 0
    G = (rng.standard_normal((k, d)) * 10.0 ** rng.uniform(-3, 2, (k, 1))).astype(np.float32)
    if B:
        code = _codes.cyclic_code(p, bits, k, min(3, k), B)
        lr = rng.uniform(1e-3, 1e-1, R).astype(np.float32)
        beta0 = rng.standard_normal(d).astype(np.float32)
        out, ref = run_both(agc, torch, G, code, p, bits, B, 4242, 9, masks, lr=lr, beta0=beta0)
        assert_exact(out, ref)
        # with the parameters as well: the R updates in order, from the stored rows
        assert (out["beta_seq"].view(np.uint32) == ref["beta"].view(np.uint32)).all()
        assert np.abs(out["beta_fused"] - ref["beta"]).max() / np.abs(ref["beta"]).max() <= 1e-5
        return
    rp, ci, a, w = _codes.identity_code(n)
    w = (1.0 / (1.0 - p)).astype(np.float32)
    ses = Session(n, k, d, rp, ci, a, w, p, bits, bucket=0, seed=17, flags=agc.AGC_FLAG_ALLOW_1BIT)
    Gd = torch.zeros((k, (d + 3) // 4 * 4), dtype=torch.float32, device="cuda")
    Gd[:, :d] = torch.from_numpy(G)
    ses.encode(Gd, 2)
    ghat = torch.full((R, d), -3.0, dtype=torch.float32, device="cuda")
    ses.decode(torch.from_numpy(masks).cuda(), ghat=ghat)
    torch.cuda.synchronize()
    oc, osc, st, _ = orp.encode_quantize_global(rp, ci, a, bits, 17, 2, G)
    og, _ = orp.decode(d, bits, 512, w, masks, oc, orp.expand_global_scales(osc, d))
    assert (ghat.cpu().numpy().view(np.uint32) == og.view(np.uint32)).all()
    ses.close()


@pytest.mark.parametrize("R,B,d,n", [(1, 512, 5000, 12), (20, 256, 70_001, 9), (64, 128, 200_000, 20), (70, 0, 40_000, 6)])
def test_residuals_of_many_realisations_without_storing_g_hat(agc, torch, R, B, d, n):
    """||g_hat^(r) - g||^2 for every realisation straight from the messages: against the oracle's
    g_hat rows (fp32, defining order), differences squared and summed in fp64 on the host. The
    library sums 128 coordinates in fp32 before it goes to fp64: 1e-6 relative."""
    from paper_2605_15890_b200.session import Session
    rng = np.random.default_rng(R * 77 + n)
    k = n
    bits = rng.integers(1, 9, n).astype(np.uint8)
    p = rng.uniform(0.05, 0.6, n)
    masks = (rng.random((R, n)) >= p).astype(np.uint8)
    masks[R // 2] = 0
    G = (rng.standard_normal((k, d)) * 10.0 ** rng.uniform(-2, 1, (k, 1))).astype(np.float32)
    g_ref = G.astype(np.float64).sum(0).astype(np.float32)
    if B:
        rp, ci, a, w = _codes.cyclic_code(p, bits, k, min(3, k), B)
    else:
        rp, ci, a, w = _codes.identity_code(n)
        w = (1.0 / (1.0 - p)).astype(np.float32)
    ses = Session(n, k, d, rp, ci, a, w, p, bits, bucket=B, seed=5, flags=agc.AGC_FLAG_ALLOW_1BIT)
    Gd = torch.zeros((k, (d + 3) // 4 * 4), dtype=torch.float32, device="cuda")
    Gd[:, :d] = torch.from_numpy(G)
    ses.encode(Gd, 3)
    got = ses.residuals(torch.from_numpy(masks).cuda(), torch.from_numpy(g_ref).cuda()).cpu().numpy()
    ses.close()
    if B:
        oc, osc, _, _ = orp.encode_quantize(rp, ci, a, bits, B, 5, 3, G, d=d)
        og, _ = orp.decode(d, bits, B, w, masks, oc, osc)
    else:
        oc, osc, _, _ = orp.encode_quantize_global(rp, ci, a, bits, 5, 3, G)
        og, _ = orp.decode(d, bits, 512, w, masks, oc, orp.expand_global_scales(osc, d))
    want = ((og.astype(np.float64) - g_ref.astype(np.float64)[None]) ** 2).sum(1)
    assert want[R // 2] == pytest.approx(float((g_ref.astype(np.float64) ** 2).sum()), rel=1e-12)   # nobody arrived
    assert np.abs(got - want).max() <= 1e-6 * want.max()
    assert (np.abs(got - want) <= 1e-6 * want).all()


@pytest.mark.parametrize("B,d,direct", [(1024, 300, False), (1024, 70_001, False), (2048, 5000, True), (2048, 600_001, False),
                                        (4096, 40_000, False), (4096, 4096 * 3 + 1, True)])
def test_buckets_of_several_pack_blocks(agc, torch, B, d, direct):
    """Buckets of 1024, 2048 and 4096 coordinates (2, 4, 8 pack blocks; two passes like the global
    norm): messages and scales against the oracle's grouped encoder bit for bit, then every
    decoder on them: single realisation with the fused update, nine realisations in one pass,
    the collapsed update and the two-track decode."""
    from paper_2605_15890_b200.session import Session
    rng = np.random.default_rng(B + d)
    n = k = 7
    bits = np.array([1, 2, 3, 4, 5, 6, 8], np.uint8)
    p = rng.uniform(0.05, 0.4, n)
    rp, ci, a, w = _codes.cyclic_code(p, bits, k, 3, 512)
    G_host = (rng.standard_normal((k, d)) * 10.0 ** rng.uniform(-2, 2, (k, 1))).astype(np.float32)
    if d > 3 * B:
        G_host[:, B:2 * B] = 0.0                       # a bucket that every worker sends as zeros
    flags = agc.AGC_FLAG_ALLOW_1BIT | (agc.AGC_FLAG_FORCE_DIRECT if direct else 0)
    ses = Session(n, k, d, rp, ci, a, w, p, bits, bucket=B, seed=17, flags=flags)
    ld = (d + 3) // 4 * 4
    G = torch.zeros((k, ld), dtype=torch.float32, device="cuda")
    G[:, :d] = torch.from_numpy(G_host)
    ses.codes.fill_(-1)
    ses.scales.fill_(-1.0)
    for rnd in (0, 4):
        ses.encode(G, rnd)
    torch.cuda.synchronize()
    assert int(ses.status.item()) == 0 and ses.uses_tma == (not direct)
    oc, osc, st, _ = orp.encode_quantize_grouped(rp, ci, a, bits, B, 17, 4, G_host)
    assert st == 0
    assert ses.scales_host().shape == osc.shape
    assert (ses.scales_host().view(np.uint32) == osc.view(np.uint32)).all()
    bad = np.nonzero(ses.codes_host() != oc)[0]
    assert bad.size == 0, f"{bad.size} code words differ, first at {bad[:5]}"
    if d > 3 * B:
        assert (osc[:, 1] == 0.0).all()
    per_block = orp.expand_grouped_scales(osc, d, B)
    R = 9
    masks = (rng.random((R, n)) >= p).astype(np.uint8)
    lr = rng.uniform(1e-3, 1e-1, R).astype(np.float32)
    beta0 = rng.standard_normal(d).astype(np.float32)
    og, ob = orp.decode(d, bits, 512, w, masks, oc, per_block, lr=lr, beta=beta0)
    m_dev = torch.from_numpy(masks).cuda()
    ghat = torch.full((R, d), -3.0, dtype=torch.float32, device="cuda")
    ses.decode(m_dev, ghat=ghat)                                     # nine realisations in one pass
    assert (ghat.cpu().numpy().view(np.uint32) == og.view(np.uint32)).all()
    g1 = torch.empty((1, d), dtype=torch.float32, device="cuda")
    b1 = torch.from_numpy(beta0.copy()).cuda()
    ses.decode(m_dev[:1], lr=lr[:1], ghat=g1, beta=b1)                # one realisation, fused update
    og1, ob1 = orp.decode(d, bits, 512, w, masks[:1], oc, per_block, lr=lr[:1], beta=beta0)
    assert (g1.cpu().numpy().view(np.uint32) == og1.view(np.uint32)).all()
    assert (b1.cpu().numpy().view(np.uint32) == ob1.view(np.uint32)).all()
    b2 = torch.from_numpy(beta0.copy()).cuda()
    ses.decode(m_dev, lr=lr, beta=b2)                                # collapsed update
    assert np.abs(b2.cpu().numpy() - ob).max() / np.abs(ob).max() <= 1e-5
    if not direct:
        v2 = (0.5 * w).astype(np.float32)
        gw = torch.empty(d, dtype=torch.float32, device="cuda")
        gv = torch.empty(d, dtype=torch.float32, device="cuda")
        agc.agc_decode_two_track(ses.plan, ses.codes, ses.scales, m_dev[0], v2, gw, gv, status_dev=ses.status)
        ogv, _ = orp.decode(d, bits, 512, v2, masks[:1], oc, per_block)
        assert (gw.cpu().numpy().view(np.uint32) == og[0].view(np.uint32)).all()
        assert (gv.cpu().numpy().view(np.uint32) == ogv[0].view(np.uint32)).all()
    torch.cuda.synchronize()
    assert int(ses.status.item()) == 0
    with pytest.raises(agc.AgcError) as e:       # a range of a longer vector starts at a bucket
        ses.set_first_block(B // 512 + 1)
    assert e.value.code == -1
    ses.set_first_block(3 * (B // 512))
    ses.close()


@pytest.mark.parametrize("kind", ["cyclic", "interval"])
def test_lemma1_bound_and_unbiasedness_measured_on_the_gpu(agc, torch, kind):
    """Lemma 1 as a measured experiment: 20 rounds x 64 straggler realisations through the CUDA
    path (fresh rounding each round, fresh Bernoulli masks each realisation). The mean of
    g_hat approaches sum_j g_j (unbiasedness, Eq. exp_g2_quant) and the mean squared error
    stays below C sum_i (1-p_i){p_i + phi(b_i)} w_i^2 (sum_j a_ij)^2 with ||g_j||^2 = C. With
    the paper's interval construction (the optimal structure of Theorem 1) that bound is
    Lemma 2's k^2 C / sum_i c_i^-1."""
    from paper_2605_15890_b200.session import Session
    rng = np.random.default_rng(31)
    n = k = 8
    d, B = 4096, 512
    bits = np.array([2, 3, 4, 6, 2, 5, 3, 4], np.uint8)
    p = rng.uniform(0.05, 0.4, n)
    if kind == "cyclic":
        rp, ci, a, w = _codes.cyclic_code(p, bits, k, 3, B)
    else:
        rp, ci, a, w = _codes.interval_code(p, bits, k, B)
    A = od.csr_to_dense(rp, ci, a.astype(np.float64), k)
    if kind == "interval":
        assert np.isclose(od.lemma1_bound(A, w.astype(np.float64), p, bits, B), od.lemma2_bound(p, bits, k, B), rtol=1e-5)
    G_host = rng.standard_normal((k, d)).astype(np.float32)
    G_host /= np.linalg.norm(G_host.astype(np.float64), axis=1, keepdims=True).astype(np.float32)   # C = 1
    g = G_host.astype(np.float64).sum(axis=0)
    ses = Session(n, k, d, rp, ci, a, w, p, bits, bucket=B, seed=77)
    G = torch.from_numpy(G_host).cuda()
    rounds, R = 20, 64
    ghat = torch.empty((R, d), dtype=torch.float32, device="cuda")
    mean = np.zeros(d)
    mse = 0.0
    for t in range(rounds):
        masks = (rng.random((R, n)) >= p).astype(np.uint8)
        ses.encode(G, t)
        ses.decode(torch.from_numpy(masks).cuda(), ghat=ghat)
        gh = ghat.cpu().numpy().astype(np.float64)
        mean += gh.sum(axis=0)
        mse += ((gh - g) ** 2).sum()
    N = rounds * R
    mean /= N
    mse /= N
    bound = od.lemma1_bound(A, w.astype(np.float64), p, bits, B, C=1.0)
    assert mse <= bound * 1.05
    assert mse >= 0.05 * bound                 # the experiment is not vacuous
    # unbiasedness: the realisations of one round share their rounding noise, so the mean has
    # at least `rounds` independent terms: its error is below 3 sqrt(mse / rounds) and far
    # below the error of a single estimate
    assert np.linalg.norm(mean - g) <= 3.0 * np.sqrt(mse / rounds)
    assert np.linalg.norm(mean - g) <= 0.3 * np.sqrt(mse)
    ses.close()


def test_lemma1_bound_at_full_size_from_residuals(agc, torch):
    """Lemma 1 measured at the size of the third configuration (n = k = 32, cyclic s = 4,
    d = 25,557,032): 3 rounds x 64 straggler realisations, squared residuals reduced on the
    device (no g_hat is stored). Their mean stays below the bound
    C sum_i (1-p_i){p_i + phi(b_i)} w_i^2 (sum_j a_ij)^2 (||g_j||^2 = C = 1), which is loose for
    nearly orthogonal g_j, and not below the part of the error that stragglers alone cause,
    sum_i p_i (1-p_i) w_i^2 ||f_i||^2 (the estimate is unbiased and the workers independent, so
    the rounding noise only adds to it)."""
    from paper_2605_15890_b200.session import Session
    wl = cfgs.config3()
    B = 512
    bits = np.array([8] * 10 + [6] + [2] * 21, np.uint8)
    rp, ci, a, w = _codes.cyclic_code(wl.p, bits, wl.k, wl.s, B)
    A = od.csr_to_dense(rp, ci, a.astype(np.float64), wl.k)
    gen = torch.Generator(device="cuda").manual_seed(5)
    G = torch.randn((wl.k, wl.d), generator=gen, device="cuda", dtype=torch.float32)
    G /= G.double().pow(2).sum(1, keepdim=True).sqrt().float()                     # C = 1
    g_ref = torch.zeros(wl.d, dtype=torch.float64, device="cuda")
    for j in range(wl.k):
        g_ref += G[j].double()
    g_ref = g_ref.float()
    ses = Session(wl.n, wl.k, wl.d, rp, ci, a, w, wl.p, bits, bucket=B, seed=11)
    rng = np.random.default_rng(12)
    rounds, R = 3, 64
    total = 0.0
    for t in range(rounds):
        masks = (rng.random((R, wl.n)) >= wl.p).astype(np.uint8)
        ses.encode(G, t)
        total += float(ses.residuals(torch.from_numpy(masks).cuda(), g_ref).sum().item())
    assert int(ses.status.item()) == 0
    mse = total / (rounds * R)
    bound = od.lemma1_bound(A, w.astype(np.float64), wl.p, bits, B, C=1.0)
    assert mse <= 1.05 * bound
    straggler_part = 0.0
    for i in range(wl.n):
        f = torch.zeros(wl.d, dtype=torch.float32, device="cuda")
        for e in range(rp[i], rp[i + 1]):
            f += float(a[e]) * G[int(ci[e])]
        straggler_part += float(wl.p[i] * (1 - wl.p[i])) * float(w[i]) ** 2 * float(f.double().pow(2).sum().item())
    assert straggler_part > 0 and mse >= 0.6 * straggler_part    # 192 realisations: the sample mean is within tens of per cent
    ses.close()


@pytest.mark.parametrize("n,d,B", [(4, 10_000, 512), (64, 4096, 256), (6, 40_000, 0)])
def test_rounds_captured_in_a_cuda_graph_replay_bit_for_bit(agc, torch, n, d, B):
    """Small problems are bound by launch latency, so a caller may record several rounds
    (encode + fused update each) in a CUDA graph: the entry points allocate nothing, copy nothing
    from the host for one realisation and synchronise nothing. A replay must give the bits of the
    same calls made one by one."""
    from paper_2605_15890_b200.session import Session
    rng = np.random.default_rng(n + d)
    k = n
    bits = rng.integers(2, 9, n).astype(np.uint8)
    p = rng.uniform(0.05, 0.4, n)
    if B:
        rp, ci, a, w = _codes.cyclic_code(p, bits, k, 2, B)
    else:
        rp, ci, a, w = _codes.identity_code(n)
        w = (1.0 / (1.0 - p)).astype(np.float32)
    ses = Session(n, k, d, rp, ci, a, w, p, bits, bucket=B, seed=3)
    G = torch.from_numpy(rng.standard_normal((k, d)).astype(np.float32)).cuda()
    mask = torch.from_numpy((rng.random(n) >= p).astype(np.uint8)).cuda()
    lr = np.array([1e-2], np.float32)
    beta0 = torch.from_numpy(rng.standard_normal(d).astype(np.float32)).cuda()
    rounds = 4

    def run_rounds(beta):
        for t in range(rounds):
            ses.encode(G, t)
            ses.decode(mask, lr=lr, beta=beta)

    eager = beta0.clone()
    run_rounds(eager)
    codes_eager = ses.codes.clone()
    torch.cuda.synchronize()
    beta = beta0.clone()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        run_rounds(beta)                      # warm-up on the capture stream
    torch.cuda.current_stream().wait_stream(side)
    beta.copy_(beta0)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        run_rounds(beta)
    beta.copy_(beta0)
    ses.codes.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(beta.view(torch.int32), eager.view(torch.int32))
    assert torch.equal(ses.codes, codes_eager)
    run_rounds(eager)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(beta.view(torch.int32), eager.view(torch.int32))
    assert int(ses.status.item()) == 0
    ses.close()


def test_decode_entry_points_reject_bad_arguments(agc, torch):
    """Error codes instead of launches: missing buffers, R out of range, misaligned messages, and
    the entry points that need the staged decoder on a plan that was told not to use it."""
    from paper_2605_15890_b200.session import Session
    n = k = 4
    d = 3000
    bits = np.array([2, 3, 4, 8], np.uint8)
    p = np.array([0.1, 0.2, 0.3, 0.4])
    rp, ci, a, w = _codes.cyclic_code(p, bits, k, 2, 512)
    ses = Session(n, k, d, rp, ci, a, w, p, bits, bucket=512, seed=1)
    direct = Session(n, k, d, rp, ci, a, w, p, bits, bucket=512, seed=1, flags=agc.AGC_FLAG_FORCE_DIRECT)
    mask = torch.ones(n, dtype=torch.uint8, device="cuda")
    ghat = torch.zeros(d, dtype=torch.float32, device="cuda")
    sq = torch.zeros(4, dtype=torch.float64, device="cuda")

    def code_of(fn):
        with pytest.raises(agc.AgcError) as e:
            fn()
        return e.value.code

    ERR_ARG, ERR_ALIGN, ERR_STATE = -1, -4, -7
    assert code_of(lambda: agc.agc_decode(ses.plan, ses.codes, ses.scales, mask, 1)) == ERR_ARG            # no output
    assert code_of(lambda: agc.agc_decode(ses.plan, ses.codes, ses.scales, mask, 0, None, ghat)) == ERR_ARG
    assert code_of(lambda: agc.agc_decode(ses.plan, ses.codes, ses.scales, mask, 1, None, None, ghat)) == ERR_ARG  # beta without lr
    assert code_of(lambda: agc.agc_decode(ses.plan, ses.codes, ses.scales, mask, 5000, None, ghat)) == ERR_STATE
    off = ses.codes.view(torch.uint8)[4:]
    assert code_of(lambda: agc.agc_decode(ses.plan, off, ses.scales, mask, 1, None, ghat)) == ERR_ALIGN
    assert code_of(lambda: agc.agc_decode_residuals(ses.plan, ses.codes, ses.scales, mask, 0, ghat, sq)) == ERR_ARG
    assert code_of(lambda: agc.agc_decode_residuals(ses.plan, ses.codes, ses.scales, mask, 1, None, sq)) == ERR_ARG
    assert code_of(lambda: agc.agc_decode_residuals(ses.plan, off, ses.scales, mask, 1, ghat, sq)) == ERR_ALIGN
    assert code_of(lambda: agc.agc_decode_residuals(direct.plan, direct.codes, direct.scales, mask, 1, ghat, sq)) == ERR_STATE
    assert code_of(lambda: agc.agc_decode_two_track(direct.plan, direct.codes, direct.scales, mask,
                                                    np.ones(n, np.float32), ghat)) == ERR_STATE
    torch.cuda.synchronize()
    ses.close()
    direct.close()


@pytest.mark.parametrize("d,B", [(1, 128), (513, 256), (70_001, 512), (40_000, 0)])
def test_kernels_write_nothing_outside_their_outputs(agc, torch, d, B):
    """Guard words before and after every output buffer (messages, scales, g_hat, parameters,
    Adam state) must survive encode, decode, the collapsed update and the two-track step."""
    rng = np.random.default_rng(d + B)
    n = k = 9
    bits = rng.integers(1, 9, n).astype(np.uint8)
    p = rng.uniform(0.05, 0.5, n)
    rp, ci, a, w = _codes.cyclic_code(p, bits, k, 3, B if B else 512)
    plan = agc.agc_plan_create(n, k, d, rp, ci, a, w, p, bits, B, 3, agc.AGC_FLAG_ALLOW_1BIT)
    pad = 1024                                             # floats / words of guard on each side
    def guarded(nelem, dtype, fill):
        buf = torch.full((nelem + 2 * pad,), fill, dtype=dtype, device="cuda")
        return buf, buf[pad:pad + nelem]
    GUARD_I, GUARD_F = 0x5A5A5A5A, -12345.5
    codes_all, codes = guarded(agc.agc_codes_bytes(plan) // 4, torch.int32, GUARD_I)
    scales_all, scales = guarded(agc.agc_scales_bytes(plan) // 4, torch.float32, GUARD_F)
    outs = {name: guarded(R_ * d, torch.float32, GUARD_F) for name, R_ in
            [("ghat", 3), ("beta", 1), ("gw", 1), ("gv", 1), ("m", 1), ("u", 1)]}
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ld = (d + 3) // 4 * 4
    G = torch.from_numpy(rng.standard_normal((k, ld)).astype(np.float32)).cuda()
    masks = torch.from_numpy((rng.random((3, n)) > 0.3).astype(np.uint8)).cuda()
    lr = np.array([1e-3, 2e-3, 3e-3], np.float32)
    for name in ("beta", "m", "u"):
        outs[name][1].zero_()
    agc.agc_encode_quantize(plan, G, ld, 4, codes, scales, status)
    agc.agc_decode(plan, codes, scales, masks, 3, lr, outs["ghat"][1], outs["beta"][1], status)
    agc.agc_decode(plan, codes, scales, masks, 3, lr, None, outs["beta"][1], status)          # collapsed
    agc.agc_decode_two_track(plan, codes, scales, masks[0], w, outs["gw"][1], outs["gv"][1], outs["beta"][1],
                             outs["m"][1], outs["u"][1], adam=(1e-3, 0.9, 0.999, 1e-8, 1), status_dev=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    def check(all_, fill):
        assert bool((all_[:pad] == fill).all()) and bool((all_[-pad:] == fill).all())
    check(codes_all, GUARD_I)
    check(scales_all, GUARD_F)
    for name, (all_, inner) in outs.items():
        check(all_, GUARD_F)
        assert not bool((inner == GUARD_F).any()), name      # every output element was written
    assert not bool((scales == GUARD_F).any())
    agc.agc_plan_destroy(plan)


def test_config5_full_size_sampled_blocks(agc, torch):
    """cfg5 at its full size (n = k = 100, s = 5, d = 10^8 Student-t(3) values, bits 1..8, 64
    straggler realisations per encode, 40 GB of partial gradients, messages beyond 4 GiB):
    sampled pack blocks - first, last, around the 4 GiB byte offset of the message buffer,
    random ones - are recomputed by the oracle from the same inputs. Codes and scales bit for
    bit; the collapsed 64-realisation update within 1e-5 of the sequential definition."""
    from paper_2605_15890_b200.session import Session
    free, _ = torch.cuda.mem_get_info()
    if free < 60e9:
        pytest.skip("needs about 50 GB of device memory")
    wl = cfgs.config5()
    B = 512
    rp, ci, a, w = _codes.cyclic_code(wl.p, wl.bits, wl.k, wl.s, B)
    ses = Session(wl.n, wl.k, wl.d, rp, ci, a, w, wl.p, wl.bits, bucket=B, seed=wl.seed, flags=agc.AGC_FLAG_ALLOW_1BIT)
    G = cfgs.partials_torch(wl, "cuda:0", ld=wl.d)
    masks = cfgs.straggler_masks(wl, rounds=1)[0]                      # 64 x 100
    lr = np.full(wl.realizations, 1e-3, np.float32)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(5)
    beta0 = torch.empty(wl.d, dtype=torch.float32, device="cuda").normal_(generator=gen)
    beta = beta0.clone()
    ses.encode(G, 3)
    ses.decode(torch.from_numpy(masks).cuda(), lr=lr, beta=beta)
    torch.cuda.synchronize()
    assert int(ses.status.item()) & 4 == 0
    nblk = (wl.d + 511) // 512
    off = orp.worker_word_offsets(wl.d, wl.bits)
    assert int(off[-1]) * 4 > (1 << 32)
    # blocks whose words straddle the 4 GiB byte offset for some worker
    cross = int(np.searchsorted(off * 4, 1 << 32) - 1)
    q_cross = int(((1 << 32) // 4 - int(off[cross])) // (16 * int(wl.bits[cross])))
    rng = np.random.default_rng(9)
    sample = {0, 1, nblk - 2, nblk - 1, max(0, q_cross - 1), min(nblk - 1, q_cross), min(nblk - 1, q_cross + 1)} | \
        {int(x) for x in rng.integers(0, nblk, 40)}
    for q in sorted(sample):
        m0, m1 = q * 512, min((q + 1) * 512, wl.d)
        blk = np.zeros((wl.k, 512), np.float32)
        blk[:, :m1 - m0] = G[:, m0:m1].cpu().numpy()
        oc, osc, st, _ = orp.encode_block(rp, ci, a, wl.bits, B, wl.seed, 3, q, blk)
        wb = 0
        for i in range(wl.n):
            b = int(wl.bits[i])
            lo = int(off[i]) + q * 16 * b
            got = ses.codes[lo:lo + 16 * b].cpu().numpy().view(np.uint32)
            assert (got == oc[wb:wb + 16 * b]).all(), (q, i)
            wb += 16 * b
        got_s = ses.scales.view(wl.n, -1)[:, q].cpu().numpy()
        assert (got_s.view(np.uint32) == osc[:, 0].view(np.uint32)).all(), q
        want = beta0[m0:m1].cpu().numpy().astype(np.float32)
        for r in range(wl.realizations):
            og = orp.decode_block(wl.bits, B, w, masks[r], oc, osc)
            want = (want.astype(np.float64) - np.float64(lr[r]) * og[:m1 - m0].astype(np.float64)).astype(np.float32)
        got_b = beta[m0:m1].cpu().numpy()
        assert np.abs(got_b - want).max() <= 1e-5 * max(1.0, np.abs(want).max()), q
    ses.close()


@pytest.mark.parametrize("B", [0, 256])
def test_encode_from_separate_row_buffers(agc, torch, B):
    """Partial gradients in k separate device buffers (an array of row pointers): the messages
    must be those of the contiguous call, bit for bit."""
    from paper_2605_15890_b200.session import Session
    rng = np.random.default_rng(44)
    n = k = 7
    d = 9000
    bits = rng.integers(1, 9, n).astype(np.uint8)
    p = rng.uniform(0.05, 0.5, n)
    rp, ci, a, w = _codes.cyclic_code(p, bits, k, 3, B if B else 512)
    ses = Session(n, k, d, rp, ci, a, w, p, bits, bucket=B, seed=8, flags=agc.AGC_FLAG_ALLOW_1BIT)
    G_host = rng.standard_normal((k, d)).astype(np.float32)
    G = torch.from_numpy(G_host).cuda()
    ses.encode(G, 6)
    want_codes, want_scales = ses.codes.clone(), ses.scales.clone()
    # separate allocations; every other row starts 4 bytes into its buffer (not 16-byte aligned)
    bufs = [torch.zeros(d + 4, dtype=torch.float32, device="cuda") for _ in range(k)]
    rows = [bufs[j][(j & 1):(j & 1) + d] for j in range(k)]
    for j in range(k):
        rows[j].copy_(torch.from_numpy(G_host[j]))
    ptrs = torch.tensor([r.data_ptr() for r in rows], dtype=torch.int64, device="cuda")
    ses.codes.fill_(-1)
    ses.scales.fill_(-1.0)
    agc.agc_encode_quantize_rows(ses.plan, ptrs, 6, ses.codes, ses.scales, ses.status)
    torch.cuda.synchronize()
    assert bool((ses.codes == want_codes).all()) and bool((ses.scales.view(torch.int32) == want_scales.view(torch.int32)).all())
    assert int(ses.status.item()) == 0
    ses.close()


def test_two_live_plans_of_different_shapes_alternate(agc, torch):
    """Plans of different worker counts and support widths need different amounts of dynamic
    shared memory from the same kernels; the second plan's creation must not lower the
    limit the first one launches with. Encode and decode alternate between the two, each
    checked against the oracle."""
    from paper_2605_15890_b200.session import Session
    rng = np.random.default_rng(77)
    shapes = [(96, 96, 5, 20_000), (5, 5, 2, 20_000)]       # (n, k, s, d): large tables first, small second
    plans = []
    for n, k, s, d in shapes:
        bits = rng.integers(2, 9, n).astype(np.uint8)
        p = rng.uniform(0.05, 0.4, n)
        code = _codes.cyclic_code(p, bits, k, s, 512)
        G = rng.standard_normal((k, d)).astype(np.float32)
        mask = (rng.random((1, n)) > 0.2).astype(np.uint8)
        plans.append(dict(n=n, k=k, d=d, bits=bits, p=p, code=code, G=G, mask=mask))
    for pl in plans:     # both created before any launch
        rp, ci, a, w = pl["code"]
        pl["ses"] = Session(pl["n"], pl["k"], pl["d"], rp, ci, a, w, pl["p"], pl["bits"], bucket=512, seed=9)
        pl["Gd"] = torch.from_numpy(pl["G"]).cuda()
        pl["md"] = torch.from_numpy(pl["mask"]).cuda()
    assert plans[0]["ses"].uses_tma and plans[1]["ses"].uses_tma
    for rnd in range(3):
        for pl in plans:
            ses = pl["ses"]
            rp, ci, a, w = pl["code"]
            ghat = torch.empty((1, pl["d"]), dtype=torch.float32, device="cuda")
            ses.encode(pl["Gd"], rnd)
            ses.decode(pl["md"], ghat=ghat)
            torch.cuda.synchronize()
            oc, osc, _, _ = orp.encode_quantize(rp, ci, a, pl["bits"], 512, 9, rnd, pl["G"])
            og, _ = orp.decode(pl["d"], pl["bits"], 512, w, pl["mask"], oc, osc)
            assert int(ses.status.item()) == 0
            assert (ses.codes_host() == oc).all()
            assert (ses.scales_host().view(np.uint32) == osc.view(np.uint32)).all()
            assert (ghat.cpu().numpy().view(np.uint32) == og.view(np.uint32)).all()
    for pl in plans:
        pl["ses"].close()
