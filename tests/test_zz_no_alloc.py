"""The allocation-free update entry point against the ordinary one.

agc_decode_update_static serves callers that may not allocate device memory (all of it
was given to a framework's pool at start-up, or the caller is a plug-in that only ever
receives buffers): it keeps its working data in a fixed array inside the library instead
of in a plan. Here it is called through the C ABI twice in a row, with different sizes,
masks and learning rates the second time, so that anything an earlier call left in the
shared array would show; each result must match what agc_decode gives for the same
messages, and what the CPU oracle gives when it applies the R updates one after the other. The file name sorts last on purpose: with `-x` every other test has already run.
"""
import numpy as np
import pytest

from tests import _codes

pytestmark = pytest.mark.gpu


def _one_case(agc, torch, n, d, B, R, seed):
    from paper_2605_15890_b200.session import Session
    rng = np.random.default_rng(seed)
    k = n
    bits = rng.integers(1, 9, n).astype(np.uint8)
    p = rng.uniform(0.05, 0.5, n)
    rp, ci, a, w = _codes.cyclic_code(p, bits, k, 3, B)
    ses = Session(n, k, d, rp, ci, a, w, p, bits, bucket=B, seed=seed, flags=agc.AGC_FLAG_ALLOW_1BIT)
    G = torch.from_numpy(rng.standard_normal((k, (d + 3) // 4 * 4)).astype(np.float32)).cuda()
    ses.encode(G, 1)
    masks = torch.from_numpy((rng.random((R, n)) >= p).astype(np.uint8)).cuda()
    lr = rng.uniform(1e-3, 1e-2, R).astype(np.float32)
    beta0 = rng.standard_normal(d).astype(np.float32)
    want = torch.from_numpy(beta0.copy()).cuda()
    ses.decode(masks, lr=lr, beta=want)                       # the existing entry point
    got = torch.from_numpy(beta0.copy()).cuda()
    agc.agc_decode_update_static(n, d, B, bits, w, ses.codes, ses.scales, masks, R, lr, got)
    torch.cuda.synchronize()
    want, got = want.cpu().numpy(), got.cpu().numpy()
    codes, scales = ses.codes_host(), ses.scales_host()
    ses.close()
    assert np.abs(want - beta0).max() > 0                     # the update did something
    rel = np.abs(got - want).max() / np.abs(want).max()
    assert rel <= 1e-5, rel
    # and against the oracle's defining order: R updates one after the other
    from oracle import roundpath as orp
    _, ob = orp.decode(d, bits, B, w, masks.cpu().numpy(), codes, scales, lr=lr, beta=beta0, want_ghat=False)
    rel = np.abs(got - ob).max() / np.abs(ob).max()
    assert rel <= 1e-5, rel


def test_static_update_matches_plan_update_twice_in_a_row():
    import torch

    import paper_2605_15890_b200 as agc
    _one_case(agc, torch, n=12, d=70_001, B=256, R=9, seed=21)
    _one_case(agc, torch, n=7, d=4_097, B=512, R=64, seed=22)   # smaller tables over the old ones
    _one_case(agc, torch, n=12, d=70_001, B=256, R=9, seed=21)


def test_static_update_rejects_sizes_beyond_its_limits():
    import torch

    import paper_2605_15890_b200 as agc
    buf = torch.zeros(1024, dtype=torch.float32, device="cuda")
    m = torch.zeros(8, dtype=torch.uint8, device="cuda")
    n_big = 1025
    with pytest.raises(agc.AgcError) as e:
        agc.agc_decode_update_static(n_big, 512, 512, np.full(n_big, 2, np.uint8), np.ones(n_big, np.float32),
                                     buf, buf, m, 1, np.ones(1, np.float32), buf)
    assert e.value.code == agc.AGC_ERR_LIMIT
    with pytest.raises(agc.AgcError) as e:
        agc.agc_decode_update_static(2, 512, 512, np.full(2, 2, np.uint8), np.ones(2, np.float32),
                                     buf, buf, m, 4097, np.ones(4097, np.float32), buf)
    assert e.value.code == agc.AGC_ERR_LIMIT
