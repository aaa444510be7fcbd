"""Two CPU ranks (gloo): the sharding recipe of the multi-GPU path. Each rank takes its
pack-block-aligned coordinate range, encodes it on its own with the global block indices
in the random stream, and the gathered pieces must equal the encoding of the whole vector;
step times are reduced with a maximum over ranks. No GPU is involved: the per-shard encode
is done by the CPU oracle, the range / reduction logic is the product's."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import roundpath as orp
from paper_2605_15890_b200 import sharding
from tests import _codes


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _problem():
    rng = np.random.default_rng(5)
    n = k = 4
    d = 512 * 7 + 100            # 8 pack blocks, ragged tail
    bits = np.array([2, 3, 5, 8], np.uint8)
    p = np.array([0.1, 0.2, 0.3, 0.4])
    code = _codes.cyclic_code(p, bits, k, 2, 256)
    G = rng.standard_normal((k, d)).astype(np.float32)
    return n, k, d, bits, code, G


def _rank_main(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        n, k, d, bits, (rp, ci, a, w), G = _problem()
        B, seed, rnd = 256, 9, 4
        lo, hi = sharding.coordinate_range(d, rank, world)
        q0 = sharding.first_block(d, rank, world)
        pieces = []
        for q in range(q0, q0 + (hi - lo + 511) // 512):
            blk = np.zeros((k, 512), np.float32)
            m0, m1 = q * 512, min((q + 1) * 512, d)
            blk[:, :m1 - m0] = G[:, m0:m1]
            c, s, st, _ = orp.encode_block(rp, ci, a, bits, B, seed, rnd, q, blk)
            assert st == 0
            pieces.append((q, c, s))
        gathered = [None] * world
        dist.all_gather_object(gathered, (lo, hi, pieces))
        ms = sharding.max_over_ranks([10.0 + rank, 5.0 - rank])
        if rank == 0:
            whole_c, whole_s, st, _ = orp.encode_quantize(rp, ci, a, bits, B, seed, rnd, G)
            off = orp.worker_word_offsets(d, bits)
            covered = np.zeros(d, bool)
            for glo, ghi, gp in gathered:
                assert not covered[glo:ghi].any()
                covered[glo:ghi] = True
                for q, c, s in gp:
                    wb = 0
                    for i in range(n):
                        b = int(bits[i])
                        got = c[wb:wb + 16 * b]
                        want = whole_c[off[i] + q * 16 * b: off[i] + (q + 1) * 16 * b]
                        assert (got == want).all(), (q, i)
                        wb += 16 * b
                        for bk in range(512 // B):
                            beta = q * (512 // B) + bk
                            if beta < whole_s.shape[1]:
                                assert s[i, bk].view(np.uint32) == whole_s[i, beta].view(np.uint32)
            assert covered.all()
            assert ms == [10.0 + world - 1, 5.0]
            with open(os.path.join(out_dir, "ok"), "w") as fh:
                fh.write("ok")
    finally:
        dist.destroy_process_group()


def test_two_ranks_reproduce_the_whole_encoding(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    assert (tmp_path / "ok").exists()


def _rank_main_global_norm(rank, world, port, out_dir):
    """The global norm (one l2 norm per worker over the whole vector) on two ranks: first pass on
    the rank's range, all-gather of n floats, the library's combine on every rank, second pass
    with the whole vector's sums. Oracle arithmetic per range; the split, the exchange and the
    combine are the product's."""
    import paper_2605_15890_b200 as agc
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        n, k, d, bits, (rp, ci, a, w), G = _problem()
        seed, rnd = 9, 4
        lo, hi = sharding.power_of_two_range(d, rank, world)
        Gr = np.ascontiguousarray(G[:, lo:hi])
        local = orp.global_sumsq(rp, ci, a, Gr)
        sums = sharding.global_norm_sums(torch.from_numpy(local), agc.agc_combine_norm_sums)
        c, s, st = orp.encode_quantize_with_norm(rp, ci, a, bits, seed, rnd, Gr, sums, first_block=lo // 512)
        assert st == 0
        gathered = [None] * world
        dist.all_gather_object(gathered, (lo, hi, c, s, sums))
        if rank == 0:
            whole_c, whole_s, st, _ = orp.encode_quantize_global(rp, ci, a, bits, seed, rnd, G)
            off = orp.worker_word_offsets(d, bits)
            prev = 0
            for glo, ghi, gc, gs, gsums in gathered:
                assert glo == prev and glo % 512 == 0
                prev = ghi
                assert (gsums.view(np.uint32) == gathered[0][4].view(np.uint32)).all()   # identical norms on all ranks
                assert (gs.view(np.uint32) == whole_s.view(np.uint32)).all()
                roff = orp.worker_word_offsets(ghi - glo, bits)
                nb_r = (ghi - glo + 511) // 512
                for i in range(n):
                    b = int(bits[i])
                    want = whole_c[off[i] + (glo // 512) * 16 * b: off[i] + (glo // 512 + nb_r) * 16 * b]
                    assert (gc[roff[i]:roff[i + 1]] == want).all(), (glo, i)
            assert prev == d
            with open(os.path.join(out_dir, "ok_global"), "w") as fh:
                fh.write("ok")
    finally:
        dist.destroy_process_group()


def test_two_ranks_global_norm_with_one_exchange(tmp_path):
    world = 2
    mp.spawn(_rank_main_global_norm, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    assert (tmp_path / "ok_global").exists()


@pytest.mark.parametrize("d,world", [(1, 2), (512 * 8, 2), (512 * 7 + 100, 2), (25_557_032, 8), (10**8, 3), (513, 4)])
def test_power_of_two_ranges_tile_the_vector(d, world):
    prev = 0
    sizes = []
    for r in range(world):
        lo, hi = sharding.power_of_two_range(d, r, world)
        assert lo == prev and lo <= hi <= d and (lo % 512 == 0 or lo == d)
        sizes.append((hi - lo + 511) // 512)
        prev = hi
    assert prev == d
    per = sizes[0]
    assert per & (per - 1) == 0                      # a power of two
    full = [s for s in sizes if s == per]
    assert all(s <= per for s in sizes) and sizes[:len(full)] == full


@pytest.mark.parametrize("d,world", [(0, 3), (1, 2), (511, 2), (512, 2), (513, 4), (25_557_032, 8), (10**8, 3)])
def test_coordinate_ranges_tile_the_vector(d, world):
    prev = 0
    for r in range(world):
        lo, hi = sharding.coordinate_range(d, r, world)
        assert lo == prev and lo <= hi <= d
        assert lo % 512 == 0 or lo == d
        assert sharding.first_block(d, r, world) * 512 == lo or lo == d
        prev = hi
    assert prev == d
    sizes = [sharding.coordinate_range(d, r, world) for r in range(world)]
    blocks = [(hi - lo + 511) // 512 for lo, hi in sizes]
    assert max(blocks) - min(blocks) <= 1


@pytest.mark.parametrize("d,world,B", [(25_557_032, 8, 1024), (10**7 + 3, 3, 4096), (5000, 4, 2048)])
def test_ranges_aligned_to_buckets_of_several_blocks(d, world, B):
    """With buckets above 512 coordinates a shard starts at a bucket and first_block still counts
    pack blocks (a multiple of the blocks per bucket, which agc_plan_set_first_block requires)."""
    prev = 0
    for r in range(world):
        lo, hi = sharding.coordinate_range(d, r, world, align=B)
        assert lo == prev and lo <= hi <= d
        assert lo % B == 0 or lo == d
        fb = sharding.first_block(d, r, world, align=B)
        assert fb * 512 == lo or lo == d
        assert fb % (B // 512) == 0 or lo == d
        prev = hi
    assert prev == d
