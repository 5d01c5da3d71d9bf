"""The list schedule that k_local_state_gather walks, checked record by record (integer work:
exact).  fda_debug_schedule returns the record of a tile; fda_debug_hash gives the bucket and
sign of every index straight from the coefficients.  A record is right when

  * every index of the tile appears exactly once per sketch row, in a list of its own cell, with
    its own sign; padding entries point at the eight zero rows behind the tile and carry no sign;
  * a lane with no list (cell id l*m) holds padding only; no list is longer than the limit;
  * a cell is flagged "add atomically" exactly when it owns more than one list, and a cell with
    n indices owns ceil(n / limit) lists;
  * in every step the eight lanes of a pass address rows in eight different 16-byte bank groups
    (row mod 8; index r of the tile is stored in row r ^ ((r >> 3) & 3)), so the shared-memory load
    of the step is conflict free;
  * items come with the most steps first, their chunk offsets follow from the steps, and the
    header's sizes add up.

Coefficient tables: random ones, bucket = index mod m (every list in one residue class when
m is a multiple of 8) and one bucket for every index (one cell cut into many lists).  Nothing here
compares against the CUDA path's own arithmetic: the hash values come from the bit-exact dump
that test_gpu_parity.py checks against Python integers.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

P = (1 << 61) - 1


@pytest.fixture(scope="module")
def env():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("CUDA device required for -m gpu tests")
    import paper_2405_20988_b200 as F
    F.load_library()
    return torch, F


def rand_coeffs(rng, l):
    c = rng.integers(0, P, size=6 * l, dtype=np.uint64)
    c[0::6] |= np.uint64(1)
    c[2::6] |= np.uint64(1)
    return c


def check_record(rec, info, l, m, buckets, signs):
    """buckets / signs: [l, tile_indices] hash values of the tile.  Returns (steps walked by a
    lane in total, entries)."""
    T, slots, max_len, oct_ = info["tile_indices"], info["slots"], info["max_len"], info["lanes_per_pass"]
    assert slots == 32 and oct_ == 8 and info["pad_rows"] == 8 and T % 1024 == 0 and T + 8 <= 8192
    hdr = rec[:16].view(np.uint32)
    items, rec_bytes, chunks = int(hdr[0]), int(hdr[1]), int(hdr[2])
    assert hdr[3] == 0
    assert rec_bytes == info["record_bytes"] == rec.size
    desc = rec[16:16 + 8 * items].view(np.uint32).reshape(items, 2)
    cells_off = (16 + 8 * items + 63) // 64 * 64
    ent_off = (cells_off + 64 * items + 255) // 256 * 256
    assert rec_bytes == ent_off + 256 * chunks
    cells = rec[cells_off:cells_off + 64 * items].view(np.uint16).reshape(items, slots).astype(np.int64)
    ent = rec[ent_off:].view(np.uint16).reshape(chunks, slots, 4).astype(np.int64)
    seen = np.zeros((l, T), dtype=np.int64)
    lists_of_cell = {}
    steps_all = (desc[:, 0] & 0xFFFF).astype(np.int64)
    assert (np.diff(steps_all) <= 0).all(), "items are ordered by steps, most first"
    blocks = (desc[:, 0] >> 16).astype(np.int64)
    assert sorted(blocks.tolist()) == list(range(items)), "every cell block is used by one item"
    used_chunks = np.zeros(chunks, dtype=np.int64)
    lane_steps = 0
    for it in range(items):
        s, first = int(steps_all[it]), int(desc[it, 1])
        assert s >= 1
        nch = (s + 3) // 4
        used_chunks[first:first + nch] += 1
        e = ent[first:first + nch].transpose(0, 2, 1).reshape(nch * 4, slots)     # [step][lane]
        row, neg = e & 0x1FFF, (e >> 15) & 1
        assert ((e & 0x6000) == 0).all()
        assert (row < T + 8).all()
        idx = row ^ ((row >> 3) & 3)          # index r of the tile is stored in row r ^ ((r >> 3) & 3)
        # the eight lanes of a pass: eight different bank groups (row mod 8), in the steps that are walked
        res = (row[:s] % 8).reshape(s, slots // 8, 8)
        assert (np.sort(res, axis=2) == np.arange(8)).all(), "bank groups collide in item %d" % it
        lane_steps += s * slots
        for ln in range(slots):
            cid = int(cells[blocks[it], ln])
            col_idx, col_neg = idx[:, ln], neg[:, ln]
            real = col_idx < T
            assert not col_neg[~real].any(), "padding carries no sign"
            assert not real[s:].any(), "entries behind the item's steps are padding"
            if cid == l * m:
                assert not real.any()
                continue
            row, b = divmod(cid & 0x7FFF, m)
            assert row < l
            n_real = int(real.sum())
            assert 1 <= n_real <= max_len
            ii = col_idx[real]
            assert (buckets[row, ii] == b).all()
            assert (col_neg[real] == (signs[row, ii] < 0)).all()
            np.add.at(seen[row], ii, 1)
            lists_of_cell.setdefault(cid & 0x7FFF, []).append((cid >> 15, n_real))
    assert (used_chunks == 1).all(), "every chunk belongs to exactly one item"
    assert (seen == 1).all(), "every index of the tile exactly once per row"
    for row in range(l):
        counts = np.bincount(buckets[row].astype(np.int64), minlength=m)
        for b in range(m):
            got = lists_of_cell.get(row * m + b, [])
            n = int(counts[b])
            assert len(got) == -(-n // max_len)
            assert all(f == (1 if len(got) > 1 else 0) for f, _ in got)
            assert sum(k for _, k in got) == n
    return lane_steps, l * T


def run(env, l, m, coeffs, d, tiles_to_check, max_steps_ratio=None):
    torch, F = env
    with F.FdaContext(l, m, coeffs, d_max=d, K_max=8) as ctx:
        _, info = ctx.fda_debug_schedule(0)
        T = info["tile_indices"]
        assert info["tiles"] == -(-d // T)
        for tile in tiles_to_check(info["tiles"]):
            b = torch.empty((l, T), dtype=torch.int16, device="cuda")
            s = torch.empty((l, T), dtype=torch.int8, device="cuda")
            ctx.fda_debug_hash(tile * T, T, b, s)
            torch.cuda.synchronize()
            bn = b.cpu().numpy().view(np.uint16).astype(np.int64)
            sn = s.cpu().numpy()
            rec, info = ctx.fda_debug_schedule(tile)
            lane_steps, entries = check_record(rec, info, l, m, bn, sn)
            if max_steps_ratio is not None:
                assert lane_steps <= max_steps_ratio * entries, (lane_steps, entries)


def test_random_tables(env):
    rng = np.random.default_rng(31)
    # with random hashes the lanes idle in less than a quarter of their steps
    run(env, 5, 250, rand_coeffs(rng, 5), 1_000_003, lambda n: [0, 1, n // 2, n - 1], max_steps_ratio=1.25)
    run(env, 3, 100, rand_coeffs(rng, 3), 300_000, lambda n: [0, n - 1])          # lists at the length limit
    run(env, 7, 500, rand_coeffs(rng, 7), 300_000, lambda n: [0, n - 1], max_steps_ratio=1.3)


def test_rotating_and_constant_buckets(env):
    l, m = 3, 256
    c = rand_coeffs(np.random.default_rng(32), l)
    c[0], c[1] = 1, 0                  # bucket = index mod m: every list inside one residue class
    c[6], c[7] = m, 11                 # every index in bucket 11
    run(env, l, m, c, 200_000, lambda n: [0, 3, n - 1])


def test_contexts_without_a_schedule_say_so(env):
    torch, F = env
    rng = np.random.default_rng(33)
    with F.FdaContext(8, 2000, rand_coeffs(rng, 8), d_max=100_000, K_max=4) as ctx:    # lists too short
        with pytest.raises(F.FdaError):
            ctx.fda_debug_schedule(0)
    with F.FdaContext(0, 0, None, d_max=1000, K_max=2) as ctx:                          # no sketch
        with pytest.raises(F.FdaError):
            ctx.fda_debug_schedule(0)
