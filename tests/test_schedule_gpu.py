"""The list schedule that k_local_state_gather walks, checked record by record (integer work:
exact).  fda_debug_schedule returns the record of a (tile, sketch row); fda_debug_hash gives the
bucket and sign of every index straight from the coefficients.  A record is right when

  * every index of the tile appears exactly once, in a list of its own cell, with its own sign;
  * padding entries point at the zero rows behind the tile and nowhere else;
  * a round has an even number of steps, at least as many as its longest list, no list is
    longer than the limit, and the chunk offsets follow from the steps;
  * a cell is flagged "add atomically" exactly when it owns more than one list;
  * unused slots carry the cell id l*m.

Coefficient tables: random ones, bucket = index mod m (lists of equal length) and one bucket
for every index (one cell split into 128 lists).  Nothing here compares against the CUDA path's
own arithmetic: the hash values come from the bit-exact dump that test_gpu_parity.py checks
against Python integers.
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


def check_record(rec, info, l, m, row, buckets, signs):
    """buckets / signs: the tile's hash values of this sketch row (length tile_indices)."""
    T, NR, hdr_bytes = info["tile_indices"], info["nr_max"], info["header_bytes"]
    slots, max_len, cells_off = info["slots"], info["max_len"], info["cells_offset"]
    words = rec.view(np.uint16)
    rounds = int(words[0])
    assert 1 <= rounds <= NR
    steps = words[2:2 + NR].astype(np.int64)
    first = words[2 + NR:2 + 2 * NR].astype(np.int64)
    cells = rec[cells_off:cells_off + NR * slots * 2].view(np.uint16).reshape(NR, slots).astype(np.int64)
    ent = rec[hdr_bytes:].view(np.uint16)
    seen = np.zeros(T, dtype=np.int64)
    lists_of_cell = {}
    chunk = 0
    for r in range(rounds):
        s = int(steps[r])
        assert s >= 2 and s % 2 == 0 and s <= max_len
        assert int(first[r]) == chunk
        longest = 0
        for q in range(slots):
            cid = int(cells[r, q])
            n_real = 0
            for t in range(s):
                e = int(ent[((chunk + t // 4) * slots + q) * 4 + t % 4])
                idx, neg = e & 0x1FFF, (e >> 15) & 1
                assert (e & 0x6000) == 0
                if idx >= T:                                  # padding: a zero row, no sign
                    assert idx < T + 4 and neg == 0
                    continue
                assert cid != l * m, "an entry in an unused slot"
                n_real += 1
                seen[idx] += 1
                assert (cid & 0x7FFF) == row * m + int(buckets[idx])
                assert neg == (1 if signs[idx] < 0 else 0)
            if cid == l * m:
                assert n_real == 0
            else:
                assert 1 <= n_real <= max_len
                lists_of_cell.setdefault(cid & 0x7FFF, []).append(cid >> 15)
            longest = max(longest, n_real)
        assert s in (longest, longest + 1)
        chunk += (s + 3) // 4
    assert (steps[rounds:] == 0).all()
    assert (seen == 1).all(), "every index of the tile exactly once"
    for cell, flags in lists_of_cell.items():
        assert all(f == (1 if len(flags) > 1 else 0) for f in flags), cell
    counts = np.bincount(buckets.astype(np.int64), minlength=m)
    assert len(lists_of_cell) == int(np.count_nonzero(counts))
    for b in np.nonzero(counts)[0]:
        assert len(lists_of_cell[row * m + int(b)]) == -(-int(counts[b]) // max_len)


def run(env, l, m, coeffs, d, tiles_to_check):
    torch, F = env
    with F.FdaContext(l, m, coeffs, d_max=d, K_max=8) as ctx:
        _, info = ctx.fda_debug_schedule(0, 0)
        T = info["tile_indices"]
        assert info["tiles"] == -(-d // T)
        for tile in tiles_to_check(info["tiles"]):
            b = torch.empty((l, T), dtype=torch.int16, device="cuda")
            s = torch.empty((l, T), dtype=torch.int8, device="cuda")
            ctx.fda_debug_hash(tile * T, T, b, s)
            torch.cuda.synchronize()
            bn = b.cpu().numpy().view(np.uint16)
            sn = s.cpu().numpy()
            for row in range(l):
                rec, info = ctx.fda_debug_schedule(tile, row)
                check_record(rec, info, l, m, row, bn[row], sn[row])


def test_random_tables(env):
    rng = np.random.default_rng(31)
    run(env, 5, 250, rand_coeffs(rng, 5), 1_000_003, lambda n: [0, 1, n // 2, n - 1])
    run(env, 3, 100, rand_coeffs(rng, 3), 300_000, lambda n: [0, n - 1])          # lists longer than the limit
    run(env, 2, 500, rand_coeffs(rng, 2), 300_000, lambda n: [0, n - 1])


def test_rotating_and_constant_buckets(env):
    l, m = 3, 250
    c = rand_coeffs(np.random.default_rng(32), l)
    c[0], c[1] = 1, 0                  # bucket = index mod m
    c[6], c[7] = m, 11                 # every index in bucket 11
    run(env, l, m, c, 200_000, lambda n: [0, 3, n - 1])


def test_contexts_without_a_schedule_say_so(env):
    torch, F = env
    rng = np.random.default_rng(33)
    with F.FdaContext(7, 500, rand_coeffs(rng, 7), d_max=100_000, K_max=4) as ctx:     # lists too short
        with pytest.raises(F.FdaError):
            ctx.fda_debug_schedule(0, 0)
    with F.FdaContext(0, 0, None, d_max=1000, K_max=2) as ctx:                          # no sketch
        with pytest.raises(F.FdaError):
            ctx.fda_debug_schedule(0, 0)
