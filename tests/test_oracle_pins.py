"""Pins the CPU oracle to things other than itself: the paper's printed values
(tests/golden/), closed forms, hand-worked examples, Python big-integer arithmetic and
brute force on tiny inputs.  Nothing here touches the CUDA library."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2501_16007_b200 import synth

P = 65521
M_LOW, M_HIGH = 2 ** 15 + 1, 2 ** 16      # Algorithm 6 search range, inclusive
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16_bits(values):
    t = torch.tensor(values, dtype=torch.float32).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def read_constants():
    out = {}
    with open(os.path.join(GOLDEN, "paper_constants.txt")) as f:
        for line in f:
            line = line.split("#")[0].split()
            if len(line) == 2:
                out[line[0]] = int(line[1])
    return out


# ---------------------------------------------------------------- field constants

def test_p_is_the_largest_prime_below_2_16():
    def is_prime(n):
        return n > 1 and all(n % d for d in range(2, int(math.isqrt(n)) + 1))
    assert is_prime(P)
    assert not any(is_prime(n) for n in range(P + 1, 2 ** 16))
    assert oracle.P_FIELD == P
    # every finite bf16 pattern (and +-Inf) stays below p, so it survives "y mod p"
    assert 0xFF80 < P


def test_paper_size_arithmetic():
    c = read_constants()
    k, n = c["top_k"], c["tokens_per_proof"]
    assert 2 + 2 * k == c["proof_bytes_k128"]
    assert 2 * k == c["coeff_bytes_k128"]
    assert 2 * 4096 == c["bytes_per_token_raw"]
    assert c["coeff_bytes_k128"] // n == c["bytes_per_token_proof"]
    assert c["bytes_per_token_raw"] // c["bytes_per_token_proof"] == c["reduction"]
    assert n * 4096 * 2 == c["chunk_bytes_8b"]
    assert len(oracle.encode(65536, np.zeros(k, np.uint16))) == c["proof_bytes_k128"]


# ---------------------------------------------------------------- top-k

def brute_topk(patterns, k, fp32=False):
    """Repeatedly pick the best remaining element: O(N k), no sort."""
    flat = patterns.reshape(-1)
    mask = 0x7FFFFFFF if fp32 else 0x7FFF
    keys = [int(v) & mask for v in flat]
    taken, out = set(), []
    for _ in range(k):
        best = None
        for i, key in enumerate(keys):
            if i in taken:
                continue
            if best is None or key > keys[best]:
                best = i
        taken.add(best)
        out.append(best)
    return out


@pytest.mark.parametrize("seed", range(6))
def test_topk_matches_brute_force_selection(seed):
    rng = np.random.default_rng(seed)
    rows, hidden, k = 3, 37, 11
    # few distinct magnitudes so that ties at the cut are the norm
    vals = rng.integers(-6, 7, size=(rows, hidden)).astype(np.float32) * 0.25
    pat = bf16_bits(vals.tolist()).reshape(rows, hidden)
    idx, bits = oracle.topk(pat, k)
    assert idx.tolist() == brute_topk(pat, k)
    assert bits.tolist() == [int(pat.reshape(-1)[i]) for i in idx]


def test_topk_all_equal_takes_the_first_indices():
    pat = np.zeros((4, 64), np.uint16)
    idx, _ = oracle.topk(pat, 17)
    assert idx.tolist() == list(range(17))
    pat[:] = bf16_bits([80.0])[0]
    pat[1, :] ^= 0x8000  # a row of -80: same magnitude
    idx, bits = oracle.topk(pat, 70)
    assert idx.tolist() == list(range(70))
    assert bits[63] == 0x42A0 and bits[64] == 0xC2A0  # 80.0 and -80.0 as bf16


def test_topk_ranks_by_magnitude_not_value():
    pat = bf16_bits([[1.0, -3.0, 2.0, -0.5, 0.0, -0.0, 2.5, -2.5]])
    idx, _ = oracle.topk(pat, 4)
    assert idx.tolist() == [1, 6, 7, 2]  # |-3| > |2.5| = |-2.5| (lower index first) > |2|


def test_topk_unaffected_by_shuffling_the_losers():
    rng = np.random.default_rng(3)
    vals = rng.standard_normal((2, 200)).astype(np.float32)
    pat = bf16_bits(vals.tolist()).reshape(2, 200)
    k = 9
    idx, bits = oracle.topk(pat, k)
    flat = pat.reshape(-1).copy()
    cut_key = int(bits[-1]) & 0x7FFF
    losers = [i for i in range(flat.size) if (int(flat[i]) & 0x7FFF) < cut_key]
    perm = rng.permutation(losers)
    shuffled = flat.copy()
    shuffled[losers] = flat[perm]
    idx2, bits2 = oracle.topk(shuffled.reshape(2, 200), k)
    assert idx2.tolist() == idx.tolist() and bits2.tolist() == bits.tolist()


def test_topk_fp32_uses_full_magnitude_and_commits_upper_half():
    vals = np.array([[1.0, 1.0000001, -1.0000002, 0.5, 3.0]], np.float32)
    idx, bits = oracle.topk(vals, 3)
    assert idx.tolist() == [4, 2, 1]  # bf16 rounding would tie 1, 1.0000001 and -1.0000002
    u = vals.view(np.uint32).reshape(-1)
    assert bits.tolist() == [int(u[i]) >> 16 for i in idx]
    assert idx.tolist() == brute_topk(vals.view(np.uint32), 3, fp32=True)


def test_topk_k_larger_than_chunk():
    assert oracle.topk(np.zeros((1, 4), np.uint16), 5) is None


# ---------------------------------------------------------------- injective modulus

def check_modulus_by_definition(indices, m):
    """m works, and every larger candidate up to 65536 fails (Algorithm 6's 'largest')."""
    def injective(mm):
        return len({(i % mm) % P for i in indices}) == len(indices)
    assert injective(m)
    assert all(not injective(mm) for mm in range(m + 1, 65537))


def test_modulus_worked_outlier_sets():
    # 4 outlier channels x 32 tokens at H = 4096; 8 channels x 16 tokens at H = 8192
    a = [t * 4096 + c for t in range(32) for c in range(4)]
    b = [t * 8192 + c for t in range(16) for c in (0, 1, 2, 3, 4096, 4097, 4098, 4099)]
    small = list(range(0, 32768, 256))
    for idx in (a, b, small):
        m = oracle.find_injective_modulus(idx)
        check_modulus_by_definition(idx, m)
    assert oracle.find_injective_modulus(a) == 65532
    assert oracle.find_injective_modulus(b) == 65532
    c8 = [t * 8192 + c for t in range(16) for c in range(8)]   # 8 adjacent channels instead
    check_modulus_by_definition(c8, oracle.find_injective_modulus(c8))
    assert oracle.find_injective_modulus(c8) == 65528
    assert oracle.find_injective_modulus(small) == 65536  # all indices below 2^15 + 1


def test_modulus_random_sets_by_definition():
    rng = np.random.default_rng(0)
    for _ in range(40):
        idx = rng.choice(131072, size=128, replace=False).tolist()
        check_modulus_by_definition(idx, oracle.find_injective_modulus(idx))


def test_modulus_field_collision_is_refused():
    # 3 and 3 + p are distinct mod 65536 but equal mod p: the literal Algorithm 6 accepts
    # 65536, the proof path must not (x-coordinates would coincide in Z_p).
    idx = [3, 3 + P, 100]
    assert oracle.find_injective_modulus(idx, field_distinct=False) == 65536
    m = oracle.find_injective_modulus(idx, field_distinct=True)
    assert m < 65536
    check_modulus_by_definition(idx, m)


def test_modulus_none_exists():
    # 65537 values in 65536 residue classes can never be injective; a much smaller clash:
    # indices that agree modulo every candidate do not exist, so use duplicates.
    assert oracle.find_injective_modulus([5, 5, 9]) == 0


def covering_index_set():
    """512 distinct indices whose pairwise differences take every value from 1 to 65536: the residues
    0..255 and the multiples 256, 512, ..., 65536 (256 j - r covers [256 j - 255, 256 j]).  Every
    candidate modulus of Algorithm 6 equals one of the differences, so none is injective."""
    return list(range(256)) + [256 * j for j in range(1, 257)]


def test_modulus_none_exists_for_a_covering_set():
    idx = covering_index_set()
    assert len(set(idx)) == 512
    diffs = {b - a for a in idx for b in idx if b > a}
    assert all(m in diffs for m in range(M_LOW, M_HIGH + 1))       # the reason, checked directly
    assert oracle.find_injective_modulus(idx) == 0
    assert oracle.find_injective_modulus(idx, field_distinct=False) == 0
    # a chunk whose 512 largest magnitudes sit exactly there: Algorithm 6 has nothing to return,
    # the chunk gets its status and a zero proof
    pat = np.full((32, 4096), 0x3C00, np.uint16)
    flat = pat.reshape(-1)
    flat[idx] = 0x4500
    proofs, status, indices = oracle.build_proofs(pat, 32, 512, 1, 32)
    assert status.tolist() == [oracle.ST_NO_MODULUS] and not proofs.any()
    assert sorted(indices[0].tolist()) == sorted(idx)


def test_modulus_distribution_matches_table_11():
    table = []
    with open(os.path.join(GOLDEN, "modulus_distribution.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                m, r = line.split()
                table.append((int(m), float(r)))
    # closed form of the first row: no two of 128 uniform residues mod 65536 coincide
    closed = math.prod(1 - i / 65536 for i in range(128))
    assert abs(closed - table[0][1]) < 5e-5
    rng = np.random.default_rng(11)
    trials = 60000
    sets = rng.integers(0, 2 ** 31, size=(trials, 128), dtype=np.int64).astype(np.uint32)
    counts = {}
    for row in sets:
        m = oracle.find_injective_modulus(row, field_distinct=False)
        counts[m] = counts.get(m, 0) + 1
    for m, ratio in table[:4]:
        got = counts.get(m, 0) / trials
        sigma = math.sqrt(ratio * (1 - ratio) / trials)
        assert abs(got - ratio) < 4.5 * sigma + 5e-5, (m, got, ratio)


# ---------------------------------------------------------------- Z_p arithmetic

def test_inverse_exhaustive():
    lib = oracle.lib()
    for a in range(1, P):
        inv = lib.oracle_mod_inverse(a)
        assert 0 < inv < P and (a * inv) % P == 1


def test_euclid_inverse_agrees_and_handles_edge_cases():
    for a in list(range(1, 400)) + [P - 1, P - 2, 32768, 40000]:
        assert oracle.mod_inverse_euclid(a, P) == pow(a, -1, P)
    assert oracle.mod_inverse_euclid(5, 1) == 0      # no ring to invert in
    assert oracle.mod_inverse_euclid(5, 0) == 0
    assert oracle.mod_inverse_euclid(6, 9) == 9      # gcd 3: no inverse exists, reported as m
    assert oracle.mod_inverse_euclid(7, 40) == pow(7, -1, 40)


def test_horner_against_python_integers():
    rng = np.random.default_rng(5)
    for k in (1, 2, 7, 128):
        c = rng.integers(0, P, size=k).astype(np.uint16)
        for x in (0, 1, 2, P - 1, 12345, 65535):
            want = sum(int(cd) * pow(x % P, d, P) for d, cd in enumerate(c)) % P
            assert oracle.horner(c, x) == want


# ---------------------------------------------------------------- interpolation

def test_interpolation_hand_example():
    # -1 + 4x - x^2 passes through (1,2), (2,3), (4,-1)
    c = oracle.interpolate([1, 2, 4], [2, 3, P - 1])
    assert c.tolist() == [P - 1, 4, P - 1]


def test_interpolation_small_closed_forms():
    assert oracle.interpolate([77], [4242]).tolist() == [4242]
    x0, y0, x1, y1 = 10, 500, 65000, 3
    slope = ((y1 - y0) * pow(x1 - x0, -1, P)) % P
    icpt = (y0 - slope * x0) % P
    assert oracle.interpolate([x0, x1], [y0, y1]).tolist() == [icpt, slope]


@pytest.mark.parametrize("k", [3, 16, 128, 256, 512])
def test_interpolant_passes_through_every_point(k):
    rng = np.random.default_rng(k)
    x = rng.choice(P, size=k, replace=False)
    y = rng.integers(0, P, size=k)
    c = oracle.interpolate(x, y)
    for xj, yj in zip(x.tolist(), y.tolist()):
        assert sum(int(cd) * pow(xj, d, P) for d, cd in enumerate(c)) % P == yj
    # uniqueness: Lagrange's form must give the same coefficients
    assert oracle.interpolate(x, y, lagrange=True).tolist() == c.tolist()
    # and the order of the points is irrelevant
    perm = rng.permutation(k)
    assert oracle.interpolate(x[perm], y[perm]).tolist() == c.tolist()


def test_interpolation_rejects_repeated_x():
    with pytest.raises(ValueError):
        oracle.interpolate([1, 2, 1 + P], [5, 6, 7])


# ---------------------------------------------------------------- encode / decode

def test_encode_decode_roundtrip_and_layout():
    rng = np.random.default_rng(9)
    c = rng.integers(0, P, size=128).astype(np.uint16)
    for m in (65536, 65535, 32769, 65532):
        proof = oracle.encode(m, c)
        assert proof.size == 258
        assert int(proof[0]) | (int(proof[1]) << 8) == (m & 0xFFFF)
        assert int(proof[2]) | (int(proof[3]) << 8) == int(c[0])       # ascending degree
        assert int(proof[256]) | (int(proof[257]) << 8) == int(c[127])
        st, k, m2, c2 = oracle.decode(proof)
        assert (st, k, m2) == (oracle.ST_OK, 128, m) and c2.tolist() == c.tolist()


def test_decode_rejects_malformed_proofs():
    c = np.arange(8, dtype=np.uint16)
    good = oracle.encode(40000, c)
    assert oracle.decode(good)[0] == oracle.ST_OK
    assert oracle.decode(good[:-1])[0] == oracle.ST_BAD_PROOF          # odd length
    low = good.copy()
    low[0], low[1] = 0x00, 0x80                                        # m = 32768 < 2^15 + 1
    assert oracle.decode(low)[0] == oracle.ST_BAD_PROOF
    big = good.copy()
    big[2], big[3] = 0xF1, 0xFF                                        # coefficient 65521 = p
    assert oracle.decode(big)[0] == oracle.ST_BAD_PROOF


# ---------------------------------------------------------------- whole chunks

def random_chunk(rng, rows, hidden):
    vals = rng.standard_t(3, size=(rows, hidden)) * 0.5
    return bf16_bits(vals.tolist()).reshape(rows, hidden)


@pytest.mark.parametrize("k", [1, 5, 32, 128])
def test_proof_commits_to_every_selected_value(k):
    rng = np.random.default_rng(100 + k)
    rows, hidden = 8, 512
    pat = random_chunk(rng, rows, hidden)
    proofs, status, indices = oracle.build_proofs(pat, rows, k, 1, rows)
    assert status.tolist() == [oracle.ST_OK] and proofs.shape == (1, 2 + 2 * k)
    st, kk, m, c = oracle.decode(proofs[0])
    assert st == oracle.ST_OK and kk == k
    idx = indices[0].tolist()
    assert idx == brute_topk(pat, k)
    assert len({(i % m) % P for i in idx}) == k
    flat = pat.reshape(-1)
    for i in idx:
        x = (i % m) % P
        assert sum(int(cd) * pow(x, d, P) for d, cd in enumerate(c)) % P == int(flat[i])


def test_identical_activations_validate_with_zero_error():
    rng = np.random.default_rng(7)
    pat = random_chunk(rng, 32, 256)
    proofs, _, indices = oracle.build_proofs(pat, 32, 128, 1, 32)
    res = oracle.verify_proofs(pat, proofs, 32, 128, 1, 32, gen_indices=indices)[0]
    assert (res["exp_mismatch"], res["n_match"], res["mant_diff_sum"]) == (0, 128, 0)
    assert res["mant_mean"] == 0.0 and res["mant_median"] == 0.0
    assert res["accept"] == 1 and res["status"] == 0 and res["topk_mismatch"] == 0


def staircase_chunk(mantissas, signs=None):
    """One row whose k leading elements have strictly decreasing exponents (so their ranks
    do not depend on the mantissa) followed by zeros."""
    k = len(mantissas)
    row = np.zeros(64, np.uint16)
    for j, mant in enumerate(mantissas):
        row[j] = ((140 - j) << 7) | mant
        if signs is not None and signs[j]:
            row[j] |= 0x8000
    assert k <= 40
    return row.reshape(1, 64)


def test_mantissa_statistics_hand_cases():
    base = [10, 20, 30, 40]
    proofs, _, _ = oracle.build_proofs(staircase_chunk(base), 1, 4, 1, 1)
    # differences 3, 0, 7, 2 -> sum 12, mean 3, median (2 + 3) / 2
    res = oracle.verify_proofs(staircase_chunk([13, 20, 23, 42]), proofs, 1, 4, 1, 1)[0]
    assert (res["exp_mismatch"], res["n_match"], res["mant_diff_sum"]) == (0, 4, 12)
    assert res["mant_mean"] == 3.0 and res["mant_median"] == 2.5 and res["accept"] == 1
    # odd count: one exponent mismatch (sign flip) leaves diffs {3, 7, 2} -> median 3
    res = oracle.verify_proofs(staircase_chunk([13, 20, 23, 42], signs=[0, 1, 0, 0]), proofs, 1, 4, 1, 1)[0]
    assert (res["exp_mismatch"], res["n_match"], res["mant_diff_sum"]) == (1, 3, 12)
    assert res["mant_mean"] == 4.0 and res["mant_median"] == 3.0
    # the narrow reading ignores the sign bit
    res = oracle.verify_proofs(staircase_chunk([13, 20, 23, 42], signs=[0, 1, 0, 0]), proofs, 1, 4, 1, 1,
                               sign_in_exponent=False)[0]
    assert (res["exp_mismatch"], res["n_match"]) == (0, 4)


def test_lsb_flips_sum_to_their_count():
    rng = np.random.default_rng(21)
    k = 32
    base = rng.integers(0, 128, size=k).tolist()
    proofs, _, _ = oracle.build_proofs(staircase_chunk(base), 1, k, 1, 1)
    flipped = list(base)
    for j in (0, 3, 4, 9, 30):
        flipped[j] ^= 1
    res = oracle.verify_proofs(staircase_chunk(flipped), proofs, 1, k, 1, 1)[0]
    assert (res["exp_mismatch"], res["n_match"], res["mant_diff_sum"]) == (0, k, 5)
    assert res["mant_mean"] == 5 / k and res["mant_median"] == 0.0


def test_thresholds_are_strict():
    base = [0] * 8
    proofs, _, _ = oracle.build_proofs(staircase_chunk(base), 1, 8, 1, 1)
    moved = staircase_chunk([4] * 8, signs=[1, 1, 0, 0, 0, 0, 0, 0])  # err_e 2, diffs all 4
    kw = dict(chunk_len=1, k=8, num_seqs=1, tokens_per_seq=1)
    def accept(**t):
        return int(oracle.verify_proofs(moved, proofs, **kw, **t)[0]["accept"])
    assert accept(t_exp=2, t_mean=4.0, t_median=4.0) == 1    # equal to a threshold passes
    assert accept(t_exp=1, t_mean=4.0, t_median=4.0) == 0
    assert accept(t_exp=2, t_mean=3.999, t_median=4.0) == 0
    assert accept(t_exp=2, t_mean=4.0, t_median=3.5) == 0


def test_nothing_matched_is_rejected():
    base = [1, 2, 3]
    proofs, _, _ = oracle.build_proofs(staircase_chunk(base), 1, 3, 1, 1)
    res = oracle.verify_proofs(staircase_chunk(base, signs=[1, 1, 1]), proofs, 1, 3, 1, 1, t_exp=100)[0]
    assert (res["exp_mismatch"], res["n_match"], res["accept"]) == (3, 0, 0)
    assert res["mant_mean"] == 0.0 and res["mant_median"] == 0.0


def test_index_overlap_hand_cases():
    """topk_mismatch = k - |generator indices ∩ validator indices| (Section 5.4), predicted by hand."""
    k = 4
    gen = np.zeros((1, 64), np.uint16)
    for j in range(k):
        gen[0, j] = (140 - j) << 7                    # the generator selects elements 0, 1, 2, 3
    proofs, _, indices = oracle.build_proofs(gen, 1, k, 1, 1)
    assert sorted(indices[0].tolist()) == [0, 1, 2, 3]
    # the validator's element 3 falls to zero and element 40 rises: it selects 0, 1, 2, 40 -> one index differs
    one_off = gen.copy()
    one_off[0, 3] = 0
    one_off[0, 40] = 137 << 7
    res = oracle.verify_proofs(one_off, proofs, 1, k, 1, 1, gen_indices=indices)[0]
    assert res["topk_mismatch"] == 1 and res["status"] == 0
    # the validator's large values sit at 10 .. 13: no index in common -> k
    moved = np.zeros((1, 64), np.uint16)
    for j in range(k):
        moved[0, 10 + j] = (140 - j) << 7
    res = oracle.verify_proofs(moved, proofs, 1, k, 1, 1, gen_indices=indices)[0]
    assert res["topk_mismatch"] == k
    # generator indices given in another order: a set difference does not depend on it
    res = oracle.verify_proofs(one_off, proofs, 1, k, 1, 1, gen_indices=indices[:, ::-1].copy())[0]
    assert res["topk_mismatch"] == 1
    # without generator indices there is nothing to compare
    assert oracle.verify_proofs(one_off, proofs, 1, k, 1, 1)[0]["topk_mismatch"] == -1


def test_thresholds_per_chunk():
    """Thresholds given per chunk (Section 6: thresholds chosen per generation) decide each chunk by
    its own entry; the statistics do not depend on them."""
    base = [0] * 8
    one = staircase_chunk(base)
    gen = np.concatenate([one, one, one])             # three identical one-row chunks
    proofs, _, _ = oracle.build_proofs(gen, 1, 8, 3, 1)
    moved_one = staircase_chunk([4] * 8, signs=[1, 1, 0, 0, 0, 0, 0, 0])   # err_e 2, diffs all 4
    moved = np.concatenate([moved_one, moved_one, moved_one])
    res = oracle.verify_proofs(moved, proofs, 1, 8, 3, 1, t_exp=[2, 1, 2], t_mean=[4.0, 4.0, 3.5],
                               t_median=[4.0, 4.0, 4.0])
    assert res["accept"].tolist() == [1, 0, 0]
    assert res["exp_mismatch"].tolist() == [2, 2, 2] and res["mant_mean"].tolist() == [4.0, 4.0, 4.0]
    # the comparison is over the integers: a negative exponent threshold is exceeded by zero mismatches
    res = oracle.verify_proofs(gen, proofs, 1, 8, 3, 1, t_exp=[-1, 0, 5])
    assert res["exp_mismatch"].tolist() == [0, 0, 0] and res["accept"].tolist() == [0, 1, 1]
    # scalars and arrays mix
    res = oracle.verify_proofs(moved, proofs, 1, 8, 3, 1, t_exp=2, t_mean=4.0, t_median=[4.0, 3.5, 5.0])
    assert res["accept"].tolist() == [1, 0, 1]


def test_bad_proof_and_short_chunk_statuses():
    pat = staircase_chunk([1, 2, 3])
    proofs, status, _ = oracle.build_proofs(pat, 1, 3, 1, 1)
    broken = proofs.copy()
    broken[0, 0], broken[0, 1] = 1, 0   # m = 1
    res = oracle.verify_proofs(pat, broken, 1, 3, 1, 1)[0]
    assert res["status"] == oracle.ST_BAD_PROOF and res["accept"] == 0
    tiny = np.zeros((1, 4), np.uint16)
    proofs, status, _ = oracle.build_proofs(tiny, 1, 8, 1, 1)
    assert status.tolist() == [oracle.ST_K_EXCEEDS] and not proofs.any()


def test_negative_nan_pattern_is_flagged():
    pat = staircase_chunk([1, 2, 3])
    pat[0, 5] = 0xFFF5   # >= p: cannot be reproduced from y mod p
    _, status, _ = oracle.build_proofs(pat, 1, 3, 1, 1)
    assert status.tolist() == [oracle.ST_NONFINITE]


def test_ragged_batches_and_row_stride():
    rng = np.random.default_rng(33)
    wide = random_chunk(rng, 23, 96)
    act = wide[:, :64]                      # row stride 96, hidden 64
    offsets = [0, 9, 9, 23]                 # lengths 9, 0, 14 with chunk_len 4 -> 3 + 0 + 4 chunks
    assert oracle.num_chunks(3, 0, 4, offsets) == 7
    proofs, status, indices = oracle.build_proofs(act, 4, 6, 3, seq_offsets=offsets)
    spans = [(0, 4), (4, 4), (8, 1), (9, 4), (13, 4), (17, 4), (21, 2)]
    for c, (row0, rows) in enumerate(spans):
        chunk = np.ascontiguousarray(act[row0:row0 + rows])
        p1, s1, i1 = oracle.build_proofs(chunk, rows, 6, 1, rows)
        assert proofs[c].tolist() == p1[0].tolist() and indices[c].tolist() == i1[0].tolist()
    res = oracle.verify_proofs(act, proofs, 4, 6, 3, seq_offsets=offsets)
    assert res["accept"].tolist() == [1] * 7


def test_several_k_over_one_ranking_equal_the_single_k_drivers():
    """The sweep drivers rank a chunk once and give every k its prefix: same bytes, statuses,
    indices and results as one call per k -- on a ragged batch whose last chunks are shorter than
    the largest k, with fp32 values as well, and with a proof built from other data."""
    rng = np.random.default_rng(34)
    for make in (lambda: random_chunk(rng, 23, 64), lambda: rng.standard_normal((23, 64)).astype(np.float32)):
        act, other = make(), make()
        offsets = [0, 9, 9, 23]                 # chunk_len 4: chunks of 4,4,1 and 4,4,4,2 rows (64..256 elements)
        ks = [200, 3, 64, 128]
        built = oracle.build_proofs_ks(act, 4, ks, 3, seq_offsets=offsets)
        foreign = oracle.build_proofs_ks(other, 4, ks, 3, seq_offsets=offsets)
        for k in ks:
            p1, s1, i1 = oracle.build_proofs(act, 4, k, 3, seq_offsets=offsets)
            assert np.array_equal(built[k][0], p1) and np.array_equal(built[k][1], s1) and np.array_equal(built[k][2], i1)
        assert oracle.ST_K_EXCEEDS in built[200][1].tolist() and oracle.ST_OK in built[200][1].tolist()
        thr = {k: (38 * k) // 128 for k in ks}
        for proofs, gen in ((built, True), (foreign, False)):
            many = oracle.verify_proofs_ks(act, {k: proofs[k][0] for k in ks}, 4, 3, seq_offsets=offsets, t_exp_by_k=thr,
                                           gen_indices_by_k={k: proofs[k][2] for k in ks} if gen else None)
            for k in ks:
                one = oracle.verify_proofs(act, proofs[k][0], 4, k, 3, seq_offsets=offsets, t_exp=thr[k],
                                           gen_indices=proofs[k][2] if gen else None)
                assert many[k].tobytes() == one.tobytes(), (k, gen)


# ---------------------------------------------------------------- seeded configurations

def tiny_config(seed=0, outliers="fixed", hidden=4096, chunks=4):
    act = synth.make_activations(1, 32 * chunks, hidden, torch.bfloat16, seed=seed, outliers=outliers)
    return act


def test_tiny_config_generate_validate_and_one_ulp_copy():
    act = tiny_config()
    pat = synth.host_patterns(act)
    proofs, status, indices = oracle.build_proofs(pat, 32, 128, 1, 128)
    assert proofs.shape == (4, 258) and status.tolist() == [0] * 4
    # with +-80 on channels 0..3 the selection is (almost surely) the 128 outliers, all tied
    for c in range(4):
        st, k, m, coef = oracle.decode(proofs[c])
        assert st == 0 and k == 128 and len({(int(i) % m) % P for i in indices[c]}) == 128
    same = oracle.verify_proofs(pat, proofs, 32, 128, 1, 128, gen_indices=indices)
    assert same["accept"].tolist() == [1] * 4 and not same["exp_mismatch"].any()
    assert not same["mant_diff_sum"].any() and same["topk_mismatch"].tolist() == [0] * 4
    ulp = synth.host_patterns(synth.plus_one_ulp(act, seed=0))
    res = oracle.verify_proofs(ulp, proofs, 32, 128, 1, 128)
    assert res["accept"].tolist() == [1] * 4
    assert (res["mant_mean"] <= 1.0).all() and (res["exp_mismatch"] <= 38).all()


def test_tampered_activations_are_rejected():
    act = tiny_config(outliers="jitter")
    pat = synth.host_patterns(act)
    proofs, _, _ = oracle.build_proofs(pat, 32, 128, 1, 128)
    other = tiny_config(seed=1000, outliers="jitter")
    res = oracle.verify_proofs(synth.host_patterns(other), proofs, 32, 128, 1, 128)
    assert res["accept"].tolist() == [0] * 4                     # other seed ("different model")
    shifted = synth.prefix_shift(act, other, 1, 128, shift=16)
    res = oracle.verify_proofs(synth.host_patterns(shifted), proofs, 32, 128, 1, 128)
    assert res["accept"].tolist() == [0] * 4                     # prepended tokens
    honest = synth.honest_noise(act, seed=0)
    res = oracle.verify_proofs(synth.host_patterns(honest), proofs, 32, 128, 1, 128)
    assert res["accept"].tolist() == [1] * 4                     # honest recomputation noise


def test_truncated_precision_is_rejected_on_ordinary_values():
    act = tiny_config(outliers="none", hidden=1024)
    pat = synth.host_patterns(act)
    proofs, _, _ = oracle.build_proofs(pat, 32, 128, 1, 128)
    coarse = synth.truncate_mantissa(act, keep_bits=1)
    res = oracle.verify_proofs(synth.host_patterns(coarse), proofs, 32, 128, 1, 128)
    assert res["accept"].tolist() == [0] * 4
    assert (res["mant_mean"] > 10).all()
