"""GPU parity of the direct commitments (index and value stored as they are, Section 4) with
the oracle: commitment bytes, statuses, every integer statistic and the exponent-deviation
counts are compared for equality, fp64 mean / median within 1e-9."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2501_16007_b200 as tl
from paper_2501_16007_b200 import synth

from helpers import assert_results_equal, oracle_thresholds

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def host_of(act):
    return synth.host_patterns(act) if act.is_contiguous() else synth.host_patterns(act._base)[:, :act.shape[1]]


def direct_case(act, chunk_len, k, num_seqs, tokens_per_seq, recomputed=None, where=""):
    lay, _ = tl.make_layout(act, chunk_len, k, num_seqs, tokens_per_seq)
    commits, status = tl.toploc_commit_direct(act, lay)
    torch.cuda.synchronize()
    ref_commits, ref_status = oracle.commit_direct(host_of(act), chunk_len, k, num_seqs, tokens_per_seq)
    assert np.array_equal(status.cpu().numpy(), ref_status), where + " status"
    bad = np.nonzero((commits.cpu().numpy() != ref_commits).any(axis=1))[0]
    assert bad.size == 0, "%s commitment bytes differ at chunks %s" % (where, bad[:8])
    cases = {"same": act}
    cases.update(recomputed or {})
    out = {}
    for name, rec in cases.items():
        res, dev = tl.toploc_verify_direct(rec, lay, commits, tl.default_thresholds(k))
        torch.cuda.synchronize()
        got = res.cpu().numpy().view(tl.RESULT_DTYPE).reshape(-1)
        ref, ref_dev = oracle.verify_direct(host_of(rec), ref_commits, chunk_len, k, num_seqs, tokens_per_seq,
                                            **oracle_thresholds(k))
        assert_results_equal(got, ref, "%s verify[%s]" % (where, name))
        assert np.array_equal(dev.cpu().numpy().astype(np.uint32), ref_dev), "%s deviation bins [%s]" % (where, name)
        out[name] = ref
    return out


@pytest.mark.parametrize("k", [1, 128, 256, 257, 512, 1000, 4096])
@pytest.mark.parametrize("outliers", ["fixed", "none"])
def test_bf16_chunks(k, outliers):
    S, T, H, L = 3, 96, 4096, 32
    act = synth.make_activations(S, T, H, torch.bfloat16, seed=40 + k, device=DEV, outliers=outliers)
    rec = {"noise": synth.honest_noise(act, seed=7), "ulp": synth.plus_one_ulp(act, seed=8),
           "other": synth.make_activations(S, T, H, torch.bfloat16, seed=900 + k, device=DEV, outliers=outliers)}
    out = direct_case(act, L, k, S, T, rec, "bf16 k=%d %s" % (k, outliers))
    assert (out["same"]["accept"] == 1).all() and (out["same"]["exp_mismatch"] == 0).all()
    if outliers == "none" and k >= 128:
        assert (out["other"]["accept"] == 0).all()


@pytest.mark.parametrize("k", [64, 1000, 2048])
def test_fp32_chunks(k):
    S, T, H, L = 2, 64, 2048, 32
    act = synth.make_activations(S, T, H, torch.float32, seed=50 + k, device=DEV, outliers="jitter")
    rec = {"noise": synth.honest_noise(act, seed=9, rel=2.0 ** -10)}
    direct_case(act, L, k, S, T, rec, "fp32 k=%d" % k)


def test_70b_shaped_chunks_and_ragged_tail():
    # 8192-wide rows, 100 tokens per sequence: three chunks of 32 rows and one of 4
    S, T, H, L, k = 2, 100, 8192, 32, 4096
    act = synth.make_activations(S, T, H, torch.bfloat16, seed=61, device=DEV)
    direct_case(act, L, k, S, T, {"noise": synth.honest_noise(act, seed=3)}, "70B-shaped")


def test_k_above_256_on_chunks_too_long_for_two_blocks_per_sm():
    # 2^19 elements per chunk: beyond the 512-thread kernels' reach, so k = 300 and 512 stay with the
    # warp-per-chunk kernels (which they leave for chunks of up to 2^18 elements)
    S, T, H, L = 2, 64, 8192, 64
    act = synth.make_activations(S, T, H, torch.bfloat16, seed=63, device=DEV, outliers="jitter")
    for k in (300, 512):
        direct_case(act, L, k, S, T, {"noise": synth.honest_noise(act, seed=5)}, "2^19-element chunks k=%d" % k)


@pytest.mark.parametrize("k", [128, 1024])
def test_full_size_launch_sampled(k):
    """The 70B-shaped batch (256 sequences x 4096 tokens, H = 8192) committed and validated in one call
    each, the launch configuration `bench.py --direct` times (k = 128: a warp per chunk; k = 1024: a
    block per chunk); whole sampled sequences against the oracle, properties of an exact copy on all
    32768 chunks."""
    S, T, H, L = 256, 4096, 8192, 32
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * 2 ** 30:
        pytest.skip("needs 40 GB of free device memory")
    act = synth.make_activations(S, T, H, torch.bfloat16, seed=4, device=DEV)
    noisy = synth.honest_noise(act, seed=5)
    lay, _ = tl.make_layout(act, L, k, S, T)
    commits, status = tl.toploc_commit_direct(act, lay)
    same, _ = tl.toploc_verify_direct(act, lay, commits, tl.default_thresholds(k))
    honest, dev = tl.toploc_verify_direct(noisy, lay, commits, tl.default_thresholds(k))
    torch.cuda.synchronize()
    assert not status.any().item()
    same = same.cpu().numpy().view(tl.RESULT_DTYPE).reshape(-1)
    assert same["accept"].all() and not same["exp_mismatch"].any() and not same["topk_mismatch"].any()
    assert (same["n_match"] == k).all() and not same["mant_diff_sum"].any()
    honest = honest.cpu().numpy().view(tl.RESULT_DTYPE).reshape(-1)
    cps = T // L
    for s in (3, 200):
        rows, chunks = slice(s * T, (s + 1) * T), slice(s * cps, (s + 1) * cps)
        ref_commits, ref_status = oracle.commit_direct(synth.host_patterns(act[rows]), L, k, 1, T)
        assert np.array_equal(commits[chunks].cpu().numpy(), ref_commits), "commitments of sequence %d" % s
        ref, ref_dev = oracle.verify_direct(synth.host_patterns(noisy[rows]), ref_commits, L, k, 1, T,
                                            **oracle_thresholds(k))
        assert_results_equal(honest[chunks], ref, "70B direct k=%d seq %d" % (k, s))
        assert np.array_equal(dev[chunks].cpu().numpy().astype(np.uint32), ref_dev)


def test_ties_decide_the_selection():
    # all equal; two values only; ascending magnitudes
    H, L = 1024, 16
    same = torch.full((L, H), 1.5, dtype=torch.bfloat16, device=DEV)
    direct_case(same, L, 300, 1, L, None, "all equal")
    two = torch.where(torch.arange(L * H, device=DEV).reshape(L, H) % 3 == 0, 2.0, -2.0).to(torch.bfloat16)
    direct_case(two, L, 777, 1, L, None, "two signs")
    asc = (torch.arange(L * H, device=DEV, dtype=torch.float32).reshape(L, H) / 64).to(torch.bfloat16)
    direct_case(asc, L, 512, 1, L, None, "ascending")


def test_rising_magnitudes_outgrow_the_candidate_buffer():
    # every element reaches the running threshold: the one-pass selection gives up and the
    # two-pass selection takes the chunk; a second, ordinary chunk rides along
    H, L, k = 4096, 32, 512
    rising = (torch.arange(L * H, device=DEV, dtype=torch.float32).reshape(L, H) / 256 + 1).to(torch.bfloat16)
    usual = synth.make_activations(1, L, H, torch.bfloat16, seed=77, device=DEV, outliers="none")
    act = torch.cat([rising, usual]).contiguous()
    direct_case(act, L, k, 2, L, {"falling": torch.cat([rising.flip(0).flip(1), usual]).contiguous()}, "rising")


def test_many_equal_values_go_to_the_rescue_launch():
    """k above 512 on chunks of the 70B shape: a chunk of equal magnitudes makes every element a
    candidate, which outgrows the half-block kernel's buffer; that chunk is marked and taken by
    the rescue launch of the same call, its ordinary neighbours are not."""
    H, L, k = 8192, 32, 1024
    usual = synth.make_activations(2, L, H, torch.bfloat16, seed=78, device=DEV, outliers="none")
    flat = torch.where(torch.arange(L * H, device=DEV).reshape(L, H) % 5 == 0, -3.0, 3.0).to(torch.bfloat16)
    act = torch.cat([usual[:L], flat, usual[L:]]).contiguous()
    out = direct_case(act, L, k, 3, L, {"noise": synth.honest_noise(act, seed=4)}, "equal values, k=1024")
    assert out["same"]["status"].tolist() == [0, 0, 0] and (out["same"]["accept"] == 1).all()
    direct_case(act, L, 4096, 3, L, None, "equal values, k=4096")
    f = act.float()
    direct_case(f, L, 2048, 3, L, None, "equal values, fp32")


@pytest.mark.parametrize("k", [200, 300, 1000])
def test_special_patterns(k):
    H, L = 512, 8
    bits = torch.randint(0, 65536, (L, H), dtype=torch.int32, device=DEV).to(torch.int16)  # NaN, Inf, subnormals
    act = bits.view(torch.bfloat16)
    direct_case(act, L, k, 1, L, None, "random patterns k=%d" % k)


@pytest.mark.parametrize("scale", [2.0 ** -40, 2.0 ** -18, 2.0 ** 9, 2.0 ** 30])
def test_magnitudes_far_from_one(scale):
    # the one-pass selection for k > 256 keeps a coarse byte per 8 elements that covers 2^-20 .. 2^12:
    # chunks that lie below, across the lower edge, across the upper edge and above the window
    S, T, H, L = 2, 64, 2048, 32
    base = synth.make_activations(S, T, H, torch.bfloat16, seed=97, device=DEV, outliers="jitter")
    act = (base.to(torch.float32) * scale).to(torch.bfloat16)
    for k in (300, 1024):
        direct_case(act, L, k, S, T, {"noise": synth.honest_noise(act, seed=6)}, "scale %g k=%d" % (scale, k))
    f = (synth.make_activations(S, T, H, torch.float32, seed=98, device=DEV, outliers="none") * scale).contiguous()
    direct_case(f, L, 600, S, T, None, "fp32 scale %g" % scale)


def test_odd_shapes_take_the_scalar_path():
    # hidden not a multiple of the vector width, and a strided view
    S, T, H, L, k = 2, 24, 1003, 8, 333
    act = synth.make_activations(S, T, H, torch.bfloat16, seed=71, device=DEV, outliers="none")
    direct_case(act, L, k, S, T, None, "H=1003")
    wide = synth.make_activations(S, T, 1024 + 64, torch.bfloat16, seed=72, device=DEV, outliers="none")
    view = wide[:, :1024]
    direct_case(view, L, k, S, T, None, "strided rows")
    f = synth.make_activations(S, T, 1001, torch.float32, seed=73, device=DEV, outliers="none")
    direct_case(f, L, 100, S, T, None, "fp32 H=1001")


def test_fewer_vectors_than_k():
    # 512 elements per chunk = 64 vectors of eight: k = 300 and k = 512 (every element) exceed the
    # number of vectors, so no threshold can come from the vectors' maxima
    S, T, H, L = 2, 16, 64, 8
    act = synth.make_activations(S, T, H, torch.bfloat16, seed=83, device=DEV, outliers="none")
    for k in (300, 512):
        direct_case(act, L, k, S, T, {"noise": synth.honest_noise(act, seed=4)}, "64 vectors, k=%d" % k)
    f = synth.make_activations(S, T, 128, torch.float32, seed=84, device=DEV, outliers="none")
    direct_case(f, 4, 400, S, T, None, "fp32: 128 vectors, k=400")


def test_chunk_smaller_than_k_and_malformed_commitments():
    S, T, H, L, k = 1, 10, 64, 4, 200      # chunks of 256, 256 and 128 elements
    act = synth.make_activations(S, T, H, torch.bfloat16, seed=81, device=DEV, outliers="none")
    out = direct_case(act, L, k, S, T, None, "short last chunk")
    assert out["same"]["status"].tolist() == [0, 0, 2]   # the last one: TOPLOC_CHUNK_K_EXCEEDS_CHUNK
    lay, _ = tl.make_layout(act, L, k, S, T)
    commits, _ = tl.toploc_commit_direct(act, lay)
    host = commits.cpu().numpy().copy()
    host[0, 6:12], host[0, 12:18] = host[0, 12:18].copy(), host[0, 6:12].copy()   # two records swapped
    host[1, 6 * (k - 1) + 2] = 0xFF                                                  # an index beyond the chunk
    bad = torch.from_numpy(host).to(DEV)
    res, dev = tl.toploc_verify_direct(act, lay, bad)
    torch.cuda.synchronize()
    got = res.cpu().numpy().view(tl.RESULT_DTYPE).reshape(-1)
    ref, ref_dev = oracle.verify_direct(synth.host_patterns(act), host, L, k, S, T, **oracle_thresholds(k))
    assert ref["status"].tolist() == [3, 3, 2]
    assert_results_equal(got, ref, "malformed")
    assert np.array_equal(dev.cpu().numpy().astype(np.uint32), ref_dev)


def test_argument_errors_come_back_before_any_launch():
    act = torch.zeros((64, 256), dtype=torch.bfloat16, device=DEV)
    lay, _ = tl.make_layout(act, 32, tl.TOPLOC_MAX_K_DIRECT + 1, 1, 64)
    with pytest.raises(tl.ToplocError, match="unsupported"):
        tl.toploc_commit_direct(act, lay)
    offs = np.array([0, 64], np.int64)
    lay, keep = tl.make_layout(act, 32, 16, 1, 0, seq_offsets=offs)
    lay.tokens_per_seq = 64
    with pytest.raises(tl.ToplocError, match="unsupported"):
        tl.toploc_commit_direct(act, lay)
    lay, _ = tl.make_layout(act, 32, 16, 1, 64)
    lib = tl.load_library()
    assert lib.toploc_commit_direct(None, ctypes.byref(lay), None, None, None) == -1


def test_agrees_with_the_proof_path_selection():
    """Same top-k as toploc_build_proofs (its optional index output, as a set)."""
    S, T, H, L, k = 4, 64, 4096, 32, 256
    act = synth.make_activations(S, T, H, torch.bfloat16, seed=91, device=DEV, outliers="jitter")
    lay, _ = tl.make_layout(act, L, k, S, T)
    _, _, indices = tl.toploc_build_proofs(act, lay, want_indices=True)
    commits, _ = tl.toploc_commit_direct(act, lay)
    torch.cuda.synchronize()
    rec = commits.cpu().numpy().reshape(-1, k, 6).astype(np.int64)
    idx = rec[..., 0] | (rec[..., 1] << 8) | (rec[..., 2] << 16) | (rec[..., 3] << 24)
    assert np.array_equal(idx, np.sort(indices.cpu().numpy().astype(np.int64), axis=1))
