"""Parity of the CUDA path with the oracle on chunks long enough to be selected in segments and
merged (a prompt processed as one chunk): more than 2^19 elements, and one beyond 2^24."""
import numpy as np
import pytest
import torch

import oracle
import paper_2501_16007_b200 as tl
from paper_2501_16007_b200 import synth
from helpers import parity_case, gpu_build, assert_build_equal

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("outliers", ["none", "fixed"])
def test_one_long_chunk(dtype, outliers):
    """700 rows x 4096 = 2.87 M elements: eleven segments.  With the outlier channels every row holds
    elements tied at the top, so the cut is decided by the flat index across segment borders."""
    act = synth.make_activations(1, 700, 4096, dtype, seed=31, device=DEV, outliers=outliers)
    rec = {"noise": synth.honest_noise(act, seed=32)}
    if dtype == torch.bfloat16:
        rec["ulp"] = synth.plus_one_ulp(act, seed=33)
    parity_case(act, 700, 128, 1, 700, recomputed=rec, where="long %s %s" % (dtype, outliers))


def test_ragged_batch_mixing_long_and_short_chunks():
    """Chunks of 1.4 M, 82 k, 2 M and 975 k elements, an empty sequence, k = 64; the recomputed copies
    include one from another seed (rejected) so the verdicts are not all alike."""
    lens = [700, 40, 0, 1500]
    offs = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    act = synth.make_activations(1, int(offs[-1]), 2048, torch.bfloat16, seed=34, device=DEV, outliers="jitter")
    other = synth.make_activations(1, int(offs[-1]), 2048, torch.bfloat16, seed=35, device=DEV, outliers="jitter")
    rec = {"noise": synth.honest_noise(act, seed=36), "other": other}
    _, out = parity_case(act, 1024, 64, len(lens), seq_offsets=offs, recomputed=rec, where="mixed")
    assert out["same"]["accept"].all() and not out["other"]["accept"].any()


def test_long_chunk_of_equal_values_keeps_the_first_indices():
    act = torch.full((600, 2048), 1.5, dtype=torch.bfloat16, device=DEV)
    lay, _ = tl.make_layout(act, 600, 128, 1, 600)
    proofs, status, indices = tl.toploc_build_proofs(act, lay, want_indices=True)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [0]
    assert indices.cpu().numpy().reshape(-1).tolist() == list(range(128))
    parity_case(act, 600, 128, 1, 600, where="equal")


def test_long_chunk_with_padded_rows_and_with_unaligned_rows():
    """Rows with padding between them (16-byte aligned) and rows of 97 elements (element-wise loads),
    k = 256."""
    base = synth.make_activations(1, 300, 4096 + 64, torch.bfloat16, seed=37, device=DEV, outliers="none")
    parity_case(base[:, :4096], 300, 256, 1, 300, where="padded")
    odd = synth.make_activations(1, 6000, 97, torch.float32, seed=38, device=DEV, outliers="none")
    parity_case(odd, 6000, 256, 1, 6000, where="unaligned")


def test_long_chunk_with_the_largest_k():
    """A prompt-sized chunk (selected in segments, merged) at k = 512: the segments and the merge
    take the larger scratch and sixteen points per lane."""
    act = synth.make_activations(1, 300, 4096, torch.bfloat16, seed=44, device=DEV, outliers="none")
    parity_case(act, 300, 512, 1, 300, where="long k512")


def test_selection_entry_point_on_a_long_chunk():
    act = synth.make_activations(1, 520, 4096, torch.float32, seed=39, device=DEV, outliers="none")
    lay, _ = tl.make_layout(act, 520, 128, 1, 520)
    idx, pat, status, ranked = tl.toploc_select_topk(act, lay, want_ranked=True)
    torch.cuda.synchronize()
    want_idx, want_bits = oracle.topk(synth.host_patterns(act), 128)
    assert status.cpu().tolist() == [0]
    assert ranked.cpu().numpy().reshape(-1).tolist() == want_idx.tolist()
    idx, pat = idx.cpu().numpy().reshape(-1), pat.cpu().numpy().view(np.uint16).reshape(-1)
    order, ref = np.argsort(idx), np.argsort(want_idx)
    assert idx[order].tolist() == want_idx[ref].tolist()            # same set ...
    assert pat[order].tolist() == want_bits[ref].tolist()           # ... with the same values


def test_chunk_beyond_two_to_the_24_elements():
    """4100 rows x 8192 = 33.6 M elements (a 4100-token prompt of a 70B-shaped model as one chunk),
    64 segments; proof, indices and the verdict on a noisy copy against the oracle."""
    act = synth.make_activations(1, 4100, 8192, torch.bfloat16, seed=40, device=DEV, outliers="jitter")
    rec = {"noise": synth.honest_noise(act, seed=41)}
    parity_case(act, 4100, 128, 1, 4100, recomputed=rec, where="33M")


def test_very_wide_rows_become_one_segment_each():
    """hidden = 2^20: 24 rows are 25 M elements; no segment may hold more than 2^24 of them, and none can
    split a row, so every row is a segment of its own (k = 64, fp32 committed as 16 bits)."""
    act = synth.make_activations(1, 24, 1 << 20, torch.float32, seed=43, device=DEV, outliers="none")
    parity_case(act, 24, 64, 1, 24, where="wide rows")


def test_host_buffer_entry_points_with_a_long_chunk():
    lens = [650, 64]
    offs = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    act = synth.make_activations(1, int(offs[-1]), 2048, torch.bfloat16, seed=42, device=DEV, outliers="none")
    g = gpu_build(act, 1024, 128, len(lens), seq_offsets=offs)
    lay, _keep = tl.make_layout(act, 1024, 128, len(lens), seq_offsets=offs)
    h_act = act.cpu().pin_memory()
    h_proofs = torch.empty((2, 258), dtype=torch.uint8).pin_memory()
    h_status = torch.empty((2,), dtype=torch.uint8).pin_memory()
    staging = torch.empty(tl.toploc_staging_bytes(lay), dtype=torch.uint8, device=DEV)   # one sequence at a time
    tl.toploc_build_proofs_host(h_act, lay, h_proofs, h_status, staging)
    assert torch.equal(h_proofs, g[0].cpu()) and torch.equal(h_status, g[1].cpu())
    h_res = torch.empty((2, 40), dtype=torch.uint8).pin_memory()
    tl.toploc_verify_proofs_host(h_act, lay, h_proofs, tl.default_thresholds(), h_res, staging)
    assert h_res.numpy().view(tl.RESULT_DTYPE).reshape(-1)["accept"].tolist() == [1, 1]
