"""Incremental proof generation (one row per sequence and decode step) against the oracle and
against toploc_build_proofs over the assembled chunks: the same bytes, statuses and indices."""
import numpy as np
import pytest
import torch

import oracle
import paper_2501_16007_b200 as tl
from paper_2501_16007_b200 import synth
from helpers import assert_build_equal

pytestmark = pytest.mark.gpu
DEV = "cuda"


def stream_chunks(act, num_seqs, tokens, k, field=0, pad=0):
    """Feeds the [num_seqs * tokens, hidden] batch row by row, as a decoder would: step t hands over
    row t of every sequence in a fresh [num_seqs, hidden (+ pad)] buffer."""
    hidden = act.shape[1]
    step_buf = torch.empty((num_seqs, hidden + pad), dtype=act.dtype, device=act.device)
    rows = step_buf[:, :hidden]
    lay, _ = tl.make_layout(rows, tokens, k, num_seqs, 1, field=field)    # one row per sequence and step
    lay.row_stride = hidden + pad
    state = torch.empty(tl.toploc_stream_state_bytes(lay), dtype=torch.uint8, device=act.device)
    tl.toploc_stream_begin(state, lay)
    by_seq = act.view(num_seqs, tokens, hidden)
    for t in range(tokens):
        rows.copy_(by_seq[:, t, :])
        tl.toploc_stream_append(rows, lay, t, state)
    out = tl.toploc_stream_finish(state, lay, want_indices=True)
    torch.cuda.synchronize()
    return out


@pytest.mark.parametrize("dtype,field,hidden,tokens,k,outliers", [
    (torch.bfloat16, 0, 4096, 32, 128, "fixed"),     # the paper's interval; ties at the top decided by index
    (torch.bfloat16, 0, 2048, 32, 128, "none"),
    (torch.bfloat16, 0, 1000, 7, 64, "jitter"),      # rows that are not a multiple of 32 vectors
    (torch.bfloat16, 0, 97, 12, 256, "none"),        # unaligned rows: element-wise loads
    (torch.float32, 0, 2048, 32, 128, "jitter"),
    (torch.float32, 1, 2048, 32, 128, "jitter"),     # whole patterns over the 32-bit field
    (torch.bfloat16, 0, 64, 3, 256, "none"),         # fewer than k elements: status, zero proof
    (torch.bfloat16, 0, 2048, 32, 512, "jitter"),    # the largest k
])
def test_streamed_chunks_equal_the_batch_path_and_the_oracle(dtype, field, hidden, tokens, k, outliers):
    S = 5
    act = synth.make_activations(S, tokens, hidden, dtype, seed=hidden + tokens, device=DEV, outliers=outliers)
    streamed = stream_chunks(act, S, tokens, k, field=field)
    ref = oracle.build_proofs(synth.host_patterns(act), tokens, k, S, tokens, wide=bool(field))
    assert_build_equal(streamed, ref, "streamed vs oracle")
    lay, _ = tl.make_layout(act, tokens, k, S, tokens, field=field)
    batch = tl.toploc_build_proofs(act, lay, want_indices=True)
    torch.cuda.synchronize()
    for a, b in zip(streamed, batch):
        assert torch.equal(a, b)


def test_padded_step_buffers_growing_values_and_reuse_of_the_state():
    S, tokens, hidden, k = 3, 32, 512, 128
    # magnitudes grow with the token index: every step replaces most of the running selection
    act = synth.make_activations(S, tokens, hidden, torch.bfloat16, seed=9, device=DEV, outliers="none")
    scale = torch.arange(1, tokens + 1, device=DEV, dtype=torch.float32).repeat(S).unsqueeze(1)
    act = (act.float() * scale).to(torch.bfloat16)
    ref = oracle.build_proofs(synth.host_patterns(act), tokens, k, S, tokens)
    assert_build_equal(stream_chunks(act, S, tokens, k, pad=8), ref, "padded step buffer")
    assert_build_equal(stream_chunks(act, S, tokens, k, pad=3), ref, "unaligned step buffer")   # 6-byte offset rows
    # one state, two chunks in a row: begin() starts afresh
    rows = torch.empty((S, hidden), dtype=torch.bfloat16, device=DEV)
    lay, _ = tl.make_layout(rows, tokens, k, S, 1)
    state = torch.empty(tl.toploc_stream_state_bytes(lay), dtype=torch.uint8, device=DEV)
    other = synth.make_activations(S, tokens, hidden, torch.bfloat16, seed=10, device=DEV, outliers="jitter")
    for data in (other, act):
        tl.toploc_stream_begin(state, lay)
        for t in range(tokens):
            rows.copy_(data.view(S, tokens, hidden)[:, t, :])
            tl.toploc_stream_append(rows, lay, t, state)
    out = tl.toploc_stream_finish(state, lay, want_indices=True)
    torch.cuda.synchronize()
    assert_build_equal(out, ref, "state reused")


def test_refusals():
    rows = torch.zeros((2, 4096), dtype=torch.bfloat16, device=DEV)
    lay, _ = tl.make_layout(rows, 32, 128, 2, 1)
    state = torch.empty(tl.toploc_stream_state_bytes(lay), dtype=torch.uint8, device=DEV)
    assert tl.toploc_stream_state_bytes(lay) == 2 * (16 + 8 * 128)
    tl.toploc_stream_begin(state, lay)
    with pytest.raises(tl.ToplocError, match="invalid argument"):
        tl.toploc_stream_append(rows, lay, 32, state)                       # beyond chunk_len
    with pytest.raises(tl.ToplocError, match="workspace"):
        tl.toploc_stream_finish(state, lay, workspace=torch.empty(64, dtype=torch.uint8, device=DEV))
    big, _ = tl.make_layout(rows, 8192, 128, 2, 1)                          # 8192 * 4096 > 2^24
    assert tl.toploc_stream_state_bytes(big) == 0
    with pytest.raises(tl.ToplocError, match="unsupported"):
        tl.toploc_stream_begin(state, big)
