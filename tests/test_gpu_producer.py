"""The producer-side hook (Section 5.5: the proof is taken inside the engine, from the kernel that
writes the last hidden states): a final RMSNorm that offers its output tile to the running top-k
while the tile is still in shared memory.  The proofs must equal the oracle's over the rows the
producer wrote, and those of the other two generation paths."""
import numpy as np
import pytest
import torch

import oracle
import paper_2501_16007_b200 as tl
from paper_2501_16007_b200 import synth
from helpers import assert_build_equal

pytestmark = pytest.mark.gpu
DEV = "cuda"


def decode_with_fused_commit(x, weight, eps, num_seqs, tokens, k, pad=0):
    """x: [num_seqs * tokens, hidden] pre-norm hidden states.  Step t normalises row t of every
    sequence; returns (proofs, status, indices) and the normalised rows [num_seqs * tokens, hidden]."""
    hidden = x.shape[1]
    y_all = torch.empty_like(x)
    step_x = torch.empty((num_seqs, hidden + pad), dtype=x.dtype, device=x.device)[:, :hidden]
    step_y = torch.empty((num_seqs, hidden + pad), dtype=x.dtype, device=x.device)[:, :hidden]
    lay, _ = tl.make_layout(step_y, tokens, k, num_seqs, 1)
    lay.row_stride = hidden + pad
    state = torch.empty(tl.toploc_stream_state_bytes(lay), dtype=torch.uint8, device=x.device)
    tl.toploc_stream_begin(state, lay)
    xs, ys = x.view(num_seqs, tokens, hidden), y_all.view(num_seqs, tokens, hidden)
    for t in range(tokens):
        step_x.copy_(xs[:, t, :])
        tl.toploc_rmsnorm_append(step_x, weight, eps, lay, t, step_y, state)
        ys[:, t, :].copy_(step_y)
    out = tl.toploc_stream_finish(state, lay, want_indices=True)
    torch.cuda.synchronize()
    return out, y_all


@pytest.mark.parametrize("hidden,tokens,k,pad,outliers", [
    (4096, 32, 128, 0, "fixed"),      # the paper's interval at the 8B hidden size
    (8192, 32, 128, 0, "jitter"),     # 70B hidden size
    (2048, 32, 256, 8, "none"),       # padded step buffers
    (4096, 16, 512, 0, "jitter"),     # the largest k
    (1000, 5, 64, 0, "none"),         # rows that are not a multiple of 32 vectors
    (64, 3, 256, 0, "none"),          # fewer than k elements in the whole chunk: status, zero proof
])
def test_fused_norm_commits_what_it_writes(hidden, tokens, k, pad, outliers):
    S, eps = 6, 1e-5
    x = synth.make_activations(S, tokens, hidden, torch.bfloat16, seed=hidden + k, device=DEV, outliers=outliers)
    g = torch.Generator(device=DEV)
    g.manual_seed(7)
    weight = (1.0 + 0.1 * torch.randn(hidden, generator=g, device=DEV)).to(torch.bfloat16)
    fused, y = decode_with_fused_commit(x, weight, eps, S, tokens, k, pad=pad)
    # the normalisation itself, against fp32 torch: within one bf16 rounding step of the exact value
    xf = x.float()
    want = xf * torch.rsqrt(xf.pow(2).mean(dim=1, keepdim=True) + eps) * weight.float()
    err = (y.float() - want).abs()
    assert (err <= want.abs() * 2.0 ** -7 + 1e-30).all(), float(err.max())
    # parity: the oracle on the bytes the producer wrote
    ref = oracle.build_proofs(synth.host_patterns(y), tokens, k, S, tokens)
    assert_build_equal(fused, ref, "fused norm vs oracle")
    # and the same bytes through the batch path
    lay, _ = tl.make_layout(y, tokens, k, S, tokens)
    batch = tl.toploc_build_proofs(y, lay, want_indices=True)
    torch.cuda.synchronize()
    for a, b in zip(fused, batch):
        assert torch.equal(a, b)


def test_norm_alone_and_refusals():
    S, hidden = 4, 1024
    x = synth.make_activations(S, 1, hidden, torch.bfloat16, seed=3, device=DEV)
    weight = torch.ones(hidden, dtype=torch.bfloat16, device=DEV)
    y = torch.empty_like(x)
    lay, _ = tl.make_layout(y, 32, 128, S, 1)
    tl.toploc_rmsnorm_append(x, weight, 1e-6, lay, 0, y, None)            # no state: a plain RMSNorm
    torch.cuda.synchronize()
    xf = x.float()
    want = xf * torch.rsqrt(xf.pow(2).mean(dim=1, keepdim=True) + 1e-6)
    assert ((y.float() - want).abs() <= want.abs() * 2.0 ** -7).all()
    with pytest.raises(tl.ToplocError, match="invalid argument"):
        tl.toploc_rmsnorm_append(x, weight, 1e-6, lay, 32, y, None)        # token beyond the chunk
    odd = torch.empty((S, 1001), dtype=torch.bfloat16, device=DEV)[:, :1000]
    lay_odd, _ = tl.make_layout(odd, 32, 64, S, 1)
    lay_odd.row_stride = 1001
    with pytest.raises(tl.ToplocError, match="unsupported"):
        tl.toploc_rmsnorm_append(odd, weight[:1000].contiguous(), 1e-6, lay_odd, 0, odd, None)
