"""Seeded synthetic activations shaped like an LLM's last hidden states, and the
perturbations the validation cases apply to them.

This module serves both the CUDA path and the CPU oracle with identical bytes
(the oracle receives a host copy of whatever tensor is produced here).  It holds
none of the proof arithmetic -- only random draws, casts and row shuffles.

Recipe (stands in for last-layer activations of Llama-3.1-8B / 70B on chat
prompts, which are not available offline): every element is 0.5 x Student-t with
3 degrees of freedom, rounded to the storage type; a few fixed "massive
activation" channels are overwritten at every token with magnitude 80 and a
random sign.  Shapes follow the models' hidden sizes (4096 and 8192) and the
32-token proof interval.
"""
import numpy as np
import torch

_SEQ_STRIDE = 1_000_003


def default_outlier_channels(hidden):
    """Channels 0..3 up to H = 4096; for wider models four more at 4096..4099."""
    if hidden > 4096:
        return (0, 1, 2, 3, 4096, 4097, 4098, 4099)
    return tuple(c for c in (0, 1, 2, 3) if c < hidden)


def _generator(device, seed):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) & 0x7FFFFFFFFFFFFFFF)
    return g


def _student_t3(shape, g, device):
    z = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
    chi = torch.zeros(shape, device=device, dtype=torch.float32)
    for _ in range(3):
        w = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
        chi.addcmul_(w, w)
    return z * torch.rsqrt(chi / 3.0)


def make_activations(num_seqs, tokens_per_seq, hidden, dtype=torch.bfloat16, seed=0, device="cpu",
                     outliers="fixed", outlier_channels=None, out=None):
    """[num_seqs * tokens_per_seq, hidden] tensor of `dtype` (bfloat16 or float32).

    outliers: "fixed"  -> +-80 on the outlier channels (the literal recipe),
              "jitter" -> 80 * (1 + 0.25 u), u ~ U(-1, 1), so the top-k varies per chunk,
              "none"   -> no outlier channels (pure heavy-tailed data),
              "rising" -> jittered outliers, and token t of a sequence scaled by 4 ** ((t mod 32) / 31):
                          magnitudes grow fourfold over every 32-token interval, so a running top-k
                          keeps admitting new elements to the end of a chunk.
    Each sequence draws from its own generator seeded with seed * 1000003 + sequence, so a
    sequence's bytes do not depend on the batch around it (on a given device type).
    """
    device = torch.device(device)
    total = num_seqs * tokens_per_seq
    if out is None:
        out = torch.empty((total, hidden), dtype=dtype, device=device)
    assert out.shape == (total, hidden) and out.dtype == dtype
    if outlier_channels is None:
        outlier_channels = default_outlier_channels(hidden)
    ch = torch.tensor(list(outlier_channels), device=device, dtype=torch.long)
    for s in range(num_seqs):
        g = _generator(device, seed * _SEQ_STRIDE + s)
        x = _student_t3((tokens_per_seq, hidden), g, device) * 0.5
        if outliers != "none" and len(outlier_channels) > 0:
            shape = (tokens_per_seq, len(outlier_channels))
            sign = torch.randint(0, 2, shape, generator=g, device=device).to(torch.float32) * 2.0 - 1.0
            mag = torch.full(shape, 80.0, device=device, dtype=torch.float32)
            if outliers in ("jitter", "rising"):
                u = torch.rand(shape, generator=g, device=device, dtype=torch.float32) * 2.0 - 1.0
                mag = mag * (1.0 + 0.25 * u)
            x[:, ch] = sign * mag
        if outliers == "rising":
            t = torch.arange(tokens_per_seq, device=device, dtype=torch.float32)
            x *= torch.pow(torch.tensor(4.0, device=device), (t % 32) / 31.0).unsqueeze(1)
        out[s * tokens_per_seq:(s + 1) * tokens_per_seq].copy_(x.to(dtype))
        del x
    return out


def honest_noise(act, seed, rel=2.0 ** -8, rows_per_step=1 << 14):
    """Recomputation noise of an honest validator: v * (1 + rel * xi), xi ~ U(-1, 1), in fp32,
    rounded back to the storage type."""
    out = torch.empty_like(act)
    g = _generator(act.device, seed * _SEQ_STRIDE + 777)
    for r in range(0, act.shape[0], rows_per_step):
        blk = act[r:r + rows_per_step].to(torch.float32)
        xi = torch.rand(blk.shape, generator=g, device=act.device, dtype=torch.float32) * 2.0 - 1.0
        out[r:r + rows_per_step].copy_((blk * (1.0 + rel * xi)).to(act.dtype))
    return out


def fp8_roundtrip(act, rows_per_step=1 << 14):
    """storage type -> fp8 e4m3 (round to nearest even, saturating at +-448) -> storage type."""
    out = torch.empty_like(act)
    for r in range(0, act.shape[0], rows_per_step):
        blk = act[r:r + rows_per_step].to(torch.float32).clamp_(-448.0, 448.0)
        out[r:r + rows_per_step].copy_(blk.to(torch.float8_e4m3fn).to(torch.float32).to(act.dtype))
    return out


def prefix_shift(act, other, num_seqs, tokens_per_seq, shift=16):
    """Row t of every sequence becomes row t - shift of the same sequence; the first `shift`
    rows come from `other` (activations of a different seed): a prepended-prompt proxy."""
    out = torch.empty_like(act)
    a = act.view(num_seqs, tokens_per_seq, -1)
    o = other.view(num_seqs, tokens_per_seq, -1)
    v = out.view(num_seqs, tokens_per_seq, -1)
    v[:, shift:].copy_(a[:, :tokens_per_seq - shift])
    v[:, :shift].copy_(o[:, :shift])
    return out


def plus_one_ulp(act, seed):
    """Adds 1 to the bit pattern of a seeded random half of the elements (bf16 only)."""
    assert act.dtype == torch.bfloat16
    g = _generator(act.device, seed * _SEQ_STRIDE + 555)
    bump = torch.randint(0, 2, act.shape, generator=g, device=act.device, dtype=torch.int16)
    return (act.view(torch.int16) + bump).view(torch.bfloat16)


def truncate_mantissa(act, keep_bits):
    """Clears all but the top `keep_bits` mantissa bits (bf16 only): a low-precision proxy."""
    assert act.dtype == torch.bfloat16
    mask = (~((1 << (7 - keep_bits)) - 1)) & 0xFFFF
    mask = mask - 0x10000 if mask >= 0x8000 else mask
    return (act.view(torch.int16) & mask).view(torch.bfloat16)


def host_patterns(act):
    """Host numpy view the oracle consumes: uint16 bit patterns for bf16, float32 otherwise."""
    t = act.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()
