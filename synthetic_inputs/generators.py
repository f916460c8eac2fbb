"""Counter-based, integer-only generators of the synthetic workloads.

Recipe (stated once here, relied on by the tests and the bench):

* ``hash_u64(seed, tensor_id, index)`` is the splitmix64 finaliser applied to
  ``index + tensor_id * 2**40 + seed * 0x9E3779B97F4A7C15`` (mod 2**64).
* A "normal" sample is an Irwin-Hall sum: the four 16-bit lanes of the hash are
  added, centred (minus 2*65535) and multiplied by ``sigma / sqrt(4*(2**32-1)/12)``
  as ONE fp32 multiply of an exactly representable integer, so CPU and CUDA
  produce the same bits.  bf16 tensors are that fp32 value rounded to nearest
  even with integer arithmetic on the bit pattern.
* Token ids are ``(hash >> 1) % vocab``.
* A skip mask marks as skipped (1) the sublayers with the smallest hash keys;
  sublayer ``2*l`` is the attention sublayer of layer ``l`` and ``2*l + 1`` its
  MLP sublayer.

Nothing here implements a step of the decoding method.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

_M64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_MIX1 = 0xBF58476D1CE4E5B9
_MIX2 = 0x94D049BB133111EB


def _s64(v: int) -> int:
    """Two's-complement reinterpretation of an unsigned 64-bit Python int."""
    v &= _M64
    return v - (1 << 64) if v >= (1 << 63) else v


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of int64 bit patterns."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def hash_u64(seed: int, tensor_id: int, index: torch.Tensor) -> torch.Tensor:
    """splitmix64 finaliser of the (seed, tensor_id, index) counter, as int64 bits."""
    assert index.dtype == torch.int64
    base = _s64((tensor_id << 40) + seed * _GOLDEN)
    z = index + base
    z = (z ^ _lsr(z, 30)) * _s64(_MIX1)
    z = (z ^ _lsr(z, 27)) * _s64(_MIX2)
    return z ^ _lsr(z, 31)


def hash_u64_int(seed: int, tensor_id: int, index: int) -> int:
    """Same hash for one Python int (used by the host-side stream generator)."""
    z = (index + (tensor_id << 40) + seed * _GOLDEN) & _M64
    z = ((z ^ (z >> 30)) * _MIX1) & _M64
    z = ((z ^ (z >> 27)) * _MIX2) & _M64
    return z ^ (z >> 31)


_IH_SIGMA = math.sqrt(4.0 * ((1 << 32) - 1) / 12.0)  # std of the sum of four uniform 16-bit lanes


def normal_f32(seed: int, tensor_id: int, index: torch.Tensor, sigma: float) -> torch.Tensor:
    h = hash_u64(seed, tensor_id, index)
    s = (h & 0xFFFF) + (_lsr(h, 16) & 0xFFFF) + (_lsr(h, 32) & 0xFFFF) + (_lsr(h, 48) & 0xFFFF)
    c = (s - 2 * 65535).to(torch.float32)
    scale = float(np.float32(sigma / _IH_SIGMA))
    return c * scale


def f32_to_bf16_bits(x: torch.Tensor) -> torch.Tensor:
    """Round-to-nearest-even fp32 -> bf16, integer arithmetic on the bits (finite inputs)."""
    b = x.contiguous().view(torch.int32).to(torch.int64) & 0xFFFFFFFF
    r = b + 0x7FFF + ((b >> 16) & 1)
    return ((r >> 16) & 0xFFFF).to(torch.int32).to(torch.int16)


def bf16_bits_to_f32(b: torch.Tensor) -> torch.Tensor:
    w = (b.to(torch.int64) & 0xFFFF) << 16
    w = torch.where(w >= (1 << 31), w - (1 << 32), w)
    return w.to(torch.int32).view(torch.float32)


def normal_weight(seed: int, tensor_id: int, rows: int, cols: int, sigma: float,
                  dtype: str, device="cpu", chunk_elems: int = 1 << 25) -> torch.Tensor:
    """[rows][cols] row-major tensor of N(0, sigma) samples; dtype 'fp32' or 'bf16'."""
    out_dtype = torch.float32 if dtype == "fp32" else torch.bfloat16
    out = torch.empty((rows, cols), dtype=out_dtype, device=device)
    rows_per = max(1, chunk_elems // cols)
    for r0 in range(0, rows, rows_per):
        r1 = min(rows, r0 + rows_per)
        idx = torch.arange(r0 * cols, r1 * cols, dtype=torch.int64, device=device)
        v = normal_f32(seed, tensor_id, idx, sigma)
        if dtype == "fp32":
            out[r0:r1] = v.view(r1 - r0, cols)
        else:
            out[r0:r1] = f32_to_bf16_bits(v).view(torch.bfloat16).view(r1 - r0, cols)
    return out


def uniform_tokens(seed: int, stream_id: int, n: int, vocab: int, device="cpu") -> torch.Tensor:
    idx = torch.arange(n, dtype=torch.int64, device=device)
    h = hash_u64(seed, TensorId.PROMPT + stream_id, idx)
    return (_lsr(h, 1) % vocab).to(torch.int32)


def uniforms(seed: int, stream_id: int, n: int) -> np.ndarray:
    """n uniforms in [0, 1) as fp64 multiples of 2**-24 (exactly representable in fp32 too): the top 24 bits of the
    hash of (seed, UNIFORM + stream_id, index).  The random draws a sampling method consumes are handed to it as inputs."""
    return np.array([(hash_u64_int(seed, TensorId.UNIFORM + stream_id, i) >> 40) / float(1 << 24) for i in range(n)],
                    dtype=np.float64)


def _ranks(seed: int, tensor_id: int, n: int) -> np.ndarray:
    keys = [hash_u64_int(seed, tensor_id, j) for j in range(n)]
    return np.argsort(np.array(keys, dtype=np.uint64), kind="stable")


def skip_mask(seed: int, n_sublayers: int, n_skip: int) -> np.ndarray:
    """uint8[n_sublayers]; 1 = skipped while drafting."""
    z = np.zeros(n_sublayers, dtype=np.uint8)
    z[_ranks(seed, TensorId.MASK, n_sublayers)[:n_skip]] = 1
    return z


def skip_mask_split(seed: int, n_layers: int, n_attn_skip: int, n_mlp_skip: int) -> np.ndarray:
    """Mask with a prescribed number of skipped attention and skipped MLP sublayers."""
    z = np.zeros(2 * n_layers, dtype=np.uint8)
    order = _ranks(seed, TensorId.MASK, 2 * n_layers)
    z[[j for j in order if j % 2 == 0][:n_attn_skip]] = 1
    z[[j for j in order if j % 2 == 1][:n_mlp_skip]] = 1
    return z


def nested_skip_masks(seed: int, n_layers: int, n_domains: int, pool_attn: int, pool_mlp: int,
                      n_attn_skip: int, n_mlp_skip: int):
    """Per-domain masks drawn from one common pool of skippable sublayers.

    Returns (pool, masks): ``pool`` uint8[2L] marks pool_attn attention and pool_mlp MLP sublayers; each of the
    ``n_domains`` rows of ``masks`` skips n_attn_skip attention and n_mlp_skip MLP sublayers chosen (by seeded rank)
    inside the pool, so the domains' masks differ but share the sublayers that matter to none of them."""
    pool = skip_mask_split(seed, n_layers, pool_attn, pool_mlp)
    masks = np.zeros((n_domains, 2 * n_layers), dtype=np.uint8)
    for i in range(n_domains):
        order = _ranks(seed + 1 + i, TensorId.MASK, 2 * n_layers)
        masks[i, [j for j in order if pool[j] and j % 2 == 0][:n_attn_skip]] = 1
        masks[i, [j for j in order if pool[j] and j % 2 == 1][:n_mlp_skip]] = 1
    return pool, masks


def domain_centroids(seed: int, n_domains: int, d: int) -> torch.Tensor:
    idx = torch.arange(n_domains * d, dtype=torch.int64)
    return normal_f32(seed, TensorId.CENTROID, idx, 1.0).view(n_domains, d)


def anchors(seed: int, n_domains: int, per_domain: int, d: int, sigma_a: float,
            normalise: bool = True, clustered: bool = True) -> torch.Tensor:
    """fp32 [n_domains*per_domain][d].  clustered: centroid + sigma_a * noise; else plain Gaussian."""
    n = n_domains * per_domain
    idx = torch.arange(n * d, dtype=torch.int64)
    noise = normal_f32(seed, TensorId.ANCHOR, idx, 1.0).view(n, d).to(torch.float64)
    if clustered:
        c = domain_centroids(seed, n_domains, d).to(torch.float64)
        a = c.repeat_interleave(per_domain, dim=0) + sigma_a * noise
    else:
        a = noise
    if normalise:
        a = a / a.norm(dim=1, keepdim=True)
    return a.to(torch.float32).contiguous()


def request_stream(seed: int, n_domains: int, per_domain: int, r: float) -> List[int]:
    """Domain label of each request: a chain that changes domain with probability r.

    With N domains the next request stays in the current domain with probability
    1 - r and moves to each other domain with probability r / (N - 1).  Each domain
    has a quota of ``per_domain`` requests; once a domain is used up the law is
    renormalised over the domains that still have requests left.
    """
    left = [per_domain] * n_domains
    total = n_domains * per_domain
    out: List[int] = []
    cur = hash_u64_int(seed, TensorId.STREAM, 0) % n_domains
    for i in range(total):
        if i > 0:
            u = (hash_u64_int(seed, TensorId.STREAM, i) >> 11) / float(1 << 53)
            w = [0.0] * n_domains
            for j in range(n_domains):
                if left[j] == 0:
                    continue
                w[j] = (1.0 - r) if j == cur else r / (n_domains - 1)
            tot = sum(w)
            if tot <= 0.0:  # only the current, forbidden-by-r domain is left (r == 1): take what remains
                w = [1.0 if left[j] else 0.0 for j in range(n_domains)]
                tot = sum(w)
            acc, pick = 0.0, None
            for j in range(n_domains):
                if w[j] == 0.0:
                    continue
                acc += w[j] / tot
                pick = j
                if u < acc:
                    break
            cur = pick
        out.append(cur)
        left[cur] -= 1
    return out


def prompt_lengths(seed: int, n: int, lo: int, hi: int) -> List[int]:
    return [lo + hash_u64_int(seed, TensorId.LENGTH, i) % (hi - lo + 1) for i in range(n)]


class TensorId:
    EMBED = 1
    FINAL_NORM = 2
    LM_HEAD = 3
    ANCHOR = 4
    CENTROID = 5
    MASK = 6
    STREAM = 7
    LENGTH = 8
    LAYER0 = 64          # layer l uses LAYER0 + 8*l + {0 wq, 1 wk, 2 wv, 3 wo, 4 gate, 5 up, 6 down, 7 gains}
    UNIFORM = 1 << 19    # + stream id
    PROMPT = 1 << 20     # + stream id


@dataclass(frozen=True)
class ModelShape:
    name: str
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    vocab: int
    dtype: str           # 'fp32' or 'bf16' (weights and KV cache)
    rms_eps: float
    rope_theta: float
    sigma: float = 0.02

    def with_layers(self, n_layers: int) -> "ModelShape":
        return replace(self, n_layers=n_layers, name=f"{self.name}-L{n_layers}")


SHAPES: Dict[str, ModelShape] = {
    # the five workload shapes, in the order the workloads are named
    "tiny": ModelShape("tiny", 4, 256, 4, 4, 64, 688, 1024, "fp32", 1e-5, 10000.0),
    "llama7b": ModelShape("llama7b", 32, 4096, 32, 32, 128, 11008, 32000, "bf16", 1e-5, 10000.0),
    "llama13b": ModelShape("llama13b", 40, 5120, 40, 40, 128, 13824, 32000, "bf16", 1e-5, 10000.0),
    "qwen14b": ModelShape("qwen14b", 48, 5120, 40, 8, 128, 13824, 152064, "bf16", 1e-6, 1000000.0),
    # small ragged shapes for kernel parity tests (odd row counts, GQA, several tiles + a tail)
    "ragged-bf16": ModelShape("ragged-bf16", 3, 320, 5, 5, 64, 872, 1000, "bf16", 1e-5, 10000.0),
    "gqa-bf16": ModelShape("gqa-bf16", 2, 512, 8, 2, 64, 1384, 2056, "bf16", 1e-6, 1000000.0),
    # every linear of this one has n_in % 128 == 0 (the streaming kernel's path), ragged row counts, two column tiles
    "stream-bf16": ModelShape("stream-bf16", 3, 768, 6, 2, 128, 1920, 3001, "bf16", 1e-5, 10000.0),
    # the same with 64-wide heads and four query heads per K/V head
    "stream64-bf16": ModelShape("stream64-bf16", 2, 512, 8, 2, 64, 1408, 2056, "bf16", 1e-6, 1000000.0),
    "gqa-fp32": ModelShape("gqa-fp32", 2, 256, 4, 2, 64, 688, 520, "fp32", 1e-6, 1000000.0),
}


def _gain(seed: int, tensor_id: int, offset: int, d: int, spread: float, device) -> torch.Tensor:
    if spread == 0.0:
        return torch.ones(d, dtype=torch.float32, device=device)
    idx = torch.arange(offset, offset + d, dtype=torch.int64, device=device)
    return (1.0 + normal_f32(seed, tensor_id, idx, spread)).contiguous()


def make_model_weights(shape: ModelShape, seed: int, device="cpu",
                       damp: Optional[Dict[int, float]] = None,
                       gain_spread: float = 0.0) -> Dict[str, object]:
    """Random-init weights of a LLaMA-style decoder, N(0, shape.sigma), gains = 1.

    ``damp`` maps a sublayer index (2l attention, 2l+1 MLP) to a factor applied to
    the standard deviation of that sublayer's OUTPUT projection (W_o or W_down):
    the "acceptance-shaped" variant in which the sublayers a mask skips matter
    little, as the method presumes of a domain's skippable layers.
    ``gain_spread`` > 0 replaces the unit RMSNorm gains by 1 + N(0, gain_spread)
    (parity tests use it so that a dropped gain cannot go unnoticed).
    """
    damp = damp or {}
    dt, s = shape.dtype, shape.sigma
    d, hq, hkv, f = shape.d_model, shape.n_heads * shape.head_dim, shape.n_kv_heads * shape.head_dim, shape.d_ff
    w: Dict[str, object] = {
        "tok_embed": normal_weight(seed, TensorId.EMBED, shape.vocab, d, s, dt, device),
        "lm_head": normal_weight(seed, TensorId.LM_HEAD, shape.vocab, d, s, dt, device),
        "final_norm": _gain(seed, TensorId.FINAL_NORM, 0, d, gain_spread, device),
    }
    names = ["attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down"]
    for n in names:
        w[n] = []
    for l in range(shape.n_layers):
        t = TensorId.LAYER0 + 8 * l
        w["attn_norm"].append(_gain(seed, t + 7, 0, d, gain_spread, device))
        w["mlp_norm"].append(_gain(seed, t + 7, d, d, gain_spread, device))
        w["wq"].append(normal_weight(seed, t + 0, hq, d, s, dt, device))
        w["wk"].append(normal_weight(seed, t + 1, hkv, d, s, dt, device))
        w["wv"].append(normal_weight(seed, t + 2, hkv, d, s, dt, device))
        w["wo"].append(normal_weight(seed, t + 3, d, hq, s * damp.get(2 * l, 1.0), dt, device))
        w["w_gate"].append(normal_weight(seed, t + 4, f, d, s, dt, device))
        w["w_up"].append(normal_weight(seed, t + 5, f, d, s, dt, device))
        w["w_down"].append(normal_weight(seed, t + 6, d, f, s * damp.get(2 * l + 1, 1.0), dt, device))
    return w
