"""Seeded synthetic workloads for SANTA++ decode attention.

This module only draws numbers and rounds them to bf16. It holds none of the
method's arithmetic and imports neither the CUDA binding nor the CPU oracle, so
both sides of a parity test can be fed from the same buffers.

The inputs stand in for the paper's captured Qwen2.5-7B-Instruct layer-14
workload (Appendix "Kernel evaluation protocol and profiling", paragraph
"Captured workload"), which is not available: same head layout (28 query heads
over 4 KV heads, head_dim 128), same context lengths, bf16 K/V.

Recipe (all draws from numpy's PCG64 `default_rng`, keyed by (seed, layer, tag)):
  keys     n_clusters centres c_j ~ N(0, I_d); row i picks a centre uniformly at
           random and k_i = c_j + 0.3 * eps_i; the first four prompt rows are
           "sink" keys, their vectors multiplied by 4
  values   v_i ~ N(0, I_d)
  suffix   rows drawn the same way as prompt rows (no sinks)
  queries  q = 2 * (k_j + 0.5 * eps) for a uniformly random prompt row j,
           independently per step, sequence and query head ("noisy copy");
           or, for the concentrated variant, q = alpha * (c_j + 0.5 * eps) with
           alpha bisected so the 64 largest softmax weights hold ~90 % of the mass
Everything is rounded to bf16 (round to nearest even) and handed out as uint16
bit patterns; `bf16_to_f64` widens them exactly.
"""
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

HEAD_DIM = 128


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest even); returns uint16 bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounding = ((b >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((b + rounding) >> np.uint32(16)).astype(np.uint16)


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float64."""
    return bf16_to_f32(bits).astype(np.float64)


def round_bits(x: np.ndarray, elem: str = "bf16") -> np.ndarray:
    """Round float32 to the 16-bit element type (nearest even); returns uint16 bit patterns."""
    if elem == "fp16":
        return np.ascontiguousarray(x, dtype=np.float32).astype(np.float16).view(np.uint16)
    return f32_to_bf16_bits(x)


def to_f32(bits: np.ndarray, elem: str = "bf16") -> np.ndarray:
    if elem == "fp16":
        return np.ascontiguousarray(bits, dtype=np.uint16).view(np.float16).astype(np.float32)
    return bf16_to_f32(bits)


def to_f64(bits: np.ndarray, elem: str = "bf16") -> np.ndarray:
    """Exact widening of 16-bit patterns of the given element type to float64."""
    return to_f32(bits, elem).astype(np.float64)


@dataclass
class WorkloadSpec:
    name: str
    n_seqs: int
    n_q_heads: int
    n_kv_heads: int
    prompt_len: List[int]            # per sequence
    n_clusters: int
    parent_size: int
    reps_per_parent: int
    n_sample: int                    # K, sampled teams per query head
    n_steps: int
    suffix_cap: int
    suffix_len0: List[int]           # suffix length at step 0, per sequence
    suffix_growth: int               # rows appended per step
    query_kind: str = "noisy_copy"   # or "concentrated"
    key_layout: str = "iid"          # cluster of each prompt row: "iid", or "runs" (geometric runs of one
                                     # cluster, mean length rows / clusters: positional locality)
    head_dim: int = HEAD_DIM
    seed: int = 0
    elem: str = "bf16"               # 16-bit element type the draws are rounded to: "bf16" or "fp16"

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def rows_total(self) -> int:
        return int(sum(self.prompt_len))

    def suffix_len(self, step: int) -> np.ndarray:
        s = np.asarray(self.suffix_len0, dtype=np.int64) + self.suffix_growth * step
        return np.minimum(s, self.suffix_cap).astype(np.int32)


def spec_tiny(seed: int = 0) -> WorkloadSpec:
    """Tiny reference: 1 query head, 1 KV head, 4096 keys + 16 suffix rows,
    64 clusters, parents of 256 with 16 representatives, 16 sampled teams."""
    return WorkloadSpec("tiny", 1, 1, 1, [4096], 64, 256, 16, 16, 32, 16, [16], 0, seed=seed)


def spec_qwen_b1(seed: int = 0, n_steps: int = 256, prompt: int = 32768) -> WorkloadSpec:
    """Qwen2.5-7B head layout, batch 1, 32K prompt, suffix growing to 256,
    2048 clusters, parents of 512 with 32 representatives, 32 sampled teams."""
    return WorkloadSpec("qwen7b_b1_32k", 1, 28, 4, [prompt], 2048, 512, 32, 32, n_steps, 256, [1], 1,
                        seed=seed)


def spec_qwen_b8(seed: int = 0, n_steps: int = 8) -> WorkloadSpec:
    """Batch of 8 independent 32K sequences, 64 sampled teams, concentrated queries."""
    return WorkloadSpec("qwen7b_b8_32k", 8, 28, 4, [32768] * 8, 2048, 512, 32, 64, n_steps, 16, [0] * 8, 0,
                        query_kind="concentrated", seed=seed)


def spec_ragged(seed: int = 0, n_steps: int = 128, n_seqs: int = 32, lo: int = 8192, hi: int = 65536
                ) -> WorkloadSpec:
    """Ragged serving batch: prompt lengths uniform in [lo, hi] rounded to 512,
    suffix lengths uniform in [1, 1024] growing by one per step, 31 sampled teams."""
    rng = np.random.default_rng([seed, 4242])
    lens = (rng.integers(lo // 512, hi // 512 + 1, size=n_seqs) * 512).tolist()
    suf0 = rng.integers(1, 1025, size=n_seqs).tolist()
    return WorkloadSpec("ragged", n_seqs, 28, 4, lens, 2048, 512, 32, 31, n_steps, 1024 + n_steps, suf0, 1,
                        seed=seed)


def spec_long(seed: int = 0, n_sample: int = 32, n_seqs: int = 4, prompt: int = 131072, n_steps: int = 4
              ) -> WorkloadSpec:
    """Long-context sweep point: batch 4, 128K prompt, no suffix."""
    return WorkloadSpec("long_128k", n_seqs, 28, 4, [prompt] * n_seqs, 2048, 512, 32, n_sample, n_steps,
                        16, [0] * n_seqs, 0, seed=seed)


def spec_paper_point(seed: int = 0, n_steps: int = 256, prompt: int = 32768) -> WorkloadSpec:
    """The paper's own operating point on the Qwen2.5-7B head layout: contiguous parents of 16 keys
    with 4 representatives (about N / 4 teams of about 4 rows), 31 sampled teams, batch 1, no suffix."""
    return WorkloadSpec("paper_point_32k", 1, 28, 4, [prompt], 2048, 16, 4, 31, n_steps, 16, [0], 0, seed=seed)


def spec_small_gqa(seed: int = 0, n_seqs: int = 2, prompt=(1536, 1000), n_sample: int = 8,
                   parent_size: int = 128, reps: int = 8, n_steps: int = 3, suffix0=(5, 0)
                   ) -> WorkloadSpec:
    """Small GQA case (28 over 4 heads) the oracle finishes in well under a second;
    prompt lengths need not be multiples of the parent size."""
    return WorkloadSpec("small_gqa", n_seqs, 28, 4, list(prompt), 32, parent_size, reps, n_sample, n_steps,
                        32, list(suffix0), 1, seed=seed)


@dataclass
class LayerData:
    """bf16 bit patterns (uint16) for one layer of one workload."""
    spec: WorkloadSpec
    layer: int
    k_prompt: np.ndarray             # [n_kv, rows_total, d], token order, sequences concatenated
    v_prompt: np.ndarray
    k_suffix: np.ndarray             # [n_seqs, n_kv, suffix_cap, d]
    v_suffix: np.ndarray
    seq_row_off: np.ndarray          # [n_seqs + 1] int64
    centres: Optional[np.ndarray] = field(default=None, repr=False)   # [n_kv, n_clusters, d] float32


def _clustered_rows(rng, n_rows, centres, sigma=0.3, layout="iid"):
    n_clusters, d = centres.shape
    if layout == "iid":
        which = rng.integers(0, n_clusters, size=n_rows)
    elif layout == "runs":
        mean_run = max(n_rows / n_clusters, 1.0)
        lengths = np.empty(0, dtype=np.int64)
        while lengths.sum() < n_rows:
            more = rng.geometric(1.0 / mean_run, size=int(1.5 * n_rows / mean_run) + 8)
            lengths = np.concatenate([lengths, more])
        ids = rng.integers(0, n_clusters, size=lengths.shape[0])
        which = np.repeat(ids, lengths)[:n_rows]
    else:
        raise ValueError(layout)
    eps = rng.standard_normal((n_rows, d), dtype=np.float32)
    return centres[which] + np.float32(sigma) * eps


def make_layer(spec: WorkloadSpec, layer: int = 0, keep_centres: bool = False) -> LayerData:
    d = spec.head_dim
    rows_total = spec.rows_total
    off = np.zeros(spec.n_seqs + 1, dtype=np.int64)
    off[1:] = np.cumsum(spec.prompt_len)
    k_prompt = np.empty((spec.n_kv_heads, rows_total, d), dtype=np.uint16)
    v_prompt = np.empty_like(k_prompt)
    cap = max(spec.suffix_cap, 1)
    k_suffix = np.empty((spec.n_seqs, spec.n_kv_heads, cap, d), dtype=np.uint16)
    v_suffix = np.empty_like(k_suffix)
    centres_all = np.empty((spec.n_kv_heads, spec.n_clusters, d), dtype=np.float32)
    for j in range(spec.n_kv_heads):
        rng = np.random.default_rng([spec.seed, layer, j, 1])
        centres = rng.standard_normal((spec.n_clusters, d), dtype=np.float32)
        centres_all[j] = centres
        for b in range(spec.n_seqs):
            n = spec.prompt_len[b]
            k = _clustered_rows(rng, n, centres, layout=spec.key_layout)
            k[: min(4, n)] *= np.float32(4.0)        # sink keys
            v = rng.standard_normal((n, d), dtype=np.float32)
            k_prompt[j, off[b]:off[b + 1]] = round_bits(k, spec.elem)
            v_prompt[j, off[b]:off[b + 1]] = round_bits(v, spec.elem)
            ks = _clustered_rows(rng, cap, centres)
            vs = rng.standard_normal((cap, d), dtype=np.float32)
            k_suffix[b, j] = round_bits(ks, spec.elem)
            v_suffix[b, j] = round_bits(vs, spec.elem)
    return LayerData(spec, layer, k_prompt, v_prompt, k_suffix, v_suffix, off,
                     centres_all if keep_centres else None)


def make_queries(spec: WorkloadSpec, data: LayerData, step: int) -> np.ndarray:
    """Queries for one decode step: uint16 bf16 bits [n_seqs, n_q_heads, d]."""
    d = spec.head_dim
    G = spec.group
    rng = np.random.default_rng([spec.seed, data.layer, step, 2])
    q = np.empty((spec.n_seqs, spec.n_q_heads, d), dtype=np.float32)
    for b in range(spec.n_seqs):
        lo, hi = int(data.seq_row_off[b]), int(data.seq_row_off[b + 1])
        keys_f32 = {}
        for h in range(spec.n_q_heads):
            j = h // G
            eps = rng.standard_normal(d, dtype=np.float32)
            if spec.query_kind == "noisy_copy":
                row = int(rng.integers(lo, hi))
                kj = to_f32(data.k_prompt[j, row], spec.elem)
                q[b, h] = np.float32(2.0) * (kj + np.float32(0.5) * eps)
            elif spec.query_kind == "concentrated":
                if data.centres is None:
                    raise ValueError("concentrated queries need make_layer(..., keep_centres=True)")
                if j not in keys_f32:
                    keys_f32[j] = to_f32(data.k_prompt[j, lo:hi], spec.elem)
                c = data.centres[j, int(rng.integers(0, spec.n_clusters))]
                base = c + np.float32(0.5) * eps
                logits = (keys_f32[j] @ base).astype(np.float64) / np.sqrt(d)
                q[b, h] = np.float32(_bisect_alpha(logits, 64, 0.90)) * base
            else:
                raise ValueError(spec.query_kind)
    return round_bits(q, spec.elem)


def _bisect_alpha(logits: np.ndarray, top: int, mass: float) -> float:
    """Scale alpha such that the `top` largest softmax weights of alpha*logits
    hold `mass` of the total (input shaping only; not part of the method)."""
    order = np.sort(logits)[::-1]

    def top_mass(alpha):
        z = alpha * (order - order[0])
        w = np.exp(z)
        return w[:top].sum() / w.sum()

    lo, hi = 0.0, 1.0
    while top_mass(hi) < mass and hi < 1e4:
        hi *= 2.0
    for _ in range(50):
        mid = 0.5 * (lo + hi)
        if top_mass(mid) < mass:
            lo = mid
        else:
            hi = mid
    return 0.5 * (lo + hi)


# ------------------------------------------------------------------------------------------------
# Shared-latent rows (the paper's appendix "Token sparsity after latent compression": one row per
# token, 512 content-latent values followed by 64 rotary-key values, shared by 16 heads). Stand-in
# for the DeepSeek-V2-Lite cache of that study, which is not available. Recipe:
#   latent part  n_clusters centres ~ N(0, I_512), row = centre + 0.3 * eps (cluster per row drawn
#                uniformly at random), the first four rows multiplied by 4 ("sinks")
#   rotary part  N(0, I_64)
#   suffix rows  drawn like prompt rows (no sinks)
#   queries      per (step, sequence, head): q = 0.55 * (row_j + 0.5 * eps) for a uniformly random
#                prompt row j, over all 576 values; used with logit scale 1 / sqrt(192) (128 content
#                + 64 rotary query values before absorption), the largest logit is then about 25
# ------------------------------------------------------------------------------------------------
LATENT_DIM, LATENT_ROPE_DIM = 512, 64
LATENT_ROW = LATENT_DIM + LATENT_ROPE_DIM
LATENT_SCALE = float(np.float32(1.0 / np.sqrt(192.0)))   # an fp32 value: the C ABI takes the scale as a float


@dataclass
class LatentSpec:
    name: str
    prompt_len: List[int]
    n_heads: int = 16
    n_clusters: int = 512
    parent_size: int = 16
    reps_per_parent: int = 4
    n_sample: int = 128              # K teams per head (the paper's S = 512 rows at team size 4)
    suffix_cap: int = 16
    suffix_len0: Optional[List[int]] = None
    suffix_growth: int = 1
    seed: int = 0

    @property
    def n_seqs(self) -> int:
        return len(self.prompt_len)

    @property
    def rows_total(self) -> int:
        return int(sum(self.prompt_len))

    def suffix_len(self, step: int) -> np.ndarray:
        s0 = np.zeros(self.n_seqs, dtype=np.int64) if self.suffix_len0 is None else np.asarray(self.suffix_len0, dtype=np.int64)
        return np.minimum(s0 + self.suffix_growth * step, self.suffix_cap).astype(np.int32)


def spec_latent_8k(seed: int = 0, n_seqs: int = 32, n_sample: int = 128, prompt: int = 8192) -> LatentSpec:
    """The paper's shared-latent study point: 8K context, P = 16, R = 4, 16 heads; a batch of sequences."""
    return LatentSpec("latent_8k", [prompt] * n_seqs, n_sample=n_sample, seed=seed)


@dataclass
class LatentLayerData:
    spec: LatentSpec
    layer: int
    rows: np.ndarray                 # [rows_total, 576] bf16 bits, token order, sequences concatenated
    suffix: np.ndarray               # [n_seqs, suffix_cap, 576]
    seq_row_off: np.ndarray


def make_latent_layer(spec: LatentSpec, layer: int = 0) -> LatentLayerData:
    off = np.zeros(spec.n_seqs + 1, dtype=np.int64)
    off[1:] = np.cumsum(spec.prompt_len)
    rows = np.empty((spec.rows_total, LATENT_ROW), dtype=np.uint16)
    cap = max(spec.suffix_cap, 1)
    suffix = np.empty((spec.n_seqs, cap, LATENT_ROW), dtype=np.uint16)
    rng = np.random.default_rng([spec.seed, layer, 0, 11])
    centres = rng.standard_normal((spec.n_clusters, LATENT_DIM), dtype=np.float32)
    for b in range(spec.n_seqs):
        n = spec.prompt_len[b]
        x = np.empty((n, LATENT_ROW), dtype=np.float32)
        x[:, :LATENT_DIM] = _clustered_rows(rng, n, centres)
        x[:, LATENT_DIM:] = rng.standard_normal((n, LATENT_ROPE_DIM), dtype=np.float32)
        x[: min(4, n)] *= np.float32(4.0)
        rows[off[b]:off[b + 1]] = round_bits(x)
        s = np.empty((cap, LATENT_ROW), dtype=np.float32)
        s[:, :LATENT_DIM] = _clustered_rows(rng, cap, centres)
        s[:, LATENT_DIM:] = rng.standard_normal((cap, LATENT_ROPE_DIM), dtype=np.float32)
        suffix[b] = round_bits(s)
    return LatentLayerData(spec, layer, rows, suffix, off)


def make_latent_queries(spec: LatentSpec, data: LatentLayerData, step: int) -> np.ndarray:
    """bf16 bits [n_seqs, n_heads, 576]."""
    rng = np.random.default_rng([spec.seed, data.layer, step, 12])
    q = np.empty((spec.n_seqs, spec.n_heads, LATENT_ROW), dtype=np.float32)
    for b in range(spec.n_seqs):
        lo, hi = int(data.seq_row_off[b]), int(data.seq_row_off[b + 1])
        for h in range(spec.n_heads):
            eps = rng.standard_normal(LATENT_ROW, dtype=np.float32)
            row = to_f32(data.rows[int(rng.integers(lo, hi))])
            q[b, h] = np.float32(0.55) * (row + np.float32(0.5) * eps)
    return round_bits(q)
