"""Seeded synthetic decode-attention inputs (paged KV caches, block tables, queries).

This module only *draws inputs*.  It contains none of the method's arithmetic
(no scores, no selection, no sampling, no budgets), so both the CPU oracle's
tests and the CUDA path's tests may use it without sharing any computation.

Layout produced (the layout the C-ABI consumes):
  q            [B, Hq, d]                       fp32 array, or bf16 bit patterns (uint16)
  k_cache      [num_blocks, Hkv, 16, d]         same element type ("HND" paged layout)
  v_cache      [num_blocks, Hkv, 16, d]
  block_table  [B, max_blocks_per_seq] int32    logical page -> physical page (seeded permutation)
  seq_lens     [B] int32

The workloads stand in for the attention geometry the paper evaluates
(Llama-3.1-8B: 32 query heads, 8 KV heads, head_dim 128, 32K context, sink =
window = 128, top-k and base rate 2.5 %, eps = delta = 0.05; Table 2 caption and
Table 3 of the paper); the paper's own models and datasets are not available.
"""
from __future__ import annotations

from dataclasses import dataclass, field
import numpy as np

BLOCK = 16  # tokens per KV page


# ----------------------------------------------------------------------------- bf16 <-> fp32 (storage only)
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounding = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + rounding) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to the fp32 values they denote (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------- case container
@dataclass
class Case:
    name: str
    dtype: str                    # "fp32" | "bf16"
    q: np.ndarray                 # [B,Hq,d] float32 or uint16 (bf16 bits)
    k_cache: np.ndarray           # [num_blocks,Hkv,16,d]
    v_cache: np.ndarray
    block_table: np.ndarray       # [B,max_blocks] int32
    seq_lens: np.ndarray          # [B] int32
    sink: int
    window: int
    k: int
    eps: float
    delta: float
    seed: int
    params: dict = field(default_factory=dict)   # base_rate, topk_frac, scale, mode, layer, step, ...
    meta: dict = field(default_factory=dict)     # generator knobs, for reports

    @property
    def batch(self): return int(self.q.shape[0])
    @property
    def num_q_heads(self): return int(self.q.shape[1])
    @property
    def num_kv_heads(self): return int(self.k_cache.shape[1])
    @property
    def head_dim(self): return int(self.q.shape[2])
    @property
    def num_blocks(self): return int(self.k_cache.shape[0])
    @property
    def max_blocks_per_seq(self): return int(self.block_table.shape[1])

    def values(self, a: np.ndarray) -> np.ndarray:
        """The real numbers stored in `a`, as fp32 (exact for both element types)."""
        return bf16_bits_to_f32(a) if self.dtype == "bf16" else np.asarray(a, dtype=np.float32)


def _store(x: np.ndarray, dtype: str) -> np.ndarray:
    return f32_to_bf16_bits(x) if dtype == "bf16" else np.ascontiguousarray(x, dtype=np.float32)


def make_block_table(rng: np.random.Generator, seq_lens, max_blocks=None, spare_frac=0.10):
    """Seeded random permutation of physical pages; pool = needed pages + `spare_frac`."""
    seq_lens = np.asarray(seq_lens, dtype=np.int64)
    need = (seq_lens + BLOCK - 1) // BLOCK
    total = int(need.sum())
    num_blocks = total + max(1, int(np.ceil(total * spare_frac)))
    perm = rng.permutation(num_blocks).astype(np.int32)
    mb = int(max_blocks if max_blocks is not None else max(1, int(need.max())))
    bt = np.full((len(seq_lens), mb), -1, dtype=np.int32)   # -1 marks an unused slot
    pos = 0
    for b, nb in enumerate(need):
        bt[b, :nb] = perm[pos:pos + nb]
        pos += int(nb)
    return bt, num_blocks


def make_case(name, *, dtype, B, Hq, Hkv, d, seq_lens, sink, window, k, eps, delta, seed,
              gen_seed, key_std=1.0, q_std=None, rho_v=1.0, heavy=None, params=None,
              max_blocks=None, poison_unused=True) -> Case:
    """Draw one synthetic decode step.

    key_std : std of the N(0, key_std^2) key entries.
    q_std   : per-query-head std of q (array [Hq] or scalar); default 1.
    rho_v   : every value row is mu_g + xi, xi ~ N(0,1)^d, mu_g = rho_v * e_g with e_g in {+-1}^d.
    heavy   : None, or dict(R=..., c1=..., alpha=(lo,hi)) planting R heavy-hitter keys per query head
              in the middle of the context: K[i] += c_r * sqrt(d) * q_h / |q_h|^2 on the head's KV
              head, c_r = max(0, c1 - alpha_h * ln r), r = 1..R.  With the default softmax scale
              1/sqrt(d) this shifts head h's logit at token i by exactly c_r.
              `heads` (optional) restricts planting to those query heads.
    poison_unused : fill never-addressed pages and the tail of each last page with large finite
              garbage, so a kernel that reads beyond seq_len shows up in the results.
    """
    rng = np.random.default_rng(gen_seed)
    seq_lens = np.asarray(seq_lens, dtype=np.int32)
    assert len(seq_lens) == B and Hq % Hkv == 0
    G = Hq // Hkv
    bt, num_blocks = make_block_table(rng, seq_lens, max_blocks)
    qs = np.ones(Hq, np.float32) if q_std is None else np.broadcast_to(np.asarray(q_std, np.float32), (Hq,))
    q = rng.standard_normal((B, Hq, d), dtype=np.float32) * qs[None, :, None]
    kc = np.empty((num_blocks, Hkv, BLOCK, d), dtype=np.float32)
    vc = np.empty((num_blocks, Hkv, BLOCK, d), dtype=np.float32)
    if poison_unused:
        kc[...] = 3.0e4
        vc[...] = -7.0e4
    else:
        kc[...] = 0.0
        vc[...] = 0.0
    e_g = rng.choice(np.array([-1.0, 1.0], np.float32), size=(Hkv, d))
    for b in range(B):
        n = int(seq_lens[b])
        if n == 0:
            continue
        K = rng.standard_normal((Hkv, n, d), dtype=np.float32) * np.float32(key_std)
        V = rng.standard_normal((Hkv, n, d), dtype=np.float32) + np.float32(rho_v) * e_g[:, None, :]
        if heavy is not None:
            lo, hi = min(sink, n), max(min(sink, n), n - window)
            R = int(min(heavy["R"], max(0, hi - lo)))
            heads = heavy.get("heads", range(Hq))
            a_lo, a_hi = heavy.get("alpha", (1.0, 1.0))
            for h in heads:
                if R == 0:
                    break
                g = h // G
                alpha = rng.uniform(a_lo, a_hi)
                pos = lo + rng.choice(hi - lo, size=R, replace=False)
                c = np.maximum(0.0, heavy["c1"] - alpha * np.log(np.arange(1, R + 1))).astype(np.float32)
                qh = q[b, h]
                K[g, pos, :] += (c[:, None] * np.float32(np.sqrt(d)) / np.float32(qh @ qh)) * qh[None, :]
        nb = (n + BLOCK - 1) // BLOCK
        pad = nb * BLOCK - n
        if pad:
            fillk = np.full((Hkv, pad, d), 3.0e4 if poison_unused else 0.0, np.float32)
            fillv = np.full((Hkv, pad, d), -7.0e4 if poison_unused else 0.0, np.float32)
            K = np.concatenate([K, fillk], axis=1)
            V = np.concatenate([V, fillv], axis=1)
        kc[bt[b, :nb]] = K.reshape(Hkv, nb, BLOCK, d).transpose(1, 0, 2, 3)
        vc[bt[b, :nb]] = V.reshape(Hkv, nb, BLOCK, d).transpose(1, 0, 2, 3)
    bt = np.where(bt < 0, 0, bt).astype(np.int32)   # unused slots point at a valid page; never read
    meta = dict(gen_seed=gen_seed, key_std=key_std, rho_v=rho_v, heavy=heavy,
                q_std=None if q_std is None else np.asarray(q_std).tolist())
    return Case(name=name, dtype=dtype, q=_store(q, dtype), k_cache=_store(kc, dtype), v_cache=_store(vc, dtype),
                block_table=bt, seq_lens=seq_lens, sink=sink, window=window, k=k, eps=eps, delta=delta,
                seed=seed, params=dict(params or {}), meta=meta)


# ----------------------------------------------------------------------------- the five workloads
C1_CALIBRATED = 9.85   # heavy-hitter strength giving ~10x sparsity on the Llama-8B-shaped layer (found by bisection on the
                       # oracle's mean density: 0.0999 at this value)


def multi_query(case: Case, q_len: int, noise=0.35, gen_seed=9009) -> np.ndarray:
    """Query rows for a call that carries `q_len` query tokens per sequence: [B, q_len, Hq, d] in the case's
    storage type.  The last token's rows are the case's own q; earlier tokens are the same rows plus Gaussian
    noise of `noise` times their standard deviation, so every token keeps the case's attention structure
    (heavy hitters, near-uniform heads) without repeating its scores."""
    rng = np.random.default_rng(gen_seed)
    base = case.values(case.q).astype(np.float32)                  # [B,Hq,d]
    rows = []
    for t in range(q_len):
        if t == q_len - 1:
            rows.append(base)
        else:
            sd = base.std(axis=-1, keepdims=True)
            rows.append((base + noise * sd * rng.standard_normal(base.shape).astype(np.float32)).astype(np.float32))
    return np.ascontiguousarray(np.stack([_store(r, case.dtype) for r in rows], axis=1))


def config1_tiny(gen_seed=1001, **over) -> Case:
    """Tiny decode: 1 head, d=64, n=1024, fp32, 8 planted heavy hitters of strength 4."""
    kw = dict(dtype="fp32", B=1, Hq=1, Hkv=1, d=64, seq_lens=[1024], sink=4, window=32, k=32,
              eps=0.05, delta=0.05, seed=0, gen_seed=gen_seed, key_std=1.0, rho_v=0.0,
              heavy=dict(R=8, c1=4.0, alpha=(0.0, 0.0)), params=dict(base_rate=0.025))
    kw.update(over)
    return make_case("cfg1_tiny", **kw)


def config2_llama8b(n=32768, c1=C1_CALIBRATED, gen_seed=2002, **over) -> Case:
    """Llama-3.1-8B-shaped layer: 32/8 heads, d=128, bf16, power-law heavy hitters per head."""
    kw = dict(dtype="bf16", B=1, Hq=32, Hkv=8, d=128, seq_lens=[n], sink=128, window=128,
              k=int(0.025 * n), eps=0.05, delta=0.05, seed=2, gen_seed=gen_seed, key_std=1.0, rho_v=1.0,
              heavy=dict(R=256, c1=c1, alpha=(0.75, 1.25)), params=dict(base_rate=0.025))
    kw.update(over)
    return make_case("cfg2_llama8b", **kw)


def config3_uniform(n=32768, gen_seed=3003, **over) -> Case:
    """Same shape, near-uniform scores: keys ~ N(0, 0.1^2), no heavy hitters, eps = delta = 0.1."""
    kw = dict(dtype="bf16", B=1, Hq=32, Hkv=8, d=128, seq_lens=[n], sink=128, window=128,
              k=int(0.025 * n), eps=0.1, delta=0.1, seed=3, gen_seed=gen_seed, key_std=0.1, rho_v=1.0,
              heavy=None, params=dict(base_rate=0.025))
    kw.update(over)
    return make_case("cfg3_uniform", **kw)


def config4_serving(B=32, lo=4096, hi=32768, c1=C1_CALIBRATED, gen_seed=4004, **over) -> Case:
    """Batched serving: mixed lengths U{lo..hi}; even query heads heavy-hitter, odd heads near-uniform."""
    rng = np.random.default_rng(gen_seed + 7)
    seq_lens = rng.integers(lo, hi + 1, size=B).astype(np.int32)
    Hq = over.get("Hq", 32)
    q_std = np.where(np.arange(Hq) % 2 == 0, 1.0, 0.1).astype(np.float32)
    kw = dict(dtype="bf16", B=B, Hq=32, Hkv=8, d=128, seq_lens=seq_lens, sink=128, window=128, k=0,
              eps=0.05, delta=0.05, seed=4, gen_seed=gen_seed, key_std=1.0, rho_v=1.0, q_std=q_std,
              heavy=dict(R=256, c1=c1, alpha=(0.75, 1.25), heads=list(range(0, Hq, 2))),
              params=dict(base_rate=0.025, topk_frac=0.02))
    kw.update(over)
    return make_case("cfg4_serving", **kw)


def config5_reasoning(n=32768, B=8, step=None, c1=C1_CALIBRATED, gen_seed=5005, max_n=32768, **over) -> Case:
    """Reasoning-length decode: batch 8 at context n (one snapshot of the growing cache).

    The cache is sized for `max_n` tokens so a harness can append rows; `step` is the Philox
    step word (defaults to n, the index of the decode iteration that sees n tokens)."""
    kw = dict(dtype="bf16", B=B, Hq=32, Hkv=8, d=128, seq_lens=[n] * B, sink=128, window=128, k=0,
              eps=0.05, delta=0.05, seed=5, gen_seed=gen_seed, key_std=1.0, rho_v=1.0,
              heavy=dict(R=256, c1=c1, alpha=(0.75, 1.25)),
              params=dict(base_rate=0.025, topk_frac=0.025, step=int(n if step is None else step)),
              max_blocks=(max_n + BLOCK - 1) // BLOCK)
    kw.update(over)
    return make_case("cfg5_reasoning", **kw)
