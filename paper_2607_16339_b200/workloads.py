"""Seeded synthetic workloads shaped like the paper's evaluation settings.

This module holds DATA generation only (shapes, seeds, value distributions,
rounding of the drawn values to the storage dtype).  It contains none of the
method's arithmetic (no RoPE, no softmax, no state merge) and is the one module
that both the CUDA-path tests and the CPU oracle tests may use.

The paper measures on public suites with trained LLaDA / Dream weights
(Sec. 4.1); neither is available, and the path only ever sees Q/K/V tensors.
These generators stand in for them: shapes follow the generation lengths the
paper's tables use (256 / 512, long generation 1024), structure follows the
method (a fixed prompt, a current block, a suffix of identical [MASK] tokens
that differ only by position; Sec. 3.3.1).

Layout of everything returned: token-major, packed, ``[T, H, d]``; block
tensors are sequence-major ``[B * L_b, H, d]`` (row ``b * L_b + r``).
"""
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np


@dataclass(frozen=True)
class Workload:
    cfg: int
    name: str
    dtype: str            # "bf16" | "fp32"  (storage type of Q/K/V)
    prompt_lens: tuple
    gen_len: int
    block_len: int
    steps_per_block: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    rope_theta: float
    scale_mode: str       # "inv_sqrt_d" | "per_head_u(0.5,2)"
    key_outlier_frac: float = 0.0
    key_outlier_mult: float = 1.0

    @property
    def batch(self):
        return len(self.prompt_lens)

    @property
    def seq_lens(self):
        return [p + self.gen_len for p in self.prompt_lens]

    @property
    def cu_seqlens(self):
        return np.concatenate([[0], np.cumsum(self.seq_lens)]).astype(np.int32)

    @property
    def total_tokens(self):
        return int(sum(self.seq_lens))

    @property
    def n_blocks(self):
        return self.gen_len // self.block_len

    @property
    def n_steps(self):
        return self.n_blocks * self.steps_per_block


# prompt lengths of the ragged config: Philox(key=4).integers(256, 1025, 8)
_RAGGED_PROMPTS = (500, 256, 798, 584, 526, 932, 396, 371)
# prompt lengths of the large-batch extension: 256 few-shot prompts of 600..1000 tokens
_LARGE_BATCH_PROMPTS = tuple(int(x) for x in
                             np.random.Generator(np.random.Philox(key=6)).integers(600, 1001, 256))

WORKLOADS = {
    1: Workload(1, "tiny-fp32", "fp32", (48,), 64, 16, 4, 4, 4, 64, 1.0e4, "inv_sqrt_d"),
    2: Workload(2, "llada8b-l1-p512-g256", "bf16", (512,), 256, 32, 32, 32, 32, 128, 5.0e5,
                "per_head_u(0.5,2)"),
    3: Workload(3, "llada8b-l1-p1024-g512", "bf16", (1024,), 512, 32, 16, 32, 32, 128, 5.0e5,
                "per_head_u(0.5,2)", 0.01, 4.0),
    4: Workload(4, "llada8b-l1-ragged8", "bf16", _RAGGED_PROMPTS, 256, 32, 32, 32, 32, 128, 5.0e5,
                "per_head_u(0.5,2)"),
    5: Workload(5, "dream7b-l1-gqa-p4096-g1024", "bf16", (4096,), 1024, 64, 64, 28, 4, 128, 1.0e6,
                "inv_sqrt_d"),
    # extension beyond the five named configurations: the large-batch setting in which the paper
    # isolates FACache (batch 256, block 32, a 28/4-head GQA model, few-shot prompts; App. table
    # "FACache only"); not a headline configuration
    6: Workload(6, "gqa-l1-batch256-p600to1000-g320", "bf16", _LARGE_BATCH_PROMPTS, 320, 32, 8, 28, 4, 128,
                1.0e6, "inv_sqrt_d"),
}


def round_to_bf16(x):
    """Round float values to the nearest bfloat16 (ties to even); returns float32."""
    a = np.ascontiguousarray(x, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    bias = ((u >> 16) & 1) + 0x7FFF
    r = ((u + bias) >> 16) << 16
    return r.astype(np.uint32).view(np.float32).reshape(a.shape)


def round_to_dtype(x, dtype):
    if dtype == "bf16":
        return round_to_bf16(x)
    if dtype == "fp32":
        return np.ascontiguousarray(x, dtype=np.float32)
    raise ValueError(dtype)


_TENSOR_IDS = {"q": 1, "k": 2, "v": 3, "scale": 4, "mask": 5, "outlier": 6,
               "embed": 7, "norm_w": 8, "w_qkv": 9, "ids": 10, "channels": 11}


def _rng(seed, cfg, tensor, block=0, step=0):
    key = [(seed << 32) | (cfg << 8) | _TENSOR_IDS[tensor], (block << 32) | step]
    return np.random.Generator(np.random.Philox(key=key))


@dataclass
class SyntheticSchedule:
    """Stateful generator of the inputs a block-wise denoising run feeds the path.

    ``q, k, v`` hold the CURRENT full pre-RoPE arrays (float32 numpy holding
    values already rounded to the storage dtype).  Protocol per block ``b``:
    ``begin_block(b)`` (block rows = the mask vector), then for each step
    ``draw_step(b, s)`` returns fresh block tensors and also writes them into
    the full arrays, so the full arrays always show what a full recompute
    would see at that moment.
    """
    wl: Workload
    seed: int = 0
    q: Optional[np.ndarray] = None
    k: Optional[np.ndarray] = None
    v: Optional[np.ndarray] = None
    head_scale_q: Optional[np.ndarray] = None
    head_scale_kv: Optional[np.ndarray] = None
    mask_q: Optional[np.ndarray] = None
    mask_k: Optional[np.ndarray] = None
    mask_v: Optional[np.ndarray] = None
    outlier_rows: List[int] = field(default_factory=list)

    def __post_init__(self):
        wl = self.wl
        d, Hq, Hkv = wl.head_dim, wl.n_q_heads, wl.n_kv_heads
        g = Hq // Hkv
        if wl.scale_mode == "inv_sqrt_d":
            self.head_scale_q = np.full(Hq, 1.0 / np.sqrt(d))
            self.head_scale_kv = np.full(Hkv, 1.0 / np.sqrt(d))
        else:
            # one scale per head shared by that head's q, k and v
            c = _rng(self.seed, wl.cfg, "scale").uniform(0.5, 2.0, Hq)
            self.head_scale_q = c
            self.head_scale_kv = c[::g].copy()
        T = wl.total_tokens
        cu = wl.cu_seqlens
        self.q = self._draw("q", 0, 0, T, Hq, self.head_scale_q)
        self.k = self._draw("k", 0, 0, T, Hkv, self.head_scale_kv, finalize=False)
        self.v = self._draw("v", 0, 0, T, Hkv, self.head_scale_kv)
        # outlier keys: a seeded subset of prompt positions, pre-RoPE K multiplied
        if wl.key_outlier_frac > 0:
            r = _rng(self.seed, wl.cfg, "outlier")
            for b, P in enumerate(wl.prompt_lens):
                n_out = int(np.floor(wl.key_outlier_frac * P))
                rows = np.sort(r.choice(P, size=n_out, replace=False)) + cu[b]
                self.k[rows] *= wl.key_outlier_mult
                self.outlier_rows.extend(int(x) for x in rows)
        self.k = round_to_dtype(self.k, wl.dtype)
        # one pre-RoPE mask vector per head
        mr = _rng(self.seed, wl.cfg, "mask")
        self.mask_q = round_to_dtype(mr.standard_normal((Hq, d)) * self.head_scale_q[:, None], wl.dtype)
        self.mask_k = round_to_dtype(mr.standard_normal((Hkv, d)) * self.head_scale_kv[:, None], wl.dtype)
        self.mask_v = round_to_dtype(mr.standard_normal((Hkv, d)) * self.head_scale_kv[:, None], wl.dtype)
        for b, P in enumerate(wl.prompt_lens):
            lo, hi = cu[b] + P, cu[b + 1]
            self.q[lo:hi] = self.mask_q
            self.k[lo:hi] = self.mask_k
            self.v[lo:hi] = self.mask_v

    def _draw(self, tensor, block, step, n, H, scales, finalize=True):
        r = _rng(self.seed, self.wl.cfg, tensor, block, step)
        x = r.standard_normal((n, H, self.wl.head_dim)) * scales[None, :, None]
        return round_to_dtype(x, self.wl.dtype) if finalize else x.astype(np.float64)

    # ---- index sets (Sec. 3.3.1: C = current block, U = the rest) ----
    def block_rows(self, b):
        """Packed token indices of block b, sequence-major [B * L_b]."""
        wl = self.wl
        cu = wl.cu_seqlens
        rows = []
        for s, P in enumerate(wl.prompt_lens):
            start = cu[s] + P + b * wl.block_len
            rows.append(np.arange(start, start + wl.block_len))
        return np.concatenate(rows).astype(np.int64)

    def is_block(self, b):
        m = np.zeros(self.wl.total_tokens, dtype=np.uint8)
        m[self.block_rows(b)] = 1
        return m

    def positions(self):
        wl = self.wl
        return np.concatenate([np.arange(n) for n in wl.seq_lens]).astype(np.int32)

    # ---- schedule ----
    def begin_block(self, b):
        """Full arrays as the build of block b sees them (block rows masked)."""
        rows = self.block_rows(b)
        self.q[rows] = self.mask_q
        self.k[rows] = self.mask_k
        self.v[rows] = self.mask_v
        return self.q, self.k, self.v

    def draw_step(self, b, s):
        """Fresh block tensors for step s (1-based) of block b; also written
        into the full arrays.  Returns (q_blk, k_blk, v_blk)."""
        wl = self.wl
        n = wl.batch * wl.block_len
        qb = self._draw("q", b + 1, s, n, wl.n_q_heads, self.head_scale_q)
        kb = self._draw("k", b + 1, s, n, wl.n_kv_heads, self.head_scale_kv)
        vb = self._draw("v", b + 1, s, n, wl.n_kv_heads, self.head_scale_kv)
        rows = self.block_rows(b)
        self.q[rows] = qb
        self.k[rows] = kb
        self.v[rows] = vb
        return qb, kb, vb


def parity_points(wl):
    """(block, step) pairs at which parity with the oracle is checked."""
    if wl.cfg == 1:
        return [(b, s) for b in range(wl.n_blocks) for s in range(1, wl.steps_per_block + 1)]
    blocks = sorted({0, wl.n_blocks // 2, wl.n_blocks - 1})
    return [(b, s) for b in blocks for s in (1, wl.steps_per_block)]


def small_workload(name="small", dtype="bf16", prompt_lens=(70,), gen_len=64, block_len=32,
                   steps=2, hq=4, hkv=4, d=128, theta=5.0e5, scale_mode="per_head_u(0.5,2)",
                   cfg=9, outlier_frac=0.0):
    """A reduced workload with the same structure, for parity cases the oracle
    finishes in seconds."""
    return Workload(cfg, name, dtype, tuple(prompt_lens), gen_len, block_len, steps, hq, hkv, d,
                    theta, scale_mode, outlier_frac, 4.0 if outlier_frac > 0 else 1.0)


@dataclass
class TokenModel:
    """Seeded synthetic weights of the token-wise operators in front of the
    first-layer attention (embedding table, norm weight, stacked Q/K/V
    projection) and the token ids a block-wise denoising run feeds them.

    They stand in for the trained first-layer weights of the models the paper
    evaluates, which are not available.  Shapes follow those models: ``d_model``
    4096 with 32 heads (LLaDA-8B), 3584 with 28/4 heads (Dream-7B).  Values: the
    embedding rows are N(0, 1) with a few seeded channels 20x larger (trained
    LLM embeddings carry such outlier channels, and the norm in front of the
    projection is what they stress); the norm weight is U(0.5, 1.5); projection
    rows are N(0, 1/d_model) times the per-head scale of the attention workload,
    so the projected q/k/v have the spread of the workload's own q/k/v.  All
    values are rounded to bf16 (returned as float32).  The last table row is
    the [MASK] token.  The vocabulary size does not change the work of a call
    (a call gathers one row per token), so it may be chosen small.
    """
    wl: Workload
    d_model: int
    vocab: int
    seed: int = 0
    rms_eps: float = 1e-5
    embed: Optional[np.ndarray] = None
    norm_weight: Optional[np.ndarray] = None
    w_qkv: Optional[np.ndarray] = None

    def __post_init__(self):
        wl, dm = self.wl, self.d_model
        d, Hq, Hkv = wl.head_dim, wl.n_q_heads, wl.n_kv_heads
        e = _rng(self.seed, wl.cfg, "embed").standard_normal((self.vocab, dm), dtype=np.float32)
        ch = _rng(self.seed, wl.cfg, "channels").choice(dm, size=max(1, dm // 1024), replace=False)
        e[:, ch] *= 20.0
        self.embed = round_to_bf16(e)
        self.norm_weight = round_to_bf16(_rng(self.seed, wl.cfg, "norm_w").uniform(0.5, 1.5, dm))
        if wl.scale_mode == "inv_sqrt_d":
            sq, skv = np.full(Hq, 1.0 / np.sqrt(d)), np.full(Hkv, 1.0 / np.sqrt(d))
        else:
            c = _rng(self.seed, wl.cfg, "scale").uniform(0.5, 2.0, Hq)
            sq, skv = c, c[::Hq // Hkv].copy()
        row_scale = np.concatenate([np.repeat(sq, d), np.repeat(skv, d), np.repeat(skv, d)])
        w = _rng(self.seed, wl.cfg, "w_qkv").standard_normal(((Hq + 2 * Hkv) * d, dm), dtype=np.float32)
        w *= (row_scale / np.sqrt(dm)).astype(np.float32)[:, None]
        self.w_qkv = round_to_bf16(w)

    @property
    def mask_id(self):
        return self.vocab - 1

    def full_ids(self, b):
        """Token ids of all T packed tokens as the build of block b sees them:
        seeded prompt and already decoded ids, [MASK] from block b on."""
        wl = self.wl
        ids = _rng(self.seed, wl.cfg, "ids").integers(0, self.vocab - 1, wl.total_tokens).astype(np.int32)
        cu = wl.cu_seqlens
        for s, P in enumerate(wl.prompt_lens):
            ids[cu[s] + P + b * wl.block_len:cu[s + 1]] = self.mask_id
        return ids

    def block_ids(self, b, s):
        """Ids of the block's B * L_b tokens at step s (1-based): a seeded subset
        of about s / steps_per_block of the positions is decoded, the rest is
        still [MASK].  Sequence-major."""
        wl = self.wl
        n = wl.batch * wl.block_len
        r = _rng(self.seed, wl.cfg, "ids", b + 1, s)
        ids = r.integers(0, self.vocab - 1, n).astype(np.int32)
        still_masked = r.uniform(size=n) >= s / wl.steps_per_block
        ids[still_masked] = self.mask_id
        return ids


class DeviceSchedule:
    """The same kind of schedule as SyntheticSchedule, drawn on the device with
    torch's generator (data generation only; for sizes where numpy on the host
    would take minutes): all inputs of the block schedule resident in HBM, per
    block the full pre-RoPE arrays the build sees, per step the block's fresh
    tensors."""

    def __init__(self, wl, seed, device, n_steps):
        import torch
        self.wl = wl
        g = torch.Generator(device=device).manual_seed(seed)
        tdt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
        d, Hq, Hkv = wl.head_dim, wl.n_q_heads, wl.n_kv_heads
        grp = Hq // Hkv
        if wl.scale_mode == "inv_sqrt_d":
            cq = torch.full((Hq,), d ** -0.5, device=device)
        else:
            cq = torch.rand(Hq, generator=g, device=device) * 1.5 + 0.5
        ckv = cq[::grp].contiguous()
        T = wl.total_tokens
        rn = lambda n, H, c: (torch.randn(n, H, d, generator=g, device=device) * c[None, :, None])
        q, k, v = rn(T, Hq, cq), rn(T, Hkv, ckv), rn(T, Hkv, ckv)
        cu = wl.cu_seqlens
        if wl.key_outlier_frac > 0:
            for b, P in enumerate(wl.prompt_lens):
                n_out = int(wl.key_outlier_frac * P)
                idx = torch.randperm(P, generator=g, device=device)[:n_out] + int(cu[b])
                k[idx] *= wl.key_outlier_mult
        mq, mk, mv = rn(1, Hq, cq)[0], rn(1, Hkv, ckv)[0], rn(1, Hkv, ckv)[0]
        for b, P in enumerate(wl.prompt_lens):
            q[cu[b] + P:cu[b + 1]] = mq; k[cu[b] + P:cu[b + 1]] = mk; v[cu[b] + P:cu[b + 1]] = mv
        S, Lb, B = wl.steps_per_block, wl.block_len, wl.batch
        self.n_blocks_used = min(wl.n_blocks, (n_steps + S - 1) // S)
        self.full = []    # per block: (q, k, v) as the build sees them
        self.steps = []   # per step: (q_blk, k_blk, v_blk)
        rows_of = lambda blk: torch.cat([torch.arange(cu[b] + P + blk * Lb, cu[b] + P + (blk + 1) * Lb)
                                         for b, P in enumerate(wl.prompt_lens)]).to(device)
        for blk in range(self.n_blocks_used):
            self.full.append((q.to(tdt).contiguous(), k.to(tdt).contiguous(), v.to(tdt).contiguous()))
            last = None
            for s in range(S):
                last = (rn(B * Lb, Hq, cq).to(tdt).contiguous(), rn(B * Lb, Hkv, ckv).to(tdt).contiguous(),
                        rn(B * Lb, Hkv, ckv).to(tdt).contiguous())
                self.steps.append(last)
            rows = rows_of(blk)
            q[rows], k[rows], v[rows] = last[0].float(), last[1].float(), last[2].float()

    def step_inputs(self, i):
        S = self.wl.steps_per_block
        n = self.n_blocks_used * S
        i = i % n
        return i // S, i % S, self.steps[i]
