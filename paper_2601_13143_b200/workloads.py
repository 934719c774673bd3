"""Seeded synthetic inputs for the FastAV prune step.

This module only *draws inputs*: it holds none of the method's arithmetic (no scoring, no
selection, no gathering), so both the CUDA path and the CPU checker can be fed from it without
sharing any code that matters.  All tensors are made on the CPU from ``torch.Generator`` seeds,
rounded to bf16 once, and handed out as the same bits to every consumer.

The five workloads mirror audio-visual LLM prefill shapes: a token sequence laid out as
``[text prefix | audio | video | text suffix]`` on a 7B-class grouped-query decoder, pruned at a
middle layer ("global" stage) and again at later layers ("fine" stages, last-token query only),
as in Section 2.2 of the paper.  They stand in for the *shapes* of the paper's AVQA /
MUSIC-AVQA / AVHBench runs on VideoLLaMA2 / video-SALMONN2; none of those datasets' items or
the models' weights are used.  A few "anchor" tokens in the first quarter of each sequence get
keys aligned with the mean scored query (the anchor-like early tokens the paper's rollout
analysis shows), so that the scores have realistic structure instead of being flat noise.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import torch

MOD_TEXT, MOD_AUDIO, MOD_VIDEO = 0, 1, 2


@dataclass(frozen=True)
class ModelShape:
    name: str
    num_layers: int
    hidden: int
    ffn: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int


TINY = ModelShape("tiny-gqa", 4, 512, 1376, 8, 2, 64)
QWEN2_7B = ModelShape("qwen2-7b", 28, 3584, 18944, 28, 4, 128)
MISTRAL_7B = ModelShape("mistral-7b", 32, 4096, 14336, 32, 8, 128)


@dataclass(frozen=True)
class Stage:
    """One pruning layer: which decoder layer, how many trailing rows are scored, keep ratio
    (None = per-sequence ratios drawn by the workload)."""
    layer: int
    rows: int
    keep: float | None


@dataclass(frozen=True)
class Workload:
    name: str
    index: int
    seed: int
    model: ModelShape
    batch: int
    seq_len: int | tuple[int, int]          # fixed length, or (lo, hi) inclusive
    segments: tuple[int, int, int, int] | None  # text prefix, audio, video, text suffix; None = 5/15/80 %
    anchors: int
    stages: tuple[Stage, ...]
    sparse_positions: bool = False          # positions = sorted random subset of [0, 2 n)
    keep_range: tuple[float, float] | None = None
    description: str = ""


WORKLOADS: dict[str, Workload] = {
    w.name: w
    for w in (
        Workload("c1_tiny", 0, 0, TINY, 1, 512, (32, 160, 288, 32), 8, (Stage(2, 4, 0.5),),
                 description="tiny single prune, L=512"),
        Workload("c2_global_2k", 1, 1, QWEN2_7B, 1, 2048, (64, 256, 1664, 64), 16, (Stage(14, 64, 0.5),),
                 description="VideoLLaMA2-like global prune at layer 14 of 28, L=2048"),
        Workload("c3_fine_chain", 2, 2, QWEN2_7B, 1, 1024, None, 8,
                 (Stage(20, 1, 0.8), Stage(24, 1, 0.8), Stage(26, 1, 0.8)), sparse_positions=True,
                 description="fine-prune chain 1024 -> 820 -> 656 -> 525, last-token query"),
        Workload("c4_long_av", 3, 3, MISTRAL_7B, 4, 16384, (128, 2048, 14080, 128), 64,
                 (Stage(16, 128, 0.4), Stage(17, 1, 0.7)),
                 description="long audio-video clip, 4 x 16384, global keep 40% then fine keep 70%"),
        Workload("c5_ragged", 4, 4, QWEN2_7B, 32, (1024, 8192), None, 16,
                 (Stage(14, 32, None), Stage(15, 1, 0.8)), keep_range=(0.3, 0.7),
                 description="ragged serving batch, 32 sequences of 1024..8192 tokens, two stages"),
        # Beyond the five configurations: the paper's own fine-pruning schedule on VideoLLaMA2-like sizes -- about 744
        # survivors of the global stage (2,230 tokens, audio 1,496 -> 10), then P = 20 % at each of the 13 later layers.
        Workload("n3_fine_chain_13", 5, 5, QWEN2_7B, 1, 744, None, 8,
                 tuple(Stage(layer, 1, 0.8) for layer in range(15, 28)), sparse_positions=True,
                 description="the paper's 13-layer fine-prune chain after the global stage, 744 -> ... -> 42, last-token query"),
    )
}
WORKLOAD_ORDER = ("c1_tiny", "c2_global_2k", "c3_fine_chain", "c4_long_av", "c5_ragged")
EXTRA_WORKLOADS = ("n3_fine_chain_13",)


def keep_count(n: int, keep_ratio: float) -> int:
    """Survivors when the bottom P % by score (P = 1 - keep_ratio; Section 2.2, "Fine pruning") of n tokens are removed: the removed
    count is floor(P n)."""
    return n - int(math.floor((1.0 - keep_ratio) * n + 1e-6))


@dataclass
class PruneInputs:
    """Everything one prune call consumes, on the CPU."""
    model: ModelShape
    q: torch.Tensor            # [sum R, Hq, d] bf16
    k: torch.Tensor            # [N, Hkv, d] bf16
    v: torch.Tensor            # [N, Hkv, d] bf16
    hidden: torch.Tensor | None  # [N, D] bf16 (None for a chained stage: comes from the previous one)
    pos: torch.Tensor | None     # [N] int32
    cu_seqlens: torch.Tensor   # [B+1] int32
    cu_qlens: torch.Tensor     # [B+1] int32
    q_idx: torch.Tensor        # [sum R] int32, sequence-local
    keep_counts: torch.Tensor  # [B] int32
    modality: torch.Tensor | None = None  # [N] uint8 (first stage only)
    anchors: list = field(default_factory=list)  # per sequence: LongTensor of anchor indices
    softmax_scale: float = 0.0
    causal: bool = True
    protect_rows: bool = True
    layer: int = 0

    @property
    def batch(self) -> int:
        return self.cu_seqlens.numel() - 1

    @property
    def total_tokens(self) -> int:
        return int(self.cu_seqlens[-1])

    @property
    def total_keep(self) -> int:
        return int(self.keep_counts.sum())


def _randn_bf16(gen: torch.Generator, *shape: int) -> torch.Tensor:
    """N(0,1) in fp32, rounded to bf16 once.  Drawn in slabs to bound the fp32 temporary."""
    out = torch.empty(shape, dtype=torch.bfloat16)
    flat = out.view(-1)
    slab = 1 << 26
    for start in range(0, flat.numel(), slab):
        stop = min(start + slab, flat.numel())
        flat[start:stop] = torch.randn(stop - start, generator=gen, dtype=torch.float32).to(torch.bfloat16)
    return out


def _segments_for(n: int, fixed: tuple[int, int, int, int] | None) -> tuple[int, int, int, int]:
    if fixed is not None and sum(fixed) == n:
        return fixed
    text = int(round(0.05 * n))
    audio = int(round(0.15 * n))
    prefix = text // 2
    suffix = text - prefix
    return prefix, audio, n - text - audio, suffix


def sequence_lengths(w: Workload) -> list[int]:
    """First-stage lengths (drawn from the workload's own seed when ragged)."""
    if isinstance(w.seq_len, tuple):
        gen = torch.Generator(device="cpu").manual_seed(1_000_003 * (w.seed + 1))
        lo, hi = w.seq_len
        return torch.randint(lo, hi + 1, (w.batch,), generator=gen).tolist()
    return [int(w.seq_len)] * w.batch


def keep_ratios(w: Workload, stage_index: int) -> list[float]:
    st = w.stages[stage_index]
    if st.keep is not None:
        return [st.keep] * w.batch
    gen = torch.Generator(device="cpu").manual_seed(2_000_003 * (w.seed + 1))
    lo, hi = w.keep_range
    return (lo + (hi - lo) * torch.rand(w.batch, generator=gen, dtype=torch.float64)).tolist()


def stage_lengths(w: Workload) -> list[list[int]]:
    """Token counts per sequence entering stage 0, 1, ... and leaving the last one."""
    lens = [sequence_lengths(w)]
    for s in range(len(w.stages)):
        ratios = keep_ratios(w, s)
        lens.append([keep_count(n, r) for n, r in zip(lens[-1], ratios)])
    return lens


def make_stage(w: Workload, stage_index: int, lengths: list[int] | None = None, rows: int | None = None) -> PruneInputs:
    """Inputs of stage ``stage_index``.  Stage 0 carries hidden states, position ids and the
    modality map; later stages draw fresh q/k/v for their layer at the survivor lengths and leave
    ``hidden``/``pos`` to be chained from the previous stage's output."""
    st = w.stages[stage_index]
    m = w.model
    all_lens = stage_lengths(w)
    lens = list(all_lens[stage_index] if lengths is None else lengths)
    rows = st.rows if rows is None else rows
    gen = torch.Generator(device="cpu").manual_seed(7919 * w.seed + 104_729 * stage_index + 17)

    cu = torch.zeros(len(lens) + 1, dtype=torch.int32)
    cu[1:] = torch.tensor(lens, dtype=torch.int64).cumsum(0).to(torch.int32)
    n_total = int(cu[-1])
    r_per = [min(rows, n) for n in lens]
    cu_q = torch.zeros(len(lens) + 1, dtype=torch.int32)
    cu_q[1:] = torch.tensor(r_per, dtype=torch.int64).cumsum(0).to(torch.int32)
    q_idx = torch.cat([torch.arange(n - r, n, dtype=torch.int32) for n, r in zip(lens, r_per)]) \
        if sum(r_per) else torch.zeros(0, dtype=torch.int32)

    q = _randn_bf16(gen, int(cu_q[-1]), m.num_q_heads, m.head_dim)
    k = _randn_bf16(gen, n_total, m.num_kv_heads, m.head_dim)
    v = _randn_bf16(gen, n_total, m.num_kv_heads, m.head_dim)

    group = m.num_q_heads // m.num_kv_heads
    anchors = []
    for b, n in enumerate(lens):
        quarter = max(n // 4, 1)
        count = min(w.anchors, quarter)
        idx = torch.randperm(quarter, generator=gen)[:count].sort().values
        anchors.append(idx)
        r0, r1 = int(cu_q[b]), int(cu_q[b + 1])
        if r1 == r0 or count == 0:
            continue
        qb = q[r0:r1].float().view(r1 - r0, m.num_kv_heads, group, m.head_dim)
        qbar = qb.mean(dim=(0, 2))                                   # [Hkv, d]
        rms = qbar.pow(2).mean(dim=1, keepdim=True).sqrt().clamp_min(1e-12)
        k[int(cu[b]) + idx] = (3.0 * qbar / rms).to(torch.bfloat16)  # broadcast over the anchors

    hidden = pos = modality = None
    if stage_index == 0:
        hidden = _randn_bf16(gen, n_total, m.hidden)
        pos_parts, mod_parts = [], []
        for n in lens:
            if w.sparse_positions:
                p = torch.randperm(2 * n, generator=gen)[:n].sort().values.to(torch.int32)
            else:
                p = torch.arange(n, dtype=torch.int32)
            pos_parts.append(p)
            pre, aud, vid, suf = _segments_for(n, w.segments)
            mod_parts.append(torch.cat([
                torch.full((pre,), MOD_TEXT, dtype=torch.uint8), torch.full((aud,), MOD_AUDIO, dtype=torch.uint8),
                torch.full((vid,), MOD_VIDEO, dtype=torch.uint8), torch.full((suf,), MOD_TEXT, dtype=torch.uint8)]))
        pos = torch.cat(pos_parts)
        modality = torch.cat(mod_parts)

    ratios = keep_ratios(w, stage_index)
    keep_counts = torch.tensor([keep_count(n, r) for n, r in zip(lens, ratios)], dtype=torch.int32)
    return PruneInputs(model=m, q=q, k=k, v=v, hidden=hidden, pos=pos, cu_seqlens=cu, cu_qlens=cu_q, q_idx=q_idx,
                       keep_counts=keep_counts, modality=modality, anchors=anchors,
                       softmax_scale=1.0 / math.sqrt(m.head_dim), causal=True, protect_rows=True, layer=st.layer)


def bf16_bits(t: torch.Tensor):
    """bf16 tensor -> uint16 numpy view of the same bits (how inputs travel to a checker that takes bit patterns)."""
    import numpy as np
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def random_problem(seed: int, lens: list[int], rows: list[int], keeps: list[int], num_q_heads: int, num_kv_heads: int,
                   head_dim: int, hidden: int, duplicate_keys: int = 0, trailing_rows: bool = True) -> PruneInputs:
    """A small free-form problem for edge-case tests: arbitrary lengths (zero allowed), rows and
    keep counts per sequence.  ``duplicate_keys`` copies that many key rows over other tokens of the
    same sequence so that exact score ties occur.  Hidden/K/V rows carry their own token index in
    their first elements, which makes a misplaced gather visible."""
    gen = torch.Generator(device="cpu").manual_seed(seed)
    model = ModelShape("free", 2, hidden, 4 * hidden, num_q_heads, num_kv_heads, head_dim)
    cu = torch.zeros(len(lens) + 1, dtype=torch.int32)
    cu[1:] = torch.tensor(lens, dtype=torch.int64).cumsum(0).to(torch.int32)
    r_per = [min(r, n) for r, n in zip(rows, lens)]
    cu_q = torch.zeros(len(lens) + 1, dtype=torch.int32)
    cu_q[1:] = torch.tensor(r_per, dtype=torch.int64).cumsum(0).to(torch.int32)
    parts = []
    for n, r in zip(lens, r_per):
        if trailing_rows:
            parts.append(torch.arange(n - r, n, dtype=torch.int32))
        else:
            parts.append(torch.randperm(max(n, 1), generator=gen)[:r].sort().values.to(torch.int32))
    q_idx = torch.cat(parts) if parts else torch.zeros(0, dtype=torch.int32)
    n_total = int(cu[-1])
    q = _randn_bf16(gen, int(cu_q[-1]), num_q_heads, head_dim)
    k = _randn_bf16(gen, n_total, num_kv_heads, head_dim)
    v = _randn_bf16(gen, n_total, num_kv_heads, head_dim)
    h = _randn_bf16(gen, n_total, hidden)
    for b, n in enumerate(lens):
        if n >= 2 and duplicate_keys:
            src = torch.randint(0, n, (duplicate_keys,), generator=gen)
            dst = torch.randint(0, n, (duplicate_keys,), generator=gen)
            k[int(cu[b]) + dst] = k[int(cu[b]) + src]
    ids = torch.arange(n_total, dtype=torch.int32)
    tag = torch.stack([(ids & 0xFF).to(torch.float32), ((ids >> 8) & 0xFF).to(torch.float32)], dim=1).to(torch.bfloat16)
    if n_total:
        h[:, :2] = tag
        v[:, :, :2] = tag[:, None, :]
    pos = (3 * ids + 5).to(torch.int32)
    return PruneInputs(model=model, q=q, k=k, v=v, hidden=h, pos=pos, cu_seqlens=cu, cu_qlens=cu_q, q_idx=q_idx,
                       keep_counts=torch.tensor(keeps, dtype=torch.int32), softmax_scale=1.0 / math.sqrt(head_dim),
                       causal=True, protect_rows=False)


def positional_keep_mask(modality: torch.Tensor, cu_seqlens: torch.Tensor, keep_first: dict[int, int]) -> torch.Tensor:
    """Keep mask of a positional rule of the kind the paper deploys at its global stage: of every modality
    named in ``keep_first`` only the first m tokens of each sequence survive (e.g. ``{MOD_AUDIO: 10}`` keeps
    the first 10 audio tokens); tokens of all other modalities survive.  Input construction only."""
    mask = torch.ones_like(modality, dtype=torch.uint8)
    cu = cu_seqlens.tolist()
    for b in range(len(cu) - 1):
        seg = modality[cu[b]:cu[b + 1]]
        for mod, m in keep_first.items():
            idx = torch.nonzero(seg == mod).flatten()
            mask[cu[b] + idx[m:]] = 0
    return mask


def random_control_scores(seed: int, total_tokens: int) -> torch.Tensor:
    """Scores of the "Random" control of the selector ablations (Tables 2-3): one seeded uniform draw per token,
    fp32.  Handed to ``fastav_select`` in place of the attention scores, they make the keep set a seeded random
    subset (protected tokens still survive, ties still go to the lower index).  Input construction only."""
    gen = torch.Generator().manual_seed(seed)
    return torch.rand(total_tokens, generator=gen, dtype=torch.float32)
