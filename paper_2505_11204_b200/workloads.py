"""Seeded synthetic weight sets shaped like the models the paper compresses.

This module holds shapes and random inputs only -- none of the method's
arithmetic (no transforms, no hashing of seeds into signs or permutations).
It serves both the CUDA library's callers and the CPU checker so that the two
see identical input bits.

The paper evaluates on public fine-tuned checkpoints (CLIP ViT-B/32 and
ViT-L/14 vision encoders, Flan-T5-base, GPT-2; Sections 5.1, 5.9 and the
appendix on model details).  None of those are used here: each workload below
reproduces only the tensor list (names, shapes, which tensors repeat across
blocks) of such a model and fills it with seeded Gaussian values.

Value recipe (per element):  W_0 ~ N(0, 0.02^2);  delta_i = scale * (0.5 c +
sqrt(0.75) e_i) with c shared by all tasks and e_i private, both N(0, 1), so
that any two deltas have cosine 0.25 before transformation;  W_i = W_0 +
delta_i rounded to the storage type.  With bf16 storage W_0 is rounded to bf16
first.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

F32 = 0
BF16 = 1
SHUFFLE = 1
FLIP = 2
GAUSS = 1 << 16   # Gaussian-like diagonal context instead of the +-1 one (RANDES_GAUSS)


@dataclass
class Workload:
    name: str
    layer_names: List[str]
    rows: List[int]
    cols: List[int]
    group: List[int]
    gflags: List[int]
    storage: int = F32
    n_tasks: int = 1
    task_ids: List[int] = field(default_factory=list)
    seeds: List[int] = field(default_factory=list)
    scale: float = 1e-3
    lam: float = 1.0
    data_seed: int = 0

    @property
    def n_layers(self) -> int:
        return len(self.rows)

    @property
    def n_params(self) -> int:
        return int(sum(r * c for r, c in zip(self.rows, self.cols)))

    @property
    def spec(self):
        return (self.rows, self.cols, self.group, self.gflags)

    def group_sizes(self) -> List[int]:
        sizes = [0] * len(self.gflags)
        for g in self.group:
            sizes[g] += 1
        return sizes

    def np_dtype(self):
        return np.uint16 if self.storage == BF16 else np.float32

    def with_storage(self, storage: int) -> "Workload":
        w = Workload(**{**self.__dict__})
        w.storage = storage
        w.name = self.name.split(":")[0] + (":bf16" if storage == BF16 else ":f32")
        return w

    def with_gaussian_context(self) -> "Workload":
        """The same set with the +-1 context of every flipped group replaced by the Gaussian-like diagonal of the paper's
        RD ablation (Section 5.5)."""
        w = Workload(**{**self.__dict__})
        w.gflags = [(f & ~FLIP) | GAUSS if f & FLIP else f for f in self.gflags]
        w.name = self.name + ":rd"
        return w

    def with_tasks(self, n_tasks: int, first_seed: Optional[int] = None) -> "Workload":
        w = Workload(**{**self.__dict__})
        s0 = self.seeds[0] if first_seed is None else first_seed
        w.n_tasks = n_tasks
        w.task_ids = list(range(n_tasks))
        w.seeds = [s0 + i for i in range(n_tasks)]
        return w


class _Builder:
    """Collects tensors; tensors added with the same ``kind`` form one group."""

    def __init__(self):
        self.names: List[str] = []
        self.rows: List[int] = []
        self.cols: List[int] = []
        self.group: List[int] = []
        self.kinds: Dict[str, int] = {}

    def add(self, name: str, rows: int, cols: int, kind: Optional[str] = None):
        kind = name if kind is None else kind
        g = self.kinds.setdefault(kind, len(self.kinds))
        self.names.append(name)
        self.rows.append(rows)
        self.cols.append(cols)
        self.group.append(g)

    def finish(self, name: str, **kw) -> Workload:
        n_groups = len(self.kinds)
        sizes = [0] * n_groups
        two_d = [False] * n_groups
        for r, g in zip(self.rows, self.group):
            sizes[g] += 1
            two_d[g] = r > 1
        # matrices: shuffle (if repeated) + column sign flip; vectors: shuffle only
        gflags = [(SHUFFLE if sizes[g] > 1 else 0) | (FLIP if two_d[g] else 0)
                  for g in range(n_groups)]
        return Workload(name=name, layer_names=self.names, rows=self.rows, cols=self.cols,
                        group=self.group, gflags=gflags, **kw)


def _task_kw(n_tasks: int, first_seed: int):
    return dict(n_tasks=n_tasks, task_ids=list(range(n_tasks)),
                seeds=[first_seed + i for i in range(n_tasks)])


def toy(n_tasks: int = 4, width: int = 512, n_blocks: int = 6) -> Workload:
    b = _Builder()
    for k in range(n_blocks):
        b.add("block%d.W" % k, width, width, "W")
        b.add("block%d.b" % k, 1, width, "b")
    return b.finish("toy:f32", storage=F32, scale=1e-3, lam=1.0, data_seed=1000,
                    **_task_kw(n_tasks, 0))


def _vit(name, width, blocks, mlp, patch_rows, pos_rows, proj_out, **kw) -> Workload:
    b = _Builder()
    b.add("patch_embed", patch_rows, width)
    b.add("class_emb", 1, width)
    b.add("pos_emb", pos_rows, width)
    b.add("ln_pre.w", 1, width)
    b.add("ln_pre.b", 1, width)
    for k in range(blocks):
        p = "blocks.%d." % k
        b.add(p + "ln1.w", 1, width, "ln1.w")
        b.add(p + "ln1.b", 1, width, "ln1.b")
        b.add(p + "qkv.w", width, 3 * width, "qkv.w")
        b.add(p + "qkv.b", 1, 3 * width, "qkv.b")
        b.add(p + "out.w", width, width, "out.w")
        b.add(p + "out.b", 1, width, "out.b")
        b.add(p + "ln2.w", 1, width, "ln2.w")
        b.add(p + "ln2.b", 1, width, "ln2.b")
        b.add(p + "fc.w", width, mlp, "fc.w")
        b.add(p + "fc.b", 1, mlp, "fc.b")
        b.add(p + "proj.w", mlp, width, "proj.w")
        b.add(p + "proj.b", 1, width, "proj.b")
    b.add("ln_post.w", 1, width)
    b.add("ln_post.b", 1, width)
    b.add("proj", width, proj_out)
    return b.finish(name, **kw)


def vit_b32(n_tasks: int = 8) -> Workload:
    return _vit("vit_b32:f32", 768, 12, 3072, 3072, 50, 512, storage=F32, scale=1e-3,
                lam=0.3, data_seed=1001, **_task_kw(n_tasks, 42))


def vit_l14(n_tasks: int = 20, storage: int = F32) -> Workload:
    w = _vit("vit_l14:f32", 1024, 24, 4096, 588, 257, 768, storage=F32, scale=1e-3,
             lam=0.3, data_seed=1004, **_task_kw(n_tasks, 42))
    return w.with_storage(storage)


def gpt2_small(n_tasks: int = 7) -> Workload:
    b = _Builder()
    d, mlp = 768, 3072
    b.add("wte", 50257, d)
    b.add("wpe", 1024, d)
    for k in range(12):
        p = "h.%d." % k
        b.add(p + "ln1.w", 1, d, "ln1.w")
        b.add(p + "ln1.b", 1, d, "ln1.b")
        b.add(p + "c_attn.w", d, 3 * d, "c_attn.w")
        b.add(p + "c_attn.b", 1, 3 * d, "c_attn.b")
        b.add(p + "c_proj.w", d, d, "c_proj.w")
        b.add(p + "c_proj.b", 1, d, "c_proj.b")
        b.add(p + "ln2.w", 1, d, "ln2.w")
        b.add(p + "ln2.b", 1, d, "ln2.b")
        b.add(p + "c_fc.w", d, mlp, "c_fc.w")
        b.add(p + "c_fc.b", 1, mlp, "c_fc.b")
        b.add(p + "mlp_proj.w", mlp, d, "mlp_proj.w")
        b.add(p + "mlp_proj.b", 1, d, "mlp_proj.b")
    b.add("ln_f.w", 1, d)
    b.add("ln_f.b", 1, d)
    return b.finish("gpt2_small:bf16", storage=BF16, scale=5e-4, lam=0.5, data_seed=1002,
                    **_task_kw(n_tasks, 42))


def flan_t5_base(n_tasks: int = 8) -> Workload:
    b = _Builder()
    d, ff, vocab = 768, 2048, 32128
    b.add("shared", vocab, d)
    b.add("lm_head", vocab, d)
    b.add("enc.rel_bias", 32, 12)
    b.add("dec.rel_bias", 32, 12)
    b.add("enc.final_ln", 1, d)
    b.add("dec.final_ln", 1, d)
    for k in range(12):
        p = "enc.%d." % k
        for m in "qkvo":
            b.add(p + "sa." + m, d, d, "enc.sa." + m)
        b.add(p + "sa.ln", 1, d, "enc.sa.ln")
        b.add(p + "wi_0", d, ff, "enc.wi_0")
        b.add(p + "wi_1", d, ff, "enc.wi_1")
        b.add(p + "wo", ff, d, "enc.wo")
        b.add(p + "ff.ln", 1, d, "enc.ff.ln")
    for k in range(12):
        p = "dec.%d." % k
        for m in "qkvo":
            b.add(p + "sa." + m, d, d, "dec.sa." + m)
        b.add(p + "sa.ln", 1, d, "dec.sa.ln")
        for m in "qkvo":
            b.add(p + "ca." + m, d, d, "dec.ca." + m)
        b.add(p + "ca.ln", 1, d, "dec.ca.ln")
        b.add(p + "wi_0", d, ff, "dec.wi_0")
        b.add(p + "wi_1", d, ff, "dec.wi_1")
        b.add(p + "wo", ff, d, "dec.wo")
        b.add(p + "ff.ln", 1, d, "dec.ff.ln")
    return b.finish("flan_t5_base:f32", storage=F32, scale=1e-3, lam=0.5, data_seed=1003,
                    **_task_kw(n_tasks, 42))


def flan_t5_lora_targets(w: Workload) -> List[int]:
    """Layer indices that carry a LoRA delta: q and v of every attention module."""
    return [l for l, n in enumerate(w.layer_names)
            if n.endswith((".sa.q", ".sa.v", ".ca.q", ".ca.v"))]


def subset(w: Workload, layers: Sequence[int], name: Optional[str] = None) -> Workload:
    """A workload holding only the chosen layers (groups renumbered densely)."""
    remap: Dict[int, int] = {}
    group, gflags = [], []
    for l in layers:
        g = w.group[l]
        if g not in remap:
            remap[g] = len(remap)
            gflags.append(w.gflags[g])
        group.append(remap[g])
    sizes = [group.count(g) for g in range(len(gflags))]
    gflags = [f if sizes[g] > 1 else (f & ~SHUFFLE) for g, f in enumerate(gflags)]
    out = Workload(**{**w.__dict__})
    out.name = name or (w.name + ":subset")
    out.layer_names = [w.layer_names[l] for l in layers]
    out.rows = [w.rows[l] for l in layers]
    out.cols = [w.cols[l] for l in layers]
    out.group = group
    out.gflags = gflags
    return out


def row_slice(w: Workload, part: int, parts: int) -> Tuple[Workload, List[Tuple[int, int]]]:
    """The workload one of ``parts`` devices holds when every layer is cut into row slices.

    Returns the sliced workload (same layers, groups, flags, tasks and seeds; fewer rows)
    and, per layer, the (first row, one past last row) it covers.  The transforms move
    data across layers and flip by column, never across rows, so each slice can be
    compressed and retrieved on its own: no exchange between devices is needed.
    """
    bounds = []
    out = Workload(**{**w.__dict__})
    out.rows = []
    for r in w.rows:
        lo, hi = (r * part) // parts, (r * (part + 1)) // parts
        bounds.append((lo, hi))
        out.rows.append(hi - lo)
    out.name = "%s:rows %d/%d" % (w.name, part, parts)
    return out, bounds


CONFIGS = {
    0: toy,
    1: vit_b32,
    2: gpt2_small,
    3: flan_t5_base,
    4: vit_l14,
}


# --------------------------------------------------------------------------- values
_KIND_BASE, _KIND_SHARED, _KIND_PRIVATE, _KIND_LORA_A, _KIND_LORA_B, _KIND_MISC = range(6)


def _rng(w: Workload, kind: int, layer: int, task: int = 0) -> np.random.Generator:
    return np.random.default_rng([int(w.data_seed), kind, int(layer), int(task)])


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (round to nearest even), via torch's conversion."""
    import torch

    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32)


def _store(w: Workload, x32: np.ndarray) -> np.ndarray:
    return to_bf16_bits(x32) if w.storage == BF16 else np.ascontiguousarray(x32, dtype=np.float32)


def _base_f32(w: Workload, layer: int) -> np.ndarray:
    shape = (w.rows[layer], w.cols[layer])
    x = _rng(w, _KIND_BASE, layer).standard_normal(shape, dtype=np.float32)
    x *= np.float32(0.02)
    if w.storage == BF16:
        x = bf16_bits_to_f32(to_bf16_bits(x))
    return x


def base_layer(w: Workload, layer: int) -> np.ndarray:
    """W_0 of one layer in storage dtype (float32, or uint16 bf16 bit patterns)."""
    x = _base_f32(w, layer)
    return to_bf16_bits(x) if w.storage == BF16 else x


def delta_f32(w: Workload, layer: int, task_id: int, shared: Optional[np.ndarray] = None) -> np.ndarray:
    shape = (w.rows[layer], w.cols[layer])
    if shared is None:
        shared = _rng(w, _KIND_SHARED, layer).standard_normal(shape, dtype=np.float32)
    e = _rng(w, _KIND_PRIVATE, layer, task_id).standard_normal(shape, dtype=np.float32)
    e *= np.float32(math.sqrt(0.75))
    e += np.float32(0.5) * shared
    e *= np.float32(w.scale)
    return e


def task_layer(w: Workload, layer: int, task_id: int, base32: Optional[np.ndarray] = None,
               shared: Optional[np.ndarray] = None) -> np.ndarray:
    """W_i of one layer in storage dtype; ``task_id`` selects the private stream."""
    if base32 is None:
        base32 = _base_f32(w, layer)
    return _store(w, base32 + delta_f32(w, layer, task_id, shared))


def layer_all_tasks(w: Workload, layer: int, task_ids: Sequence[int]) -> Tuple[np.ndarray, List[np.ndarray]]:
    """(W_0, [W_i for i in task_ids]) of one layer, sharing the common draws."""
    shape = (w.rows[layer], w.cols[layer])
    base32 = _base_f32(w, layer)
    shared = _rng(w, _KIND_SHARED, layer).standard_normal(shape, dtype=np.float32)
    tasks = [task_layer(w, layer, t, base32, shared) for t in task_ids]
    return _store(w, base32), tasks


def model_set(w: Workload, task_ids: Optional[Sequence[int]] = None, threads: int = 8):
    """(base, tasks): base[l], tasks[i][l] for the whole workload, generated in parallel."""
    from concurrent.futures import ThreadPoolExecutor

    task_ids = list(w.task_ids if task_ids is None else task_ids)
    with ThreadPoolExecutor(max_workers=max(1, threads)) as ex:
        res = list(ex.map(lambda l: layer_all_tasks(w, l, task_ids), range(w.n_layers)))
    base = [r[0] for r in res]
    tasks = [[r[1][i] for r in res] for i in range(len(task_ids))]
    return base, tasks


def lora_delta_layer(w: Workload, layer: int, task_id: int, rank: int = 16, std: float = 0.01) -> np.ndarray:
    """delta = B A of a rank-``rank`` adapter, materialised in fp32 then stored.

    A is [rank, cols], B is [rows, rank], both N(0, std^2).  Section 5.8 of the
    paper compresses such adapter deltas; rank and std are this repository's
    choice (the paper states neither).
    """
    rows, cols = w.rows[layer], w.cols[layer]
    A = _rng(w, _KIND_LORA_A, layer, task_id).standard_normal((rank, cols), dtype=np.float32) * np.float32(std)
    B = _rng(w, _KIND_LORA_B, layer, task_id).standard_normal((rows, rank), dtype=np.float32) * np.float32(std)
    d = np.zeros((rows, cols), dtype=np.float32)
    for k in range(rank):  # k-ascending fp32 accumulation
        d += np.outer(B[:, k], A[k, :]).astype(np.float32)
    return _store(w, d)


def dyadic_model_set(w: Workload, task_ids: Sequence[int], denom_log2: int = 10, span: int = 1 << 10):
    """Weights on the grid k / 2^denom_log2, |k| <= span: every fp32 (and bf16-free)
    sum the path forms is exact, so add followed by remove restores M bit for bit."""
    assert w.storage == F32
    base, tasks = [], [[] for _ in task_ids]
    for l in range(w.n_layers):
        shape = (w.rows[l], w.cols[l])
        k0 = _rng(w, _KIND_MISC, l).integers(-span, span + 1, size=shape)
        base.append((k0 / float(1 << denom_log2)).astype(np.float32))
        for j, t in enumerate(task_ids):
            kt = _rng(w, _KIND_MISC, l, t + 1).integers(-span, span + 1, size=shape)
            tasks[j].append((kt / float(1 << denom_log2)).astype(np.float32))
    return base, tasks
