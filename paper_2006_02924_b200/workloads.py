"""Seeded synthetic gradient workloads (input generation only; none of the method's arithmetic).

The paper reduces the per-layer gradients of ResNet-50 and BERT-Large across workers.  Neither
its datasets nor trained weights are needed to exercise the combine itself: what matters is the
tensor list (how many layers, how large each one is), the dtype, the number of workers and how
correlated the workers' gradients are (they start nearly parallel and grow orthogonal during
training).  This module builds those lists from the architectures' public hyper-parameters and
fills them with correlated Gaussians:

    g[w, l] = sigma_l * (sqrt(rho_l) * s_l + sqrt(1 - rho_l) * n[w, l]),   s_l, n ~ N(0, 1)

so that the expected cosine between two workers' tensors is rho_l.  The generated bits are the
single source of truth handed to every consumer.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np
import torch

BASE_SEED = 20060292400


def resnet50_tensor_sizes() -> list[int]:
    """Parameter tensors of ResNet-50 v1.5 in module order: 161 tensors, 25,557,032 elements."""
    sizes = [64 * 3 * 7 * 7, 64, 64]                      # stem conv + BN (weight, bias)
    in_ch = 64
    for width, blocks in ((64, 3), (128, 4), (256, 6), (512, 3)):
        for block in range(blocks):
            sizes += [width * in_ch, width, width]         # 1x1 reduce + BN
            sizes += [width * width * 9, width, width]     # 3x3 + BN
            sizes += [4 * width * width, 4 * width, 4 * width]  # 1x1 expand + BN
            if block == 0:
                sizes += [4 * width * in_ch, 4 * width, 4 * width]  # downsample conv + BN
            in_ch = 4 * width
    sizes += [1000 * 2048, 1000]                           # classifier
    return sizes


def bert_large_tensor_sizes() -> list[int]:
    """Parameter tensors of BERT-Large (24 layers, hidden 1024, FFN 4096, vocab 30522,
    512 positions): 391 tensors, 335,141,888 elements."""
    h, ffn = 1024, 4096
    sizes = [30522 * h, 512 * h, 2 * h, h, h]              # embeddings + LayerNorm
    for _ in range(24):
        sizes += [h * h, h] * 4                            # Q, K, V, attention output
        sizes += [h, h]                                    # LayerNorm
        sizes += [ffn * h, ffn, h * ffn, h]                # FFN in / out
        sizes += [h, h]                                    # LayerNorm
    sizes += [h * h, h]                                    # pooler
    return sizes


@dataclasses.dataclass(frozen=True)
class WorkloadSpec:
    name: str
    n_workers: int
    dtype: str                     # "f32" | "f16" | "bf16"
    tensor_list: str               # "single" | "resnet50" | "bert_large"
    rho: tuple[float, float]       # rho_l drawn uniformly in [lo, hi] (lo == hi: constant)
    sigma: tuple[float, float]     # sigma_l log-uniform in [lo, hi]
    zero_tensor_fraction: float = 0.0   # this share of tensors is exactly zero on half the workers
    seed_index: int = 0

    def tensor_sizes(self) -> list[int]:
        if self.tensor_list == "single":
            return [1_000_000]
        if self.tensor_list == "resnet50":
            return resnet50_tensor_sizes()
        if self.tensor_list == "bert_large":
            return bert_large_tensor_sizes()
        raise ValueError(self.tensor_list)


# The five benchmark configurations.
SPECS = {
    "c1": WorkloadSpec("c1", 2, "f32", "single", (0.5, 0.5), (1.0, 1.0), seed_index=1),
    "c2": WorkloadSpec("c2", 8, "f32", "resnet50", (0.3, 0.3), (1e-4, 1e-1), seed_index=2),
    "c3": WorkloadSpec("c3", 16, "f32", "bert_large", (0.3, 0.3), (1e-4, 1e-1), seed_index=3),
    "c4": WorkloadSpec("c4", 64, "f16", "bert_large", (0.0, 0.9), (1e-5, 1e-1), seed_index=4),
    "c5": WorkloadSpec("c5", 256, "f32", "resnet50", (0.1, 0.1), (1e-4, 1e-1),
                       zero_tensor_fraction=0.05, seed_index=5),
}

TORCH_DTYPES = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16, "f64": torch.float64}
DTYPE_BYTES = {"f32": 4, "f16": 2, "bf16": 2, "f64": 8}


@dataclasses.dataclass
class Workload:
    spec: WorkloadSpec
    grads: list                    # N tensors, each one fused buffer of total_elems elements
    offsets: np.ndarray            # int64, num_tensors + 1
    rho: np.ndarray                # per tensor
    sigma: np.ndarray              # per tensor
    zeroed: dict                   # tensor index -> sorted list of workers whose copy is zero

    @property
    def n_workers(self) -> int:
        return len(self.grads)

    @property
    def total_elems(self) -> int:
        return int(self.offsets[-1])

    @property
    def num_tensors(self) -> int:
        return len(self.offsets) - 1

    @property
    def input_bytes(self) -> int:
        return self.n_workers * self.total_elems * DTYPE_BYTES[self.spec.dtype]


def offsets_from_sizes(sizes) -> np.ndarray:
    offs = np.zeros(len(sizes) + 1, dtype=np.int64)
    np.cumsum(np.asarray(sizes, dtype=np.int64), out=offs[1:])
    return offs


def per_tensor_parameters(spec: WorkloadSpec, num_tensors: int):
    """rho_l, sigma_l and the zeroed (tensor -> workers) map, drawn on the host from the seed."""
    rng = np.random.Generator(np.random.Philox(BASE_SEED + spec.seed_index))
    rho = rng.uniform(spec.rho[0], spec.rho[1], size=num_tensors)
    sigma = np.exp(rng.uniform(math.log(spec.sigma[0]), math.log(spec.sigma[1]), size=num_tensors))
    zeroed = {}
    if spec.zero_tensor_fraction > 0.0:
        count = max(1, int(round(spec.zero_tensor_fraction * num_tensors)))
        tensors = rng.choice(num_tensors, size=min(count, num_tensors), replace=False)
        for t in sorted(int(v) for v in tensors):
            workers = rng.choice(spec.n_workers, size=spec.n_workers // 2, replace=False)
            zeroed[t] = sorted(int(v) for v in workers)
    return rho, sigma, zeroed


def generate(spec: WorkloadSpec | str, device="cpu", tensor_sizes=None, n_workers=None,
             replica: int = 0) -> Workload:
    """Materialise a workload on ``device``.  ``tensor_sizes`` / ``n_workers`` override the
    spec's (used for reduced-size test cases that keep the same structure); ``replica`` selects
    an independent draw of the element noise (one per GPU in a multi-GPU run)."""
    if isinstance(spec, str):
        spec = SPECS[spec]
    if n_workers is not None:
        spec = dataclasses.replace(spec, n_workers=int(n_workers))
    sizes = list(tensor_sizes) if tensor_sizes is not None else spec.tensor_sizes()
    offsets = offsets_from_sizes(sizes)
    total = int(offsets[-1])
    rho, sigma, zeroed = per_tensor_parameters(spec, len(sizes))
    device = torch.device(device)
    seed = BASE_SEED + 1000 * spec.seed_index + 100_000 * int(replica)

    lengths = torch.as_tensor(np.asarray(sizes, dtype=np.int64), device=device)
    shared_scale = torch.repeat_interleave(
        torch.as_tensor(sigma * np.sqrt(rho), dtype=torch.float32, device=device), lengths)
    noise_scale = torch.repeat_interleave(
        torch.as_tensor(sigma * np.sqrt(1.0 - rho), dtype=torch.float32, device=device), lengths)
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    shared = torch.randn(total, generator=gen, device=device, dtype=torch.float32)
    shared.mul_(shared_scale)
    del shared_scale

    # The N worker buffers are the rows of one [N, pitch] allocation, pitch = the buffer length rounded
    # up to 64 elements (what stacking the workers' fused buffers gives); each is handed out as a
    # separate one-dimensional view.
    pitch = (total + 63) // 64 * 64
    store = torch.zeros((spec.n_workers, max(pitch, 1)), dtype=TORCH_DTYPES[spec.dtype], device=device)
    grads = []
    for w in range(spec.n_workers):
        gen.manual_seed(seed + 1 + w)
        g = torch.randn(total, generator=gen, device=device, dtype=torch.float32)
        g.mul_(noise_scale).add_(shared)
        for t, workers in zeroed.items():
            if w in workers:
                g[int(offsets[t]):int(offsets[t + 1])] = 0.0
        store[w, :total].copy_(g)
        grads.append(store[w, :total])
        del g
    return Workload(spec, grads, offsets, rho, sigma, zeroed)


def reduced_sizes(sizes, divisor: int, keep_ragged: bool = True, smallest: int = 16) -> list[int]:
    """Shrink a tensor list for quick tests while keeping its shape mix; optionally make some
    sizes odd so that tensor starts lose their vector alignment.  Tensors are not shrunk below
    `smallest` elements: a one-element "tensor" of many weakly correlated workers is a sum of
    scalars of random sign, which no floating-point evaluation of the method resolves."""
    out = []
    for i, s in enumerate(sizes):
        r = max(min(smallest, s), s // divisor)
        if keep_ragged and i % 3 == 1:
            r += 1 + (i % 5)
        out.append(r)
    return out


def element_shards(offsets, world: int, align: int = 64):
    """Split every tensor of a fused buffer into `world` contiguous element ranges (the layout the
    element-sharded reduce expects: rank r holds piece r of every tensor).  Cuts are rounded to
    `align` elements, so short tensors live on the first ranks only and are empty elsewhere.
    Returns, per rank, (local_offsets, pieces) with pieces[t] = (lo, hi) in the global buffer."""
    offsets = np.asarray(offsets, dtype=np.int64)
    shards = []
    for rank in range(world):
        pieces, sizes = [], []
        for t in range(len(offsets) - 1):
            lo, hi = int(offsets[t]), int(offsets[t + 1])
            per = -(-(hi - lo) // world)
            per = -(-per // align) * align
            a = min(hi, lo + rank * per)
            b = min(hi, lo + (rank + 1) * per)
            pieces.append((a, b))
            sizes.append(b - a)
        shards.append((offsets_from_sizes(sizes), pieces))
    return shards
