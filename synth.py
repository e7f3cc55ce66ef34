"""Seeded synthetic gradient workloads.

Input generation only: nothing here selects, quantises or sums anything.
The buckets stand in for real training gradients (the paper trained
ResNet18 / VGG16 on CIFAR-100; neither data nor trained weights are needed to
exercise the compression path).  They take tensor shapes from the public
architectures named below and the value structure listed per generator.

Every tensor is drawn from its own generator seeded with (seed, tensor index),
so any bucket of a large gradient set can be produced without generating the
rest.
"""
from __future__ import annotations

from typing import Iterator, List, Sequence, Tuple

import numpy as np

Shape = Tuple[str, Tuple[int, ...]]


# --------------------------------------------------------------------------
# tensor-shape lists
# --------------------------------------------------------------------------
def resnet50_shapes() -> List[Shape]:
    """Parameter tensors of ResNet-50 (7x7 stem, bottleneck stages [3,4,6,3],
    widths 64/128/256/512 with 4x expansion, a BatchNorm weight and bias after
    every convolution, 2048->1000 classifier with bias): 161 tensors,
    25,557,032 elements."""
    shapes: List[Shape] = [("conv1.w", (64, 3, 7, 7)), ("bn1.w", (64,)), ("bn1.b", (64,))]
    cin = 64
    for s, (blocks, width) in enumerate(zip((3, 4, 6, 3), (64, 128, 256, 512))):
        for b in range(blocks):
            p = f"layer{s + 1}.{b}"
            shapes += [
                (p + ".conv1.w", (width, cin, 1, 1)), (p + ".bn1.w", (width,)), (p + ".bn1.b", (width,)),
                (p + ".conv2.w", (width, width, 3, 3)), (p + ".bn2.w", (width,)), (p + ".bn2.b", (width,)),
                (p + ".conv3.w", (4 * width, width, 1, 1)), (p + ".bn3.w", (4 * width,)), (p + ".bn3.b", (4 * width,)),
            ]
            if b == 0:
                shapes += [
                    (p + ".down.w", (4 * width, cin, 1, 1)), (p + ".down.bn.w", (4 * width,)),
                    (p + ".down.bn.b", (4 * width,)),
                ]
            cin = 4 * width
    shapes += [("fc.w", (1000, 2048)), ("fc.b", (1000,))]
    return shapes


def _decoder_shapes(layers: int, d: int, ffn: int, vocab: int, npos: int) -> List[Shape]:
    shapes: List[Shape] = [("wte", (vocab, d)), ("wpe", (npos, d))]
    for l in range(layers):
        p = f"h{l}"
        shapes += [
            (p + ".ln1.w", (d,)), (p + ".ln1.b", (d,)),
            (p + ".attn.qkv.w", (d, 3 * d)), (p + ".attn.qkv.b", (3 * d,)),
            (p + ".attn.proj.w", (d, d)), (p + ".attn.proj.b", (d,)),
            (p + ".ln2.w", (d,)), (p + ".ln2.b", (d,)),
            (p + ".mlp.fc.w", (d, ffn)), (p + ".mlp.fc.b", (ffn,)),
            (p + ".mlp.proj.w", (ffn, d)), (p + ".mlp.proj.b", (d,)),
        ]
    shapes += [("lnf.w", (d,)), ("lnf.b", (d,))]
    return shapes


def gpt2_small_shapes() -> List[Shape]:
    """GPT-2 small (12 layers, d=768, ffn 3072, vocab 50257, 1024 positions):
    124,439,808 elements."""
    return _decoder_shapes(12, 768, 3072, 50257, 1024)


def decoder_1p3b_shapes() -> List[Shape]:
    """A 1.3B-parameter decoder (24 layers, d=2048, ffn 8192; vocab 50257 and
    2048 positions assumed): 1,315,723,264 elements."""
    return _decoder_shapes(24, 2048, 8192, 50257, 2048)


def numel(shape: Sequence[int]) -> int:
    out = 1
    for s in shape:
        out *= int(s)
    return out


def total_elements(shapes: Sequence[Shape]) -> int:
    return sum(numel(s) for _, s in shapes)


def bucket_ranges(total: int, bucket_elems: int) -> List[Tuple[int, int]]:
    """Flat concatenation in layer order cut at fixed element counts; the
    last bucket is short."""
    return [(lo, min(total, lo + bucket_elems)) for lo in range(0, total, bucket_elems)]


# --------------------------------------------------------------------------
# value generators
# --------------------------------------------------------------------------
def config1_bucket(n: int = 1 << 20, seed: int = 0) -> np.ndarray:
    """Single fp32 vector: per 4096-element block a scale 10**U(-4,-1) times
    N(0,1); then an i.i.d. 20 % of the elements set to exactly +0.0."""
    rng = np.random.default_rng([seed, 1])
    nblk = (n + 4095) // 4096
    scale = (10.0 ** rng.uniform(-4.0, -1.0, nblk)).astype(np.float32)
    g = rng.standard_normal(n, dtype=np.float32) * np.repeat(scale, 4096)[:n]
    g[rng.random(n) < 0.2] = np.float32(0.0)
    return g.astype(np.float32)


def _resnet_tensor(rng: np.random.Generator, count: int) -> np.ndarray:
    scale = 10.0 ** rng.uniform(-5.0, -1.0)
    g = rng.standard_normal(count, dtype=np.float32) * np.float32(scale)
    outl = rng.random(count) < 0.05
    g[outl] = rng.laplace(0.0, 10.0 * scale, int(outl.sum())).astype(np.float32)
    return g


def _gauss_tensor(rng: np.random.Generator, count: int, lo_exp: float, hi_exp: float) -> np.ndarray:
    sigma = 10.0 ** rng.uniform(lo_exp, hi_exp)
    return rng.standard_normal(count, dtype=np.float32) * np.float32(sigma)


def _embedding_90pct_zero_rows(rng: np.random.Generator, rows: int, cols: int) -> np.ndarray:
    sigma = 10.0 ** rng.uniform(-4.0, -2.0)
    g = rng.standard_normal(rows * cols, dtype=np.float32).reshape(rows, cols) * np.float32(sigma)
    g[rng.random(rows) < 0.9, :] = np.float32(0.0)
    return g.reshape(-1)


def _tensor_values(kind: str, t: int, name: str, shape: Sequence[int], seed: int) -> np.ndarray:
    rng = np.random.default_rng([seed, t])
    count = numel(shape)
    if kind == "resnet50":
        # per-tensor scale log-uniform [1e-5, 1e-1]; 95 % Gaussian, 5 % Laplace
        # outliers ten times wider
        return _resnet_tensor(rng, count)
    if kind == "gpt2":
        # token-embedding rows 90 % zero; everything else Gaussian with a
        # per-tensor sigma log-uniform [1e-4, 1e-2]
        if name == "wte":
            return _embedding_90pct_zero_rows(rng, shape[0], shape[1])
        return _gauss_tensor(rng, count, -4.0, -2.0)
    if kind == "decoder":
        # Gaussian, per-tensor sigma log-uniform [1e-6, 1e-2]
        return _gauss_tensor(rng, count, -6.0, -2.0)
    raise ValueError(kind)


def flat_slice(kind: str, shapes: Sequence[Shape], lo: int, hi: int, seed: int) -> np.ndarray:
    """float32 values of flat positions [lo, hi) of the concatenated gradient
    set; only the tensors that overlap the range are generated."""
    out = np.empty(hi - lo, dtype=np.float32)
    pos = 0
    for t, (name, shape) in enumerate(shapes):
        cnt = numel(shape)
        a, b = max(lo, pos), min(hi, pos + cnt)
        if a < b:
            vals = _tensor_values(kind, t, name, shape, seed)
            out[a - lo:b - lo] = vals[a - pos:b - pos]
        pos += cnt
        if pos >= hi:
            break
    return out


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 bit patterns (nearest even); used only to
    produce bf16-typed inputs."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    r = (b + np.uint64(0x7FFF) + ((b >> np.uint64(16)) & np.uint64(1))) >> np.uint64(16)
    return r.astype(np.uint16)


def resnet50_buckets(seed: int = 1, bucket_elems: int = 6_553_600) -> Iterator[np.ndarray]:
    shapes = resnet50_shapes()
    for lo, hi in bucket_ranges(total_elements(shapes), bucket_elems):
        yield flat_slice("resnet50", shapes, lo, hi, seed)


def gpt2_bucket(b: int, seed: int, bucket_elems: int = 25_000_000) -> np.ndarray:
    shapes = gpt2_small_shapes()
    lo, hi = bucket_ranges(total_elements(shapes), bucket_elems)[b]
    return flat_slice("gpt2", shapes, lo, hi, seed)


def decoder_bucket_bf16(b: int, seed: int = 20, bucket_elems: int = 1 << 26) -> np.ndarray:
    """bf16 bit patterns (uint16) of bucket b of the 1.3B decoder set."""
    shapes = decoder_1p3b_shapes()
    lo, hi = bucket_ranges(total_elements(shapes), bucket_elems)[b]
    return f32_to_bf16_bits(flat_slice("decoder", shapes, lo, hi, seed))


# --------------------------------------------------------------------------
# synthetic payload contents (aggregation stress)
# --------------------------------------------------------------------------
def _mix32(x: np.ndarray) -> np.ndarray:
    """A 32-bit integer finaliser (xor-shift / multiply), for jitter only."""
    x = x.astype(np.uint64) & np.uint64(0xFFFFFFFF)
    x ^= x >> np.uint64(16)
    x = (x * np.uint64(0x7FEB352D)) & np.uint64(0xFFFFFFFF)
    x ^= x >> np.uint64(15)
    x = (x * np.uint64(0x846CA68B)) & np.uint64(0xFFFFFFFF)
    x ^= x >> np.uint64(16)
    return x


def stress_payload_parts(n: int, k: int, worker_seed: int, shared_seed: int,
                         overlap: float = 0.3, qblock: int = 1024):
    """Contents of one synthetic int8 payload: k strictly ascending indices by
    jittered stride (entry j falls in [j*stride, (j+1)*stride); its jitter uses
    a seed shared by all workers with probability `overlap`, else the worker's
    own, so about that fraction of indices coincide across workers), codes
    uniform in [-127, 127], block scales log-uniform in [1e-6, 1e-2]."""
    stride = n // k
    if stride < 1:
        raise ValueError("k must not exceed n")
    j = np.arange(k, dtype=np.uint64)
    pick_shared = (_mix32(j * np.uint64(2654435761) + np.uint64(shared_seed) * np.uint64(97)) % np.uint64(1000)) \
        < np.uint64(int(overlap * 1000))
    seed_j = np.where(pick_shared, np.uint64(shared_seed), np.uint64(worker_seed))
    jitter = _mix32(j ^ (seed_j * np.uint64(0x9E3779B1))) % np.uint64(stride)
    idx = (j * np.uint64(stride) + jitter).astype(np.uint32)
    rng = np.random.default_rng([worker_seed, 5])
    codes = rng.integers(-127, 128, size=k, dtype=np.int8)
    nblocks = (k + qblock - 1) // qblock
    scales = (10.0 ** rng.uniform(-6.0, -2.0, nblocks)).astype(np.float32)
    return idx, codes, scales
