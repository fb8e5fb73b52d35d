"""Seeded synthetic inputs: block shapes and gradient streams.

This module holds input generators only.  It describes the tensor shapes of
the five benchmark workloads (toy, ResNet-50-, GPT-2-small-, diffusion-UNet-
and LLaMA-1B-shaped) and draws reproducible bf16 gradient streams, fp32
parameters and time-ratio tables for them.  None of the method's arithmetic
(statistics, risk, allocation, update rules) lives here, so both the CUDA
library's tests and the CPU oracle's tests can use it without sharing any
code of the method.

Gradient model (one definition for every workload).  For block ``b`` with
stability ``a_b`` in [0, 1], log-normal width ``tau_b`` and scale ``s_b``:

    g_t[j] = bf16( s_b * sigma_j * ( sqrt(a_b) * u_j + sqrt(1 - a_b) * xi_{t,j} ) )

``u_j`` (a fixed direction) and ``sigma_j = exp(tau_b * n_j)`` are drawn once
per block, ``xi_{t,j}`` is drawn per step (standard normal, or Student-t with
3 degrees of freedom for heavy-tailed blocks).  The expected cosine between
successive gradients is then close to ``a_b``.  Every draw comes from a
``torch.Generator`` whose seed is a hash of (seed, block, stream id, step),
so any block at any step can be regenerated on its own.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence

import torch

_MASK64 = (1 << 64) - 1


def _mix64(x: int) -> int:
    """SplitMix64 finaliser: a bijective 64-bit hash."""
    x = (x + 0x9E3779B97F4A7C15) & _MASK64
    x = ((x ^ (x >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & _MASK64
    return x ^ (x >> 31)


def stream_seed(seed: int, block: int, stream: int, step: int = 0) -> int:
    """Seed of the generator for (seed, block, stream, step)."""
    h = _mix64(seed & _MASK64)
    h = _mix64(h ^ (block + 1))
    h = _mix64(h ^ ((stream + 1) << 20))
    h = _mix64(h ^ ((step + 1) << 40))
    return h & ((1 << 63) - 1)


@dataclasses.dataclass
class Block:
    """One parameter block: ``numel`` parameters viewed as rows x cols.

    A 1-D tensor has rows = numel and cols = 1.  Tensors with more than two
    dimensions are flattened to (dim0, product of the rest).
    """

    name: str
    rows: int
    cols: int
    stability: float = 0.5      # a_b
    tau: float = 1.0            # width of the log-normal per-coordinate scale
    scale: float = 1e-2         # s_b
    heavy_tail: bool = False    # Student-t(3) step noise instead of normal

    @property
    def numel(self) -> int:
        return self.rows * self.cols

    @property
    def is_matrix(self) -> bool:
        return self.cols > 1


@dataclasses.dataclass
class Workload:
    name: str
    blocks: List[Block]
    window: int                 # T, length of the sampling window
    mem_budget_frac: float      # fraction of the all-fp32-Adam state bytes (8 B per parameter)
    time_budget: float          # B_time, in units of the plain fp32 Adam step
    seed: int = 0

    @property
    def numel(self) -> int:
        return sum(b.numel for b in self.blocks)


def _mat(name: str, rows: int, cols: int) -> Block:
    return Block(name, rows, cols)


def _vec(name: str, n: int) -> Block:
    return Block(name, n, 1)


# ----------------------------------------------------------------------------
# Shapes
# ----------------------------------------------------------------------------

def _toy_blocks() -> List[Block]:
    # Multiset {256x256 x4, 512x512 x1, 1024x256 x2, 256 x5}: 12 blocks, 1 049 856 parameters.
    shapes = [(256, 256), (512, 512), (1024, 256), (256, 1), (256, 256), (256, 1),
              (1024, 256), (256, 1), (256, 256), (256, 1), (256, 256), (256, 1)]
    return [Block(f"toy{i}", r, c) for i, (r, c) in enumerate(shapes)]


def _resnet50_blocks() -> List[Block]:
    out: List[Block] = []

    def conv(name, cout, cin, k):
        out.append(_mat(name, cout, cin * k * k))

    def norm(name, c):
        out.append(_vec(name + ".scale", c))
        out.append(_vec(name + ".shift", c))

    conv("stem.conv", 64, 3, 7)
    norm("stem.norm", 64)
    cin = 64
    for s, (n_blk, width) in enumerate(zip([3, 4, 6, 3], [64, 128, 256, 512])):
        for k in range(n_blk):
            p = f"stage{s}.{k}"
            conv(p + ".conv1", width, cin, 1); norm(p + ".norm1", width)
            conv(p + ".conv2", width, width, 3); norm(p + ".norm2", width)
            conv(p + ".conv3", width * 4, width, 1); norm(p + ".norm3", width * 4)
            if k == 0:
                conv(p + ".down", width * 4, cin, 1); norm(p + ".down_norm", width * 4)
            cin = width * 4
    out.append(_mat("head.weight", 1000, 2048))
    out.append(_vec("head.bias", 1000))
    return out


def _gpt2_small_blocks() -> List[Block]:
    d, ff, layers, vocab, ctx = 768, 3072, 12, 50257, 1024
    out = [_mat("tok_emb", vocab, d), _mat("pos_emb", ctx, d)]
    for l in range(layers):
        p = f"h{l}"
        out += [_vec(p + ".ln1.w", d), _vec(p + ".ln1.b", d),
                _mat(p + ".attn.qkv.w", d, 3 * d), _vec(p + ".attn.qkv.b", 3 * d),
                _mat(p + ".attn.out.w", d, d), _vec(p + ".attn.out.b", d),
                _vec(p + ".ln2.w", d), _vec(p + ".ln2.b", d),
                _mat(p + ".mlp.fc.w", d, ff), _vec(p + ".mlp.fc.b", ff),
                _mat(p + ".mlp.proj.w", ff, d), _vec(p + ".mlp.proj.b", d)]
    out += [_vec("ln_f.w", d), _vec("ln_f.b", d)]
    return out


def _llama_1b_blocks(layers: int = 16, with_table: bool = True) -> List[Block]:
    d, ff, vocab = 2048, 8192, 32000
    out = [_mat("tok_emb", vocab, d)] if with_table else []
    for l in range(layers):
        p = f"l{l}"
        out += [_vec(p + ".norm1", d)]
        out += [_mat(p + f".attn.{n}", d, d) for n in ("q", "k", "v", "o")]
        out += [_vec(p + ".norm2", d)]
        out += [_mat(p + ".ffn.gate", ff, d), _mat(p + ".ffn.up", ff, d), _mat(p + ".ffn.down", d, ff)]
    out += [_vec("norm_f", d)]
    return out


def _unet_blocks() -> List[Block]:
    """Latent-diffusion-style UNet: channels 320/640/1280/1280, two residual
    blocks per level, cross-attention to a 768-wide context."""
    out: List[Block] = []
    temb, ctx = 1280, 768

    def conv(name, cout, cin, k, bias=True):
        out.append(_mat(name + ".w", cout, cin * k * k))
        if bias:
            out.append(_vec(name + ".b", cout))

    def lin(name, cout, cin, bias=True):
        out.append(_mat(name + ".w", cout, cin))
        if bias:
            out.append(_vec(name + ".b", cout))

    def norm(name, c):
        out.append(_vec(name + ".w", c))
        out.append(_vec(name + ".b", c))

    def res(name, cin, cout):
        norm(name + ".norm1", cin); conv(name + ".conv1", cout, cin, 3)
        lin(name + ".temb", cout, temb)
        norm(name + ".norm2", cout); conv(name + ".conv2", cout, cout, 3)
        if cin != cout:
            conv(name + ".skip", cout, cin, 1)

    def xf(name, d):
        norm(name + ".norm", d); conv(name + ".proj_in", d, d, 1)
        norm(name + ".ln1", d)
        for n in ("q", "k", "v"):
            lin(name + ".self." + n, d, d, bias=False)
        lin(name + ".self.o", d, d)
        norm(name + ".ln2", d)
        lin(name + ".cross.q", d, d, bias=False)
        lin(name + ".cross.k", d, ctx, bias=False)
        lin(name + ".cross.v", d, ctx, bias=False)
        lin(name + ".cross.o", d, d)
        norm(name + ".ln3", d)
        lin(name + ".ff.gate", 8 * d, d); lin(name + ".ff.out", d, 4 * d)
        conv(name + ".proj_out", d, d, 1)

    chans = [320, 640, 1280, 1280]
    conv("in", 320, 4, 3)
    lin("time.0", temb, 320); lin("time.1", temb, temb)
    skips = [320]
    c = 320
    for lvl, ch in enumerate(chans):
        for k in range(2):
            res(f"down{lvl}.res{k}", c, ch); c = ch
            if lvl < 3:
                xf(f"down{lvl}.attn{k}", ch)
            skips.append(c)
        if lvl < 3:
            conv(f"down{lvl}.downsample", ch, ch, 3); skips.append(c)
    res("mid.res0", c, c); xf("mid.attn", c); res("mid.res1", c, c)
    for lvl in (3, 2, 1, 0):
        ch = chans[lvl]
        for k in range(3):
            res(f"up{lvl}.res{k}", c + skips.pop(), ch); c = ch
            if lvl < 3:
                xf(f"up{lvl}.attn{k}", ch)
        if lvl > 0:
            conv(f"up{lvl}.upsample", ch, ch, 3)
    norm("out.norm", 320); conv("out", 4, 320, 3)
    return out


def _level_of(name: str) -> int:
    for tag in ("down", "up"):
        if name.startswith(tag):
            return int(name[len(tag)])
    return 3 if name.startswith("mid") else 0


def make_workload(name: str, seed: int = 0) -> Workload:
    """Build one of: toy, resnet50, gpt2_small, unet, llama_1b (and llama_2l, a two-layer cut of it for profiling)."""
    if name == "toy":
        wl = Workload(name, _toy_blocks(), window=8, mem_budget_frac=0.50, time_budget=1.3, seed=seed)
    elif name == "resnet50":
        wl = Workload(name, _resnet50_blocks(), window=32, mem_budget_frac=0.40, time_budget=1.1, seed=seed)
    elif name == "gpt2_small":
        wl = Workload(name, _gpt2_small_blocks(), window=32, mem_budget_frac=0.35, time_budget=1.3, seed=seed)
    elif name == "unet":
        wl = Workload(name, _unet_blocks(), window=32, mem_budget_frac=0.30, time_budget=1.05, seed=seed)
    elif name == "llama_1b":
        wl = Workload(name, _llama_1b_blocks(), window=64, mem_budget_frac=0.25, time_budget=1.3, seed=seed)
    elif name == "llama_2l":
        # two layers of the LLaMA-1B shape without the token table (121.6 M parameters): same matrix shapes as the
        # full workload at a size small enough for multi-pass profiler captures
        wl = Workload(name, _llama_1b_blocks(2, False), window=64, mem_budget_frac=0.25, time_budget=1.3, seed=seed)
    else:
        raise ValueError(f"unknown workload {name!r}")

    # Per-block generator parameters, drawn from one generator per workload.
    gen = torch.Generator().manual_seed(stream_seed(seed, 1 << 19, 7))
    u = torch.rand((len(wl.blocks), 3), generator=gen, dtype=torch.float64)
    for i, b in enumerate(wl.blocks):
        lo, hi = (0.05, 0.95) if name.startswith("llama") else (0.0, 1.0)
        b.stability = float(lo + (hi - lo) * u[i, 0])
        b.tau = float(2.0 * u[i, 1])
        b.scale = float(10.0 ** (-3.0 + 2.0 * u[i, 2]))
        if name == "unet":
            # per-level noise scale 0.1 .. 10, log-spaced over the four levels
            b.scale = 1e-2 * 10.0 ** (-1.0 + 2.0 * _level_of(b.name) / 3.0)
        if name == "gpt2_small":
            b.heavy_tail = ("emb" in b.name) or (".attn." in b.name)
    return wl


WORKLOADS = ("toy", "resnet50", "gpt2_small", "unet", "llama_1b")


# ----------------------------------------------------------------------------
# Streams
# ----------------------------------------------------------------------------

def _gen(device, seed: int) -> torch.Generator:
    return torch.Generator(device=device).manual_seed(seed)


def block_fixed_parts(wl: Workload, i: int, device="cpu"):
    """(u_j, sigma_j) of block i as fp32 tensors."""
    b = wl.blocks[i]
    g = _gen(device, stream_seed(wl.seed, i, 0))
    u = torch.randn(b.numel, generator=g, device=device, dtype=torch.float32)
    n = torch.randn(b.numel, generator=g, device=device, dtype=torch.float32)
    return u, torch.exp(b.tau * n)


def block_grad(wl: Workload, i: int, t: int, device="cpu", fixed=None, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """bf16 gradient of block i at step t (1-based), flat, ``numel`` elements."""
    b = wl.blocks[i]
    u, sigma = fixed if fixed is not None else block_fixed_parts(wl, i, device)
    g = _gen(device, stream_seed(wl.seed, i, 1, t))
    xi = torch.randn(b.numel, generator=g, device=device, dtype=torch.float32)
    if b.heavy_tail:
        chi = torch.randn((3, b.numel), generator=g, device=device, dtype=torch.float32).square_().sum(0)
        xi = xi / torch.sqrt(chi / 3.0)
    val = (b.scale * sigma) * (math.sqrt(b.stability) * u + math.sqrt(1.0 - b.stability) * xi)
    if out is not None:
        out.copy_(val)
        return out
    return val.to(torch.bfloat16)


def block_param(wl: Workload, i: int, device="cpu") -> torch.Tensor:
    """fp32 initial parameters of block i: normal with standard deviation 0.02."""
    b = wl.blocks[i]
    g = _gen(device, stream_seed(wl.seed, i, 2))
    return 0.02 * torch.randn(b.numel, generator=g, device=device, dtype=torch.float32)


def time_ratio_table(wl: Workload, base_ratios: Sequence[float], jitter: float = 0.1) -> torch.Tensor:
    """Seeded [n_blocks, n_cfg] table of relative update times r_{i,c}.

    ``base_ratios[c]`` is the nominal ratio of configuration c to the plain
    fp32 Adam step; each entry is multiplied by 1 + jitter * U(-1, 1).  It
    stands in for the one-step timing measurement the method takes on the
    target hardware, so that a tight time budget binds in tests.
    """
    g = torch.Generator().manual_seed(stream_seed(wl.seed, 1 << 19, 11))
    u = torch.rand((len(wl.blocks), len(base_ratios)), generator=g, dtype=torch.float64)
    base = torch.tensor(list(base_ratios), dtype=torch.float64)
    return base[None, :] * (1.0 + jitter * (2.0 * u - 1.0))


def sample_subgrids(wl: Workload, s_frac: float):
    """A seeded sub-grid sample of every block's coordinates: about ``s_frac`` of them.  A vector block gets
    ceil(s d) sorted distinct indices; a rows x cols block gets ceil(sqrt(s) rows) rows and ceil(sqrt(s) cols) columns
    (their product is at least ceil(s d)).  Returns one (rows, cols-or-None) pair of int64 / int32 numpy arrays per
    block, drawn once per (seed, block)."""
    out = []
    for i, b in enumerate(wl.blocks):
        g = torch.Generator().manual_seed(stream_seed(wl.seed, i, 3))
        if b.cols <= 1:
            n = max(1, math.ceil(s_frac * b.rows))
            rows = torch.randperm(b.rows, generator=g)[:n].sort().values
            out.append((rows.numpy().astype("int64"), None))
        else:
            nr = max(1, min(b.rows, math.ceil(math.sqrt(s_frac) * b.rows)))
            nc = max(1, min(b.cols, math.ceil(math.sqrt(s_frac) * b.cols)))
            rows = torch.randperm(b.rows, generator=g)[:nr].sort().values
            cols = torch.randperm(b.cols, generator=g)[:nc].sort().values
            out.append((rows.numpy().astype("int64"), cols.numpy().astype("int32")))
    return out


def flat_layout(wl: Workload, align_elems: int = 128):
    """Element offset of every block in one flat buffer, each start aligned to
    ``align_elems`` elements, and the total length."""
    offs, cur = [], 0
    for b in wl.blocks:
        offs.append(cur)
        cur += (b.numel + align_elems - 1) // align_elems * align_elems
    return offs, cur
