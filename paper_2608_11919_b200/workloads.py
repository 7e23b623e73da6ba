"""Seeded synthetic workloads: tensor shapes and value generators for the five configurations.

This module holds NO arithmetic of the optimizer step. It only decides shapes, lays tensors out in
flat buffers and fills parameters and gradients with seeded random values, so it can serve both the
CUDA path and the CPU checker without making them share code of the method.

The workloads stand in for the paper's Qwen-family fine-tuning runs (Sec. 4 setup and the training
configuration table): only parameter shapes and value distributions are used, no dataset or weights.

Recipes
  tiny    8 fp32 tensors [512,512]x4, [512,2048]x2, [2048,512], [512]; p ~ N(0, 0.02^2);
          g ~ N(0, (1e-3)^2) rounded to bf16, step-2 gradients scaled by 1e3; seed 0.
  ragged  1000 fp32 tensors packed back to back (bases are element-aligned only);
          size = floor(exp(U(0, ln max_numel))), with probability 0.70 rounded to the nearest positive
          multiple of 2048, else forced off a multiple of 2048; 5 % of tensors have all-zero
          gradients every step; g ~ 1e-3 * Student-t(3) rounded to bf16; seed 1.
  3b      Qwen2.5-3B-shaped list (hidden 2048, 36 layers, 16 q / 2 kv heads of 128, intermediate
          11008, vocab 151936 tied): fp32 params, bf16 grads ~ N(0, s_l^2) with
          s_l = 1e-4 * 10^(u_l - 0.5), u_l ~ U(0,1) per layer; seed 2.
  7b      Qwen2.5-7B-shaped list (hidden 3584, 28 layers, 28 / 4 heads, intermediate 18944, vocab
          152064 untied): fp32 params, bf16 grads ~ N(0, (1e-4)^2); seed 3.
  27b     dense decoder (hidden 5120, 56 layers, 40 / 8 heads, intermediate 25600, vocab 151936
          untied): bf16 params, bf16 grads ~ N(0, (5e-5)^2); seed 4.
Norm weights are initialised to 1, every other parameter ~ N(0, 0.02^2).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np
import torch

HEAD_DIM = 128


@dataclass
class Spec:
    name: str
    names: List[str]
    sizes: List[int]
    layer_of: List[int]              # layer index per tensor (-1: not in a decoder layer)
    param_dtype: torch.dtype
    grad_dtype: torch.dtype = torch.bfloat16
    seed: int = 0
    grad_std: float = 1e-3
    grad_kind: str = "normal"        # "normal" | "student3" | "layer_normal"
    zero_grad_frac: float = 0.0
    max_norm: float = 1.0
    steps: int = 3
    step_scale: dict = field(default_factory=dict)   # {step: factor} applied to that step's grads
    align_elems: int = 1             # each tensor's offset in the flat buffers is a multiple of this
    state_f32: Optional[List[bool]] = None   # per tensor: plain fp32 moments instead of 8-bit codes (hybrid split)

    @property
    def numel(self) -> int:
        return int(sum(self.sizes))

    def n_blocks(self, block: int) -> int:
        return int(sum((s + block - 1) // block for s in self.sizes))


def _decoder(name, hidden, layers, q_heads, kv_heads, inter, vocab, tied, **kw) -> Spec:
    names, sizes, layer_of = [], [], []

    def add(n, s, l):
        names.append(n); sizes.append(int(s)); layer_of.append(l)

    add("embed", vocab * hidden, -1)
    for l in range(layers):
        add(f"l{l}.q_proj", q_heads * HEAD_DIM * hidden, l)
        add(f"l{l}.k_proj", kv_heads * HEAD_DIM * hidden, l)
        add(f"l{l}.v_proj", kv_heads * HEAD_DIM * hidden, l)
        add(f"l{l}.o_proj", hidden * q_heads * HEAD_DIM, l)
        add(f"l{l}.gate_proj", inter * hidden, l)
        add(f"l{l}.up_proj", inter * hidden, l)
        add(f"l{l}.down_proj", hidden * inter, l)
        add(f"l{l}.input_norm", hidden, l)
        add(f"l{l}.post_attn_norm", hidden, l)
    add("final_norm", hidden, -1)
    if not tied:
        add("lm_head", vocab * hidden, -1)
    return Spec(name=name, names=names, sizes=sizes, layer_of=layer_of, align_elems=16, **kw)


def tiny_spec() -> Spec:
    shapes = [(512, 512)] * 4 + [(512, 2048)] * 2 + [(2048, 512), (512,)]
    sizes = [int(np.prod(s)) for s in shapes]
    return Spec("tiny", [f"t{i}" for i in range(len(sizes))], sizes, [-1] * len(sizes), torch.float32,
                seed=0, grad_std=1e-3, grad_kind="normal", max_norm=1.0, steps=3, step_scale={2: 1e3},
                align_elems=16)


def ragged_spec(n_tensors: int = 1000, max_numel: int = 4 << 20, seed: int = 1, multiple: int = 2048) -> Spec:
    rng = np.random.default_rng(seed)
    sizes = []
    for _ in range(n_tensors):
        s = int(math.floor(math.exp(rng.uniform(0.0, math.log(max_numel)))))
        s = max(1, min(s, max_numel))
        if rng.uniform() < 0.70:
            s = max(multiple, int(round(s / multiple)) * multiple)
        elif s % multiple == 0:
            s += 1 + int(rng.integers(0, multiple - 1))
        sizes.append(s)
    return Spec("ragged", [f"r{i}" for i in range(n_tensors)], sizes, [-1] * n_tensors, torch.float32,
                seed=seed, grad_std=1e-3, grad_kind="student3", zero_grad_frac=0.05, max_norm=0.5,
                steps=10, align_elems=1)


def qwen3b_spec() -> Spec:
    return _decoder("3b", 2048, 36, 16, 2, 11008, 151936, True, param_dtype=torch.float32, seed=2,
                    grad_std=1e-4, grad_kind="layer_normal", max_norm=1.0, steps=1)


def qwen7b_spec() -> Spec:
    return _decoder("7b", 3584, 28, 28, 4, 18944, 152064, False, param_dtype=torch.float32, seed=3,
                    grad_std=1e-4, grad_kind="normal", max_norm=1.0, steps=5)


def dense27b_spec() -> Spec:
    return _decoder("27b", 5120, 56, 40, 8, 25600, 151936, False, param_dtype=torch.bfloat16, seed=4,
                    grad_std=5e-5, grad_kind="normal", max_norm=1.0, steps=3)


def scaled_decoder_spec(name: str, hidden: int, layers: int, q_heads: int, kv_heads: int, inter: int,
                        vocab: int, tied: bool, param_dtype=torch.float32, seed: int = 7,
                        grad_std: float = 1e-4, grad_kind: str = "layer_normal") -> Spec:
    """A decoder-shaped list with caller-chosen dimensions (small cases for tests and profiling)."""
    return _decoder(name, hidden, layers, q_heads, kv_heads, inter, vocab, tied, param_dtype=param_dtype,
                    seed=seed, grad_std=grad_std, grad_kind=grad_kind, max_norm=1.0, steps=1)


def small_spec() -> Spec:
    """About 0.5 B parameters (4 GB resident, well above L2): a 3B-like list with 6 layers and a
    32768-row embedding; the case profiler captures run on."""
    return _decoder("small", 2048, 6, 16, 2, 11008, 32768, True, param_dtype=torch.float32, seed=5,
                    grad_std=1e-4, grad_kind="layer_normal", max_norm=1.0, steps=1)


def small_bf16_spec() -> Spec:
    s = small_spec()
    s.name, s.param_dtype, s.seed = "small_bf16", torch.bfloat16, 6
    return s


SPECS = {"7b_hybrid": lambda: hybrid_split(qwen7b_spec()), "small_hybrid": lambda: hybrid_split(small_spec()),
         "small": small_spec, "small_bf16": small_bf16_spec, "tiny": tiny_spec, "ragged": ragged_spec, "3b": qwen3b_spec, "7b": qwen7b_spec, "27b": dense27b_spec}


def subset_spec(spec: Spec, indices: Sequence[int], suffix: str = "") -> Spec:
    """The same workload restricted to the tensors `indices` (one rank's shard of the list). Layer indices
    are kept, so layer grouping and per-layer gradient scales stay those of the full list."""
    import dataclasses
    idx = list(indices)
    return dataclasses.replace(
        spec, name=spec.name + suffix, names=[spec.names[i] for i in idx], sizes=[spec.sizes[i] for i in idx],
        layer_of=[spec.layer_of[i] for i in idx], step_scale=dict(spec.step_scale),
        state_f32=None if spec.state_f32 is None else [spec.state_f32[i] for i in idx])


def shard_spec(spec: Spec, block: int, rank: int, world: int) -> Spec:
    """Rank `rank`'s share of ONE list cut into `world` block-balanced shards (sharding.partition_blocks): the
    tensors the rank touches, each with the size of the block run the rank owns of it (a rank allocates only
    what it owns; a tensor cut by the partition appears on both neighbours with its part)."""
    from .sharding import partition_blocks
    mine = partition_blocks(spec.sizes, block, world)[rank]
    idx = sorted({t for t, _, _ in mine})
    pos = {t: i for i, t in enumerate(idx)}
    out = subset_spec(spec, idx, suffix=f"[rank {rank}/{world}]")
    out.sizes = [0] * len(idx)
    for t, b0, nb in mine:      # the pieces of one tensor are consecutive: the owned part is one run
        out.sizes[pos[t]] += min(spec.sizes[t], (b0 + nb) * block) - b0 * block
    return out


def layer_groups(spec: Spec, layers_per_group: int = 8) -> List[List[int]]:
    """Tensor indices grouped for chunked update: non-layer tensors first, then runs of layers."""
    groups = [[i for i, l in enumerate(spec.layer_of) if l < 0]]
    n_layers = max(spec.layer_of) + 1 if spec.layer_of else 0
    for l0 in range(0, n_layers, layers_per_group):
        groups.append([i for i, l in enumerate(spec.layer_of) if l0 <= l < l0 + layers_per_group])
    return [g for g in groups if g]


class Buffers:
    """Flat device (or host) buffers for one workload; tensor t occupies [off[t], off[t]+size[t]) of
    param / grad. Tensors with 8-bit state own [off8[t], ...) of m_code / v_code and [boff[t], boff[t]+nb[t])
    of the two scale arrays; tensors with fp32 state own [off32[t], ...) of m_f32 / v_f32."""

    def __init__(self, spec: Spec, block: int, device, pin: bool = False, guard_bytes: int = 0):
        """guard_bytes > 0: every flat buffer is followed by that many bytes of a fixed pattern which
        check_guards() verifies (a write past the end of the last tensor shows up there)."""
        self.spec, self.block, self.device = spec, int(block), torch.device(device)
        self._guards = []
        a = spec.align_elems
        self.f32 = list(spec.state_f32) if spec.state_f32 is not None else [False] * len(spec.sizes)
        self.off, self.boff, self.off8, self.off32 = [], [], [], []
        o = b = o8 = o32 = 0
        for s, f in zip(spec.sizes, self.f32):
            o = (o + a - 1) // a * a
            o8 = (o8 + a - 1) // a * a
            o32 = (o32 + a - 1) // a * a
            self.off.append(o); self.boff.append(b); self.off8.append(o8); self.off32.append(o32)
            o += s
            if f:
                o32 += s
            else:
                o8 += s; b += (s + block - 1) // block
        self.total, self.total_blocks = o, b
        kw = dict(device=self.device)
        if pin and self.device.type == "cpu":
            kw["pin_memory"] = True
        def flat(n, dtype):
            n = max(n, 1)
            if guard_bytes <= 0:
                return torch.empty(n, dtype=dtype, **kw)
            es = torch.empty(0, dtype=dtype).element_size()
            raw = torch.empty(n * es + guard_bytes, dtype=torch.uint8, **kw)
            raw[n * es:] = 0xA5
            self._guards.append(raw[n * es:])
            return raw[:n * es].view(dtype)

        self.param = flat(o, spec.param_dtype)
        self.grad = flat(o, spec.grad_dtype)
        self.m_code = flat(o8, torch.uint8)
        self.v_code = flat(o8, torch.uint8)
        self.m_absmax = flat(b, torch.float32)
        self.v_absmax = flat(b, torch.float32)
        self.m_f32 = flat(o32, torch.float32)
        self.v_f32 = flat(o32, torch.float32)

    def check_guards(self) -> None:
        for i, g in enumerate(self._guards):
            assert bool((g == 0xA5).all()), f"guard bytes after flat buffer {i} were overwritten"

    def view(self, which: str, t: int) -> torch.Tensor:
        size = self.spec.sizes[t]
        if which in ("m_absmax", "v_absmax"):
            nb = 0 if self.f32[t] else (size + self.block - 1) // self.block
            return getattr(self, which)[self.boff[t]: self.boff[t] + nb]
        if which in ("m_code", "v_code"):          # the moment storage, whichever kind this tensor has
            if self.f32[t]:
                return (self.m_f32 if which == "m_code" else self.v_f32)[self.off32[t]: self.off32[t] + size]
            return getattr(self, which)[self.off8[t]: self.off8[t] + size]
        return getattr(self, which)[self.off[t]: self.off[t] + size]

    def resident_bytes(self) -> int:
        return sum(getattr(self, k).numel() * getattr(self, k).element_size()
                   for k in ("param", "grad", "m_code", "v_code", "m_absmax", "v_absmax", "m_f32", "v_f32"))


def hybrid_split(spec: Spec, eight_bit_fraction: float = 0.02) -> Spec:
    """Marks tensors as fp32-state so that about `eight_bit_fraction` of the parameters keep 8-bit state
    (the paper's hybrid configuration: a 2 % 8-bit slice, ordinary Adam states elsewhere). The 8-bit slice
    is taken from the smaller matrices of the last layers until the fraction is reached."""
    target = eight_bit_fraction * spec.numel
    order = sorted(range(len(spec.sizes)), key=lambda i: (-spec.layer_of[i], spec.sizes[i]))
    f32 = [True] * len(spec.sizes)
    got = 0
    for i in order:
        if spec.layer_of[i] < 0 or spec.sizes[i] < 4096:
            continue
        if got + spec.sizes[i] > 1.25 * target:
            continue
        f32[i] = False
        got += spec.sizes[i]
        if got >= target:
            break
    spec.state_f32 = f32
    spec.name = spec.name + "_hybrid"
    return spec


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def fill_params(buf: Buffers) -> None:
    """p ~ N(0, 0.02^2); tensors whose name ends in 'norm' are set to 1."""
    spec = buf.spec
    gen = _gen(buf.device, spec.seed * 1000 + 1)
    if buf.total > sum(spec.sizes):
        buf.param.zero_()
    for t, name in enumerate(spec.names):
        v = buf.view("param", t)
        if name.endswith("norm"):
            v.fill_(1.0)
        else:
            v.normal_(0.0, 0.02, generator=gen)


def layer_stds(spec: Spec) -> List[float]:
    """Per-tensor gradient standard deviation (layer_normal: one draw per layer, 10x spread)."""
    if spec.grad_kind != "layer_normal":
        return [spec.grad_std] * len(spec.sizes)
    rng = np.random.default_rng(spec.seed * 1000 + 7)
    n_layers = max(spec.layer_of) + 1
    u = rng.uniform(0.0, 1.0, n_layers + 1)
    return [spec.grad_std * 10.0 ** (u[l if l >= 0 else n_layers] - 0.5) for l in spec.layer_of]


def zero_grad_mask(spec: Spec) -> List[bool]:
    rng = np.random.default_rng(spec.seed * 1000 + 3)
    return [bool(rng.uniform() < spec.zero_grad_frac) for _ in spec.sizes]


def fill_grads(buf: Buffers, step: int, max_chunk: int = 1 << 26) -> None:
    """Fresh gradients for optimizer step `step` (1-based), reproducible per (seed, step)."""
    spec = buf.spec
    gen = _gen(buf.device, spec.seed * 1000 + 100 + step)
    stds = layer_stds(spec)
    zeros = zero_grad_mask(spec)
    scale = float(spec.step_scale.get(step, 1.0))
    if buf.total > sum(spec.sizes):
        buf.grad.zero_()
    for t in range(len(spec.sizes)):
        v = buf.view("grad", t)
        if zeros[t]:
            v.zero_()
            continue
        if spec.grad_kind == "student3":
            for a in range(0, v.numel(), max_chunk):
                w = v[a: a + max_chunk]
                z = torch.empty(4, w.numel(), dtype=torch.float32, device=buf.device)
                z.normal_(0.0, 1.0, generator=gen)
                tval = z[0] / torch.sqrt((z[1] * z[1] + z[2] * z[2] + z[3] * z[3]) / 3.0)
                w.copy_((tval * (stds[t] * scale)).to(spec.grad_dtype))
        else:
            v.normal_(0.0, stds[t] * scale, generator=gen)


def numpy_view(t: torch.Tensor) -> np.ndarray:
    """Host numpy array sharing memory with a CPU tensor (bf16 as its uint16 bit pattern)."""
    t = t.detach()
    assert t.device.type == "cpu"
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()
