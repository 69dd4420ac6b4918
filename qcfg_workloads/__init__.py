"""Seeded synthetic workloads and layer tables for the bit-configuration evaluator.

This module holds NO quantization arithmetic.  It only describes models as lists of
layers (shapes, data dependences, non-linearities) and draws seeded random inputs,
weights, bit vectors and accept/reject streams.  Both the CPU oracle's tests and the
CUDA path's tests/bench take their inputs from here, so the two sides see the same
arrays without sharing any code of the method itself.

The models are stand-ins shaped like the paper's workloads (Section 4: ResNet50 on
ImageNet at batch 128, BERT on SQuAD at 384-token sequences).  The layer tables are
pinned to the paper's Table 1 "Size (MB)" rows: 51.00 MB at 16 bit = 25,502,912
parameters over 54 layers (53 convolutions + fc); 603.98 MB at 16 bit = 301,989,888
parameters = the 144 encoder linears of a 24-block, hidden-1024 transformer.

Draw order from the single numpy Generator of a workload is fixed: input, then weights
layer by layer, then the outlier mask layer by layer, then bit draws, then the
accept/reject stream.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

ACT_NONE = 0
ACT_RELU = 1
ACT_GELU_TANH = 2

POOL_NONE = 0
POOL_MAX3S2 = 1      # 3x3 max-pool, stride 2, pad 1, applied to the source before the layer
POOL_GLOBAL_AVG = 2  # global average pool over H*W, applied to the source before the layer


@dataclass
class Layer:
    """One "tensor" of the bit configuration: a linear or convolution layer.

    The layer's weight (n_out x k_in, row = output channel; for a convolution
    k_in = kh*kw*in_c in (kh, kw, cin) order) and its input activation share one bit
    width (Algorithms 1 and 2 index the working configuration by layer).
    """
    name: str
    n_out: int
    k_in: int
    src: int = -1            # -1: external input, else index of the producing layer
    src_col0: int = 0        # first column of the producer's output that is read
    act: int = ACT_NONE      # applied to this layer's output (after the residual add)
    # convolution geometry; all zero for a linear layer
    kh: int = 0
    kw: int = 0
    stride: int = 0
    pad: int = 0
    in_h: int = 0            # spatial size of the layer's input (after pool_before)
    in_w: int = 0
    in_c: int = 0
    pool_before: int = POOL_NONE
    src_h: int = 0           # spatial size of the source output (before pool_before)
    src_w: int = 0
    residual_from: int = -1  # layer whose output is added in fp32 before `act`

    @property
    def is_conv(self) -> bool:
        return self.kh > 0

    @property
    def out_h(self) -> int:
        return (self.in_h + 2 * self.pad - self.kh) // self.stride + 1 if self.is_conv else 0

    @property
    def out_w(self) -> int:
        return (self.in_w + 2 * self.pad - self.kw) // self.stride + 1 if self.is_conv else 0

    @property
    def params(self) -> int:
        return self.n_out * self.k_in


def param_count(layers: Sequence[Layer]) -> int:
    return sum(l.params for l in layers)


def size_mb(layers: Sequence[Layer], bits: Sequence[int]) -> float:
    """Model size as the paper's Table 1 counts it: weights only, params*b/8 bytes, MB=1e6."""
    return sum(l.params * int(b) for l, b in zip(layers, bits)) / 8.0 / 1e6


# --------------------------------------------------------------------------- model tables

def mlp_layers(dims: Sequence[int]) -> List[Layer]:
    """Chain of linears dims[0] -> dims[1] -> ... with ReLU between layers (not after the last)."""
    out = []
    for i in range(len(dims) - 1):
        out.append(Layer(name=f"fc{i}", n_out=dims[i + 1], k_in=dims[i], src=i - 1,
                         act=ACT_RELU if i < len(dims) - 2 else ACT_NONE))
    return out


def bert_layers(hidden: int, ffn: int, n_blocks: int) -> List[Layer]:
    """Encoder linears of a transformer stack as a stand-in graph.

    Per block: Wq, Wk, Wv read the block input; Wo reads V's output (stand-in for the
    attention context, same shape); W1 reads Wo's output and is followed by tanh-GELU;
    W2 reads that; the next block reads W2's output.  Q and K outputs are consumed by
    nobody (returned as fp32 taps).  No layernorm, softmax or residual.
    """
    out: List[Layer] = []
    for blk in range(n_blocks):
        base = 6 * blk
        h_src = base - 1  # previous block's W2, or -1 (external input) for block 0
        out.append(Layer(f"b{blk}.q", hidden, hidden, src=h_src))
        out.append(Layer(f"b{blk}.k", hidden, hidden, src=h_src))
        out.append(Layer(f"b{blk}.v", hidden, hidden, src=h_src))
        out.append(Layer(f"b{blk}.o", hidden, hidden, src=base + 2))
        out.append(Layer(f"b{blk}.ffn1", ffn, hidden, src=base + 3, act=ACT_GELU_TANH))
        out.append(Layer(f"b{blk}.ffn2", hidden, ffn, src=base + 4))
    return out


def bert_layers_wide_qkv(hidden: int, ffn: int, n_blocks: int) -> List[Layer]:
    """The same stand-in graph with the three projections of a block as ONE layer of
    3*hidden output channels (rows 0..hidden-1 = Wq, then Wk, then Wv).  Wo reads the
    V columns of that layer's output through src_col0 = 2*hidden; two tap layers read
    the Q and K column slices, so every third of the wide output has a reader."""
    out: List[Layer] = []
    for blk in range(n_blocks):
        base = 6 * blk
        h_src = base - 1
        out.append(Layer(f"b{blk}.qkv", 3 * hidden, hidden, src=h_src))
        out.append(Layer(f"b{blk}.qtap", hidden, hidden, src=base, src_col0=0))
        out.append(Layer(f"b{blk}.ktap", hidden, hidden, src=base, src_col0=hidden))
        out.append(Layer(f"b{blk}.o", hidden, hidden, src=base, src_col0=2 * hidden))
        out.append(Layer(f"b{blk}.ffn1", ffn, hidden, src=base + 3, act=ACT_GELU_TANH))
        out.append(Layer(f"b{blk}.ffn2", hidden, ffn, src=base + 4))
    return out


def resnet50_layers(in_hw: int = 224, width: int = 64, n_classes: int = 1000,
                    blocks: Sequence[int] = (3, 4, 6, 3)) -> List[Layer]:
    """ResNet-50 v1.5 as NHWC im2col GEMMs (stride 2 sits in the 3x3 convolution).

    Folded batch-norm is the identity; ReLU after every convolution except a block's
    last one, whose output gets the shortcut added in fp32 and then ReLU; 3x3/2 max-pool
    after conv1; global average pool before fc.
    """
    L: List[Layer] = []

    def conv(name, cout, cin, k, stride, pad, h, w, src, act, pool=POOL_NONE, sh=0, sw=0, res=-1):
        L.append(Layer(name, cout, k * k * cin, src=src, act=act, kh=k, kw=k, stride=stride,
                       pad=pad, in_h=h, in_w=w, in_c=cin, pool_before=pool,
                       src_h=sh or h, src_w=sw or w, residual_from=res))
        return len(L) - 1

    h = in_hw
    c1 = conv("conv1", width, 3, 7, 2, 3, h, h, -1, ACT_RELU)
    h1 = (h + 6 - 7) // 2 + 1            # conv1 output size (112 for 224)
    hp = (h1 + 2 - 3) // 2 + 1           # after 3x3/2 max-pool (56)
    cur, cur_c, cur_h = c1, width, hp
    cur_pool, cur_sh = POOL_MAX3S2, h1   # the first block reads max-pool(conv1)
    for s, nb in enumerate(blocks):
        mid = width * (2 ** s)
        outc = mid * 4
        for b in range(nb):
            stride = 2 if (b == 0 and s > 0) else 1
            name = f"s{s + 1}b{b}"
            a = conv(name + ".a", mid, cur_c, 1, 1, 0, cur_h, cur_h, cur, ACT_RELU,
                     pool=cur_pool, sh=cur_sh, sw=cur_sh)
            bb = conv(name + ".b", mid, mid, 3, stride, 1, cur_h, cur_h, a, ACT_RELU)
            oh = (cur_h + 2 - 3) // stride + 1
            if b == 0:
                d = conv(name + ".down", outc, cur_c, 1, stride, 0, cur_h, cur_h, cur, ACT_NONE,
                         pool=cur_pool, sh=cur_sh, sw=cur_sh)
                short = d
            else:
                short = cur
            c = conv(name + ".c", outc, mid, 1, 1, 0, oh, oh, bb, ACT_RELU, res=short)
            cur, cur_c, cur_h = c, outc, oh
            cur_pool, cur_sh = POOL_NONE, oh
    L.append(Layer("fc", n_classes, cur_c, src=cur, act=ACT_NONE, pool_before=POOL_GLOBAL_AVG,
                   src_h=cur_h, src_w=cur_h))
    return L


def layer_rows(layers: Sequence[Layer], l: int, m_ext: int) -> int:
    """Number of GEMM rows (tokens or output pixels) of layer l for m_ext external rows.

    For the convolutional table the external input is an image batch and m_ext is the
    batch size; for linear stacks m_ext is the token count.
    """
    lay = layers[l]
    if lay.is_conv:
        return m_ext * lay.out_h * lay.out_w
    if lay.pool_before == POOL_GLOBAL_AVG:
        return m_ext
    return m_ext if lay.src < 0 else layer_rows(layers, lay.src, m_ext)


# --------------------------------------------------------------------------- generators

@dataclass
class Workload:
    name: str
    seed: int
    layers: List[Layer]
    m: int                          # external rows (tokens) or batch size (conv table)
    x: np.ndarray                   # fp32 external input, [m, k] or [m, H, W, C]
    weights: List[np.ndarray]       # fp32 [n_out, k_in] per layer
    bits: Optional[np.ndarray] = None          # one configuration (uint8 per layer)
    accept: Optional[np.ndarray] = None        # scripted accept/reject stream (bool)
    meta: dict = field(default_factory=dict)


def _normal_weights(rng, layers, sigma_fn):
    return [(rng.standard_normal((l.n_out, l.k_in), dtype=np.float32) * np.float32(sigma_fn(l)))
            for l in layers]


def _apply_outliers(rng, weights, prob=1e-3, factor=20.0):
    for w in weights:
        mask = rng.random(w.shape, dtype=np.float32) < np.float32(prob)
        w[mask] *= np.float32(factor)


def tiny_mlp(seed: int = 0, m: int = 64, dims: Sequence[int] = (256, 256, 256, 10),
             bits: Sequence[int] = (8, 4, 8)) -> Workload:
    """Three fp32 linears with N(0, 1/fan_in) weights, N(0,1) input, ReLU between layers."""
    rng = np.random.default_rng(seed)
    layers = mlp_layers(dims)
    x = rng.standard_normal((m, dims[0]), dtype=np.float32)
    weights = _normal_weights(rng, layers, lambda l: 1.0 / np.sqrt(l.k_in))
    return Workload("tiny_mlp", seed, layers, m, x, weights, bits=np.asarray(bits, dtype=np.uint8))


def bert_stack(seed: int, m: int, hidden: int, ffn: int, n_blocks: int,
               bit_choices: Optional[Sequence[int]] = (4, 8, 16), n_accept: int = 0,
               name: str = "bert") -> Workload:
    """Transformer-encoder linears: N(0,1) input, N(0,0.02) weights with 0.1% entries x20."""
    rng = np.random.default_rng(seed)
    layers = bert_layers(hidden, ffn, n_blocks)
    x = rng.standard_normal((m, hidden), dtype=np.float32)
    weights = _normal_weights(rng, layers, lambda l: 0.02)
    _apply_outliers(rng, weights)
    bits = None
    if bit_choices is not None:
        bits = rng.choice(np.asarray(bit_choices, dtype=np.uint8), size=len(layers))
    accept = rng.random(n_accept) < 0.5 if n_accept else None
    return Workload(name, seed, layers, m, x, weights, bits=bits, accept=accept,
                    meta={"hidden": hidden, "ffn": ffn, "n_blocks": n_blocks})


def bert_stack_wide_qkv(seed: int, m: int, hidden: int, ffn: int, n_blocks: int,
                        bit_choices: Sequence[int] = (4, 8, 16)) -> Workload:
    """bert_stack's draws for the wide-projection graph (column-slice consumers)."""
    rng = np.random.default_rng(seed)
    layers = bert_layers_wide_qkv(hidden, ffn, n_blocks)
    x = rng.standard_normal((m, hidden), dtype=np.float32)
    weights = _normal_weights(rng, layers, lambda l: 0.02)
    _apply_outliers(rng, weights)
    bits = rng.choice(np.asarray(bit_choices, dtype=np.uint8), size=len(layers))
    return Workload("bert_wide_qkv", seed, layers, m, x, weights, bits=bits,
                    meta={"hidden": hidden, "ffn": ffn, "n_blocks": n_blocks})


def bert_base_block(seed: int = 1, m: int = 8 * 384) -> Workload:
    return bert_stack(seed, m, 768, 3072, 1, name="bert_base_block")


def bert_base_x12(seed: int = 2, m: int = 32 * 384) -> Workload:
    return bert_stack(seed, m, 768, 3072, 12, bit_choices=None, n_accept=72, name="bert_base_x12")


def bert_large_x24(seed: int = 4, m: int = 16 * 384) -> Workload:
    return bert_stack(seed, m, 1024, 4096, 24, bit_choices=None, n_accept=8, name="bert_large_x24")


def resnet50(seed: int = 3, batch: int = 128, in_hw: int = 224, width: int = 64,
             n_classes: int = 1000, blocks: Sequence[int] = (3, 4, 6, 3)) -> Workload:
    """Convolutional table: N(0,1) NHWC input, Laplace(0, 0.02) weights, bits from {4,6,8},
    first convolution and fc forced to 16."""
    rng = np.random.default_rng(seed)
    layers = resnet50_layers(in_hw, width, n_classes, blocks)
    x = rng.standard_normal((batch, in_hw, in_hw, 3), dtype=np.float32)
    weights = [rng.laplace(0.0, 0.02, size=(l.n_out, l.k_in)).astype(np.float32) for l in layers]
    bits = rng.choice(np.asarray((4, 6, 8), dtype=np.uint8), size=len(layers))
    bits[0] = 16
    bits[-1] = 16
    return Workload("resnet50", seed, layers, batch, x, weights, bits=bits,
                    meta={"in_hw": in_hw, "width": width})


# ------------------------------------------------------------- scripted search sequences

def standard_normal_like(weights, seed: int):
    """One array of standard-normal draws per weight tensor (the random numbers E_N's noise is built from)."""
    rng = np.random.default_rng(seed)
    return [rng.standard_normal(w.shape).astype(np.float32) for w in weights]


def greedy_sequence(ranking: Sequence[int], accept: Sequence[bool], start_bits: int = 8,
                    low_bits: int = 4) -> List[np.ndarray]:
    """Configurations visited by one pass of the greedy loop (Algorithm 2, inner loop).

    Starts with every layer at start_bits; evaluation i lowers layer ranking[i] to
    low_bits; an accepted change persists, a rejected one is reverted.  The accept
    decisions come from a scripted stream instead of an accuracy measurement, so that
    two implementations evaluate identical configurations.
    """
    n = len(ranking)
    w = np.full(n, start_bits, dtype=np.uint8)
    configs = []
    for i, l in enumerate(ranking):
        w[l] = low_bits
        configs.append(w.copy())
        if not bool(accept[i]):
            w[l] = start_bits
    return configs


def bisection_sequence(ranking: Sequence[int], accept: Sequence[bool], n_quantized: int,
                       n_evals: int, hi_bits: int = 16, mid_bits: int = 8,
                       low_bits: int = 4) -> List[np.ndarray]:
    """Configurations visited by one bisection pass (Algorithm 1, inner repeat loop).

    State: the n_quantized least-sensitive layers sit at mid_bits, the rest at hi_bits.
    The pass bisects low_bits over those n_quantized layers (threshold starts at half
    the list, integer floor division) for n_evals evaluations driven by the scripted
    accept stream.
    """
    n = len(ranking)
    w = np.full(n, hi_bits, dtype=np.uint8)
    ll = list(ranking[:n_quantized])
    w[ll] = mid_bits
    thr, upl, lowl = len(ll) // 2, len(ll), 0
    configs = []
    for i in range(n_evals):
        lw = w.copy()
        lw[ll[:thr]] = low_bits
        configs.append(lw)
        if bool(accept[i]):
            lowl = thr
            thr = thr + (upl - thr) // 2
        else:
            upl = thr
            thr = thr - (thr - lowl) // 2
    return configs
