"""Seeded synthetic workloads shared by the CUDA path's tests/bench and by the CPU oracle.

This module holds shapes, wiring and random draws only. It contains none of the
method's arithmetic (no GEMM, no activation, no gradient, no importance, no
selection): both sides receive the same arrays from here and compute on their own.

Layer / tensor indexing is forward execution order, 0 = nearest the input
(the paper lists trainable tensors in execution order, Section 5).  Tensor
``2*l`` is the kernel of layer ``l`` and tensor ``2*l + 1`` its bias
(Section 5.1: a dense layer carries a Kernel and a Bias tensor); for a
normalisation layer they are its Gamma and Beta (Section 5.2).

The stacks stand in for the models the paper trains (ViT, ResNet50; Section 8)
with every non-dense operator replaced by the identity, so that the whole
backward pass is dense-layer work.  No dataset item is reproduced: inputs and
targets are N(0,1) draws.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

# activation / post-op codes (mirrored by include/et.h)
ACT_NONE, ACT_GELU_TANH, ACT_RELU = 0, 1, 2
DT_F32, DT_BF16 = 0, 1
# layer kinds: a dense layer (kernel, bias) or a layer normalisation over the feature axis, whose two
# trainable tensors gamma and beta take the kernel and bias slots (Section 5.2: Gamma and Beta)
KIND_DENSE, KIND_NORM, KIND_ATTENTION, KIND_IM2COL, KIND_BATCHNORM = 0, 1, 2, 3, 4
# KIND_BATCHNORM: batch normalisation in training mode (statistics of each feature over all rows), optional
# activation after it; Gamma and Beta in the kernel and bias slots like KIND_NORM (Section 5.2)
# KIND_IM2COL: the patch-gathering half of a k x k convolution (stride 1, zero padding k // 2) on NHWC
# rows; followed by a dense layer with in_features = k * k * channels it is that convolution.  No tensors.
# KIND_ATTENTION: the softmax attention core, a layer without trainable tensors (Section 5.3 / 5.4:
# attention operations are non-trainable layers); its two tensor slots are empty


@dataclass(frozen=True)
class Layer:
    in_features: int
    out_features: int          # width of Z = X W + b
    act: int = ACT_NONE
    fold: int = 1              # output = sum of `fold` equal column slices of act(Z)
    residual_src: int = -1     # -1, or j: add activation a_j (a_0 = stack input,
                               # a_{j+1} = output of layer j) to this layer's output
    kind: int = KIND_DENSE     # KIND_NORM: in_features == out_features, no act / fold / residual
    eps: float = 1e-5          # KIND_NORM: added to the variance
    heads: int = 0             # KIND_ATTENTION: in_features = 3 * out_features = 3 * heads * head_dim,
    seq: int = 0               #   rows come in sequences of `seq` consecutive tokens
    height: int = 0            # KIND_IM2COL: rows are images of height x width pixels (row = (n, h, w)),
    width: int = 0             #   in_features = channels, out_features = ksize * ksize * channels,
    ksize: int = 0             #   column (kh * ksize + kw) * channels + c holds pixel (h + kh - k//2, w + kw - k//2)

    @property
    def out_width(self) -> int:
        return self.out_features // self.fold


@dataclass
class Workload:
    name: str
    layers: List[Layer]
    M: int                     # tokens (rows)
    dtype: int                 # storage type of weights / activations
    lr: float
    mask: np.ndarray           # uint8[2L], tensor order
    W: List[np.ndarray] = field(default_factory=list)   # float64 values, exactly representable in `dtype`
    b: List[np.ndarray] = field(default_factory=list)
    x: Optional[np.ndarray] = None
    target: Optional[np.ndarray] = None

    @property
    def L(self) -> int:
        return len(self.layers)


# --------------------------------------------------------------------------- rounding of inputs
def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float values to the nearest bfloat16 (ties to even); returns float64
    holding exactly those bf16 values.  Used only so that both sides start from
    identical input bits."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    u = (u + 0x7FFF + lsb) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(a.shape)


def round_to_f32(a: np.ndarray) -> np.ndarray:
    return np.asarray(a, dtype=np.float32).astype(np.float64)


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of values that are already exactly bf16-representable."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    return (f.view(np.uint32) >> 16).astype(np.uint16).reshape(a.shape)


def from_bf16_bits(u: np.ndarray) -> np.ndarray:
    return (u.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def _store(a: np.ndarray, dtype: int) -> np.ndarray:
    return round_to_bf16(a) if dtype == DT_BF16 else round_to_f32(a)


# --------------------------------------------------------------------------- stack shapes
def mlp_blocks(n_blocks: int, d: int, hidden: int, act: int) -> List[Layer]:
    """[Linear d->hidden, act, Linear hidden->d, + block input] repeated."""
    layers: List[Layer] = []
    for blk in range(n_blocks):
        base = 2 * blk
        layers.append(Layer(d, hidden, act=act))
        layers.append(Layer(hidden, d, residual_src=base))
    return layers


def vit_blocks(n_blocks: int, d: int, ffn: int) -> List[Layer]:
    """Transformer block with the attention core replaced by identity:
    QKV d->3d whose three slices are summed, out-proj d->d + block input,
    fc1 d->ffn with tanh-GELU, fc2 ffn->d + fc1's input."""
    layers: List[Layer] = []
    for blk in range(n_blocks):
        base = 4 * blk
        layers.append(Layer(d, 3 * d, fold=3))
        layers.append(Layer(d, d, residual_src=base))
        layers.append(Layer(d, ffn, act=ACT_GELU_TANH))
        layers.append(Layer(ffn, d, residual_src=base + 2))
    return layers


def norm_layer(d: int, eps: float = 1e-5) -> Layer:
    return Layer(d, d, kind=KIND_NORM, eps=eps)


def batchnorm_layer(d: int, act: int = ACT_NONE, eps: float = 1e-5) -> Layer:
    return Layer(d, d, act=act, kind=KIND_BATCHNORM, eps=eps)


def attention_layer(d: int, heads: int, seq: int) -> Layer:
    return Layer(3 * d, d, kind=KIND_ATTENTION, heads=heads, seq=seq)


def vit_blocks_full(n_blocks: int, d: int, ffn: int, heads: int, seq: int) -> List[Layer]:
    """The whole pre-norm transformer block: LN, QKV d->3d, softmax attention over sequences of `seq`
    tokens with `heads` heads, out-proj d->d + block input, LN, fc1 with tanh-GELU, fc2 + the second
    LN's input."""
    layers: List[Layer] = []
    for blk in range(n_blocks):
        base = 7 * blk
        layers.append(norm_layer(d))
        layers.append(Layer(d, 3 * d))
        layers.append(attention_layer(d, heads, seq))
        layers.append(Layer(d, d, residual_src=base))
        layers.append(norm_layer(d))
        layers.append(Layer(d, ffn, act=ACT_GELU_TANH))
        layers.append(Layer(ffn, d, residual_src=base + 4))
    return layers


def conv_layers(c_in: int, c_out: int, height: int, width: int, ksize: int = 3, act: int = ACT_NONE,
                residual_src: int = -1) -> List[Layer]:
    """A k x k convolution (stride 1, "same" zero padding) on NHWC rows as two stack layers: the patch
    gather and a dense layer whose kernel is the convolution kernel in (kh, kw, c_in) x c_out layout."""
    return [Layer(c_in, ksize * ksize * c_in, kind=KIND_IM2COL, height=height, width=width, ksize=ksize),
            Layer(ksize * ksize * c_in, c_out, act=act, residual_src=residual_src)]


def resnet_bottleneck_blocks(n_blocks: int, c: int, mid: int, height: int, width: int, bn: bool = False,
                             act: int = ACT_RELU) -> List[Layer]:
    """ResNet bottleneck: 1x1 c->mid ReLU, 3x3 mid->mid ReLU, 1x1 mid->c + block input (4 layers);
    bn=True puts a batch normalisation between each of the first two convolutions and its ReLU (6 layers)."""
    layers: List[Layer] = []
    for blk in range(n_blocks):
        base = (6 if bn else 4) * blk
        if bn:
            layers += [Layer(c, mid), batchnorm_layer(mid, act)]
            layers += conv_layers(mid, mid, height, width, 3) + [batchnorm_layer(mid, act)]
        else:
            layers.append(Layer(c, mid, act=act))
            layers += conv_layers(mid, mid, height, width, 3, act=act)
        layers.append(Layer(mid, c, residual_src=base))
    return layers


def vit_blocks_prenorm(n_blocks: int, d: int, ffn: int) -> List[Layer]:
    """Pre-norm transformer block, attention core still the identity:
    LN, QKV d->3d (three slices summed), out-proj d->d + block input,
    LN, fc1 d->ffn with tanh-GELU, fc2 ffn->d + the second LN's input."""
    layers: List[Layer] = []
    for blk in range(n_blocks):
        base = 6 * blk
        layers.append(norm_layer(d))
        layers.append(Layer(d, 3 * d, fold=3))
        layers.append(Layer(d, d, residual_src=base))
        layers.append(norm_layer(d))
        layers.append(Layer(d, ffn, act=ACT_GELU_TANH))
        layers.append(Layer(ffn, d, residual_src=base + 3))
    return layers


# --------------------------------------------------------------------------- draws
def _draw_params(rng, layers, dtype, w_std=None, he_init=False):
    W, b = [], []
    for ly in layers:
        if ly.kind in (KIND_ATTENTION, KIND_IM2COL):
            W.append(np.zeros(0)); b.append(np.zeros(0))
            continue
        if ly.kind in (KIND_NORM, KIND_BATCHNORM):
            W.append(_store(1.0 + rng.normal(0.0, 0.1, size=ly.out_features), dtype))     # gamma
            b.append(_store(rng.normal(0.0, 0.1, size=ly.out_features), dtype))           # beta
            continue
        std = np.sqrt(2.0 / ly.in_features) if he_init else w_std
        W.append(_store(rng.normal(0.0, std, size=(ly.in_features, ly.out_features)), dtype))
        b.append(np.zeros(ly.out_features, dtype=np.float64))
    return W, b


def bernoulli_weight_mask(rng, L: int, p: float) -> np.ndarray:
    """One Bernoulli(p) draw per kernel tensor; each bias follows its kernel."""
    bits = (rng.random(L) < p).astype(np.uint8)
    return np.repeat(bits, 2)


def _finish(name, layers, M, dtype, lr, mask, rng, w_std=None, he_init=False, params=True):
    wl = Workload(name=name, layers=layers, M=M, dtype=dtype, lr=lr, mask=mask)
    if params:
        wl.W, wl.b = _draw_params(rng, layers, dtype, w_std=w_std, he_init=he_init)
        wl.x = _store(rng.normal(size=(M, layers[0].in_features)), dtype)
        wl.target = _store(rng.normal(size=(M, layers[-1].out_width)), dtype)
    return wl


def tiny_mlp(seed: int = 0, params: bool = True) -> Workload:
    """fp32, 2 blocks of [128->512, tanh-GELU, 512->128, residual], 256 tokens;
    only the first layer of block 2 (kernel + bias) is selected."""
    rng = np.random.default_rng(seed)
    layers = mlp_blocks(2, 128, 512, ACT_GELU_TANH)
    mask = np.zeros(2 * len(layers), dtype=np.uint8)
    mask[4] = mask[5] = 1
    return _finish("tiny_mlp_fp32", layers, 256, DT_F32, 0.01, mask, rng, w_std=0.02, params=params)


def vit_b(seed: int = 1, p_select: float = 0.3, n_blocks: int = 12, tokens: int = 64 * 197,
          d: int = 768, ffn: int = 3072, params: bool = True, name: str = "vit_b_linear_bf16") -> Workload:
    """bf16 ViT-B/16-shaped linear-only stack, Bernoulli(p_select) mask over kernels."""
    rng = np.random.default_rng(seed)
    layers = vit_blocks(n_blocks, d, ffn)
    mask = bernoulli_weight_mask(rng, len(layers), p_select)
    return _finish(name, layers, tokens, DT_BF16, 0.01, mask, rng, w_std=0.02, params=params)


def vit_b_prenorm(seed: int = 4, p_select: float = 0.3, n_blocks: int = 12, tokens: int = 64 * 197,
                  d: int = 768, ffn: int = 3072, params: bool = True) -> Workload:
    """The ViT-B/16-shaped stack with its two layer normalisations per block (gamma and beta are
    selectable tensors); Bernoulli(p_select) over layers, both tensors of a layer follow the draw."""
    rng = np.random.default_rng(seed)
    layers = vit_blocks_prenorm(n_blocks, d, ffn)
    mask = bernoulli_weight_mask(rng, len(layers), p_select)
    return _finish("vit_b_prenorm_bf16", layers, tokens, DT_BF16, 0.01, mask, rng, w_std=0.02, params=params)


def vit_b_full(seed: int = 5, p_select: float = 0.3, n_blocks: int = 12, batch: int = 64, seq: int = 197,
               d: int = 768, ffn: int = 3072, heads: int = 12, params: bool = True) -> Workload:
    """ViT-B/16 with its normalisation layers and attention core: `batch` sequences of `seq` tokens.
    Bernoulli(p_select) over layers; the attention layers own no tensors and are never selected."""
    rng = np.random.default_rng(seed)
    layers = vit_blocks_full(n_blocks, d, ffn, heads, seq)
    mask = bernoulli_weight_mask(rng, len(layers), p_select)
    for l, ly in enumerate(layers):
        if ly.kind == KIND_ATTENTION:
            mask[2 * l] = mask[2 * l + 1] = 0
    return _finish("vit_b_full_bf16", layers, batch * seq, DT_BF16, 0.01, mask, rng, w_std=0.02, params=params)


def vit_l(seed: int = 3, params: bool = True, n_blocks: int = 24, tokens: int = 32 * 197,
          d: int = 1024, ffn: int = 4096) -> Workload:
    """bf16 ViT-L-shaped linear-only stack; the mask starts all-selected and is
    replaced by the selector while training."""
    rng = np.random.default_rng(seed)
    layers = vit_blocks(n_blocks, d, ffn)
    mask = np.ones(2 * len(layers), dtype=np.uint8)
    # std 0.01: without normalisation layers 24 blocks of std-0.02 kernels at d = 1024 multiply the
    # activation variance by about 1.9 per block (5e6 overall); 0.01 keeps it near 3x overall
    return _finish("vit_l_linear_bf16", layers, tokens, DT_BF16, 0.01, mask, rng, w_std=0.01, params=params)


def vit_l_full(seed: int = 9, params: bool = True, n_blocks: int = 24, batch: int = 32, seq: int = 197,
               d: int = 1024, ffn: int = 4096, heads: int = 16) -> Workload:
    """bf16 ViT-L/16 with its normalisation layers and attention core; the mask starts with every
    trainable tensor selected and is replaced by the selector while training."""
    rng = np.random.default_rng(seed)
    layers = vit_blocks_full(n_blocks, d, ffn, heads, seq)
    mask = np.array([0 if ly.kind == KIND_ATTENTION else 1 for ly in layers for _ in (0, 1)], dtype=np.uint8)
    return _finish("vit_l_full_bf16", layers, batch * seq, DT_BF16, 0.01, mask, rng, w_std=0.02, params=params)


def resnet_1x1(seed: int = 2, p_select: float = 0.5, n_blocks: int = 6, tokens: int = 32 * 14 * 14,
               params: bool = True) -> Workload:
    """bf16 ResNet-50 conv4_x 1x1 bottleneck convs as NHWC GEMMs:
    [1024->256, ReLU, 256->1024 (3x3 replaced by identity), + block input]."""
    rng = np.random.default_rng(seed)
    layers = mlp_blocks(n_blocks, 1024, 256, ACT_RELU)
    mask = bernoulli_weight_mask(rng, len(layers), p_select)
    return _finish("resnet50_conv4_1x1_bf16", layers, tokens, DT_BF16, 0.01, mask, rng,
                   he_init=True, params=params)


def resnet_bottleneck(seed: int = 6, p_select: float = 0.5, n_blocks: int = 6, images: int = 32, height: int = 14,
                      width: int = 14, c: int = 1024, mid: int = 256, params: bool = True, bn: bool = False,
                      act: int = ACT_RELU, dtype: int = DT_BF16) -> Workload:
    """bf16 ResNet-50 conv4_x bottlenecks with their 3x3 convolutions (NHWC rows), optionally with their
    batch normalisations."""
    rng = np.random.default_rng(seed)
    layers = resnet_bottleneck_blocks(n_blocks, c, mid, height, width, bn, act)
    mask = bernoulli_weight_mask(rng, len(layers), p_select)
    for l, ly in enumerate(layers):
        if ly.kind == KIND_IM2COL:
            mask[2 * l] = mask[2 * l + 1] = 0
    return _finish("resnet50_conv4_bottleneck" + ("_bn" if bn else ""), layers, images * height * width, dtype, 0.01, mask,
                   rng, he_init=True, params=params)


def small_stack(layers: List[Layer], M: int, dtype: int, seed: int, mask=None, w_std: float = 0.05,
                bias_std: float = 0.0, lr: float = 0.01) -> Workload:
    """Arbitrary small stack for parity and oracle tests (ragged sizes, every act/fold/residual kind)."""
    rng = np.random.default_rng(seed)
    if mask is None:
        mask = (rng.random(2 * len(layers)) < 0.5).astype(np.uint8)
    wl = _finish("small", layers, M, dtype, lr, np.asarray(mask, dtype=np.uint8), rng, w_std=w_std)
    if bias_std > 0:
        wl.b = [np.zeros(0) if ly.kind in (KIND_ATTENTION, KIND_IM2COL)
                else _store(rng.normal(0.0, bias_std, size=ly.out_features), dtype) for ly in layers]
    return wl


def selector_instance(rng, n: int, t_max: int = 20, integer: bool = True):
    """Random importances and per-tensor costs for selector tests (biases get t_dy = 0
    on odd indices, Section 5.1)."""
    I = rng.random(n)
    if integer:
        t_dw = rng.integers(0, t_max, size=n).astype(np.float64)
        t_dy = rng.integers(0, t_max, size=n).astype(np.float64)
    else:
        t_dw = rng.random(n) * t_max
        t_dy = rng.random(n) * t_max
    t_dy[1::2] = 0.0
    return I, t_dw, t_dy


def draw_delta(w: Workload, seed: int, std: float = 1e-3):
    """A recent weight update dw for every tensor (the second factor of the importance
    sum), in tensor order [dW_0, db_0, ...], representable in the workload's dtype."""
    rng = np.random.default_rng(seed)
    out = []
    for ly in w.layers:
        if ly.kind in (KIND_ATTENTION, KIND_IM2COL):
            out += [np.zeros(0), np.zeros(0)]
            continue
        shape = (ly.out_features,) if ly.kind in (KIND_NORM, KIND_BATCHNORM) else (ly.in_features, ly.out_features)
        out.append(_store(rng.normal(0.0, std, size=shape), w.dtype))
        out.append(_store(rng.normal(0.0, std, size=ly.out_features), w.dtype))
    return out


def flop_costs(layers, M: int):
    """Per-tensor cost vectors (t_dw, t_dy) proportional to the work of each backward operation, for
    selector inputs when measured times are not wanted: a kernel costs 2*M*K*N for its weight gradient
    and as much for passing the error gradient on, a bias M*N and 0 (Section 5.1); a normalisation layer
    is one pass over its rows, all of it charged to beta's error-gradient time (Section 5.2); layers
    without tensors have empty slots that cost nothing."""
    t_dw, t_dy = [], []
    for ly in layers:
        if ly.kind in (KIND_ATTENTION, KIND_IM2COL):
            t_dw += [0.0, 0.0]
            t_dy += [0.0, 0.0]
        elif ly.kind in (KIND_NORM, KIND_BATCHNORM):
            t_dw += [0.0, 0.0]
            t_dy += [0.0, 8.0 * M * ly.out_features]
        else:
            f = 2.0 * M * ly.in_features * ly.out_features
            t_dw += [f, float(M * ly.out_features)]
            t_dy += [f, 0.0]
    return np.array(t_dw), np.array(t_dy)
