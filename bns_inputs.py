"""Seeded synthetic inputs for BN-sampling experiments.

This module only *draws* data: activations, upstream gradients, affine parameters,
sample indices, patch offsets and virtual samples, plus the bf16 <-> fp32 bit
conversion used to hand the same values to every consumer.  It contains none of the
normalisation arithmetic.  All randomness comes from one counter-based generator
(Philox-4x64, numpy's implementation) keyed by ``(seed, stream tag)`` so that every
tensor of a case has its own independent, reproducible stream.

The activation recipes stand in for CNN feature maps of the networks the paper trains
(Table 1: ResNet-20/56 on CIFAR with 128 samples per GPU, ResNet-18/50 on ImageNet);
only the shapes and the statistical structure are copied, no dataset is involved:

* ``tiny_activations``   - per-channel offset U(-1,1) + per-sample offset N(0, std 0.5)
  + iid N(0,1): the offsets make the per-channel mean non-trivial and make different
  sample subsets give visibly different statistics.
* ``correlated_activations`` - per (sample, channel) map a 3x3 box blur (replicated
  border) of N(0,1) noise plus a per-channel offset U(-1,1): neighbouring pixels are
  correlated, as the paper assumes for real feature maps (Sec. 4.1, "Data Randomness and
  Correlation").
"""
from __future__ import annotations

import numpy as np

# stream tags: one independent Philox stream per tensor of a case
TAG_X, TAG_DY, TAG_GAMMA, TAG_BETA, TAG_INDEX, TAG_XV, TAG_DYV, TAG_CHAN, TAG_SAMPLE = range(9)


def stream(seed: int, tag: int) -> np.random.Generator:
    """Independent generator for ``(seed, tag)``: Philox-4x64 keyed by the pair."""
    key = np.array([np.uint64(seed), np.uint64(tag)], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


# ----------------------------------------------------------------------------- dtype plumbing
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even), returned as uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    rounded = u + np.uint32(0x7FFF) + lsb
    out = (rounded >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(a)
    if nan.any():
        out[nan] = np.uint16(0x7FC0)
    return out


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """fp32 array whose every value is exactly representable in bf16."""
    return bf16_bits_to_f32(f32_to_bf16_bits(a))


# ----------------------------------------------------------------------------- tensors
def _normal(rng: np.random.Generator, shape, std: float = 1.0) -> np.ndarray:
    a = rng.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    return a


def tiny_activations(N: int, C: int, H: int, W: int, seed: int) -> np.ndarray:
    """fp32 [N,C,H,W]: channel offset U(-1,1) + sample offset N(0, std 0.5) + iid N(0,1)."""
    x = _normal(stream(seed, TAG_X), (N, C, H, W))
    chan = stream(seed, TAG_CHAN).uniform(-1.0, 1.0, size=C).astype(np.float32)
    samp = _normal(stream(seed, TAG_SAMPLE), (N,), std=0.5)
    x += chan[None, :, None, None]
    x += samp[:, None, None, None]
    return x


def box_blur3(a: np.ndarray) -> np.ndarray:
    """3x3 mean filter over the last two axes with a replicated (clamp-to-edge) border."""
    H, W = a.shape[-2:]
    rows = np.empty_like(a)
    # horizontal pass
    if W > 1:
        rows[..., 1:-1] = a[..., :-2] + a[..., 1:-1] + a[..., 2:]
        rows[..., 0] = 2.0 * a[..., 0] + a[..., 1]
        rows[..., -1] = a[..., -2] + 2.0 * a[..., -1]
    else:
        rows[...] = 3.0 * a
    out = np.empty_like(a)
    # vertical pass
    if H > 1:
        out[..., 1:-1, :] = rows[..., :-2, :] + rows[..., 1:-1, :] + rows[..., 2:, :]
        out[..., 0, :] = 2.0 * rows[..., 0, :] + rows[..., 1, :]
        out[..., -1, :] = rows[..., -2, :] + 2.0 * rows[..., -1, :]
    else:
        out[...] = 3.0 * rows
    out *= np.float32(1.0 / 9.0)
    return out


def correlated_activations(N: int, C: int, H: int, W: int, seed: int) -> np.ndarray:
    """fp32 [N,C,H,W]: 3x3 box-blurred N(0,1) field per map + per-channel offset U(-1,1)."""
    rng = stream(seed, TAG_X)
    chan = stream(seed, TAG_CHAN).uniform(-1.0, 1.0, size=C).astype(np.float32)
    x = np.empty((N, C, H, W), dtype=np.float32)
    # generate in sample blocks so the temporaries stay small for the big layers
    block = max(1, (1 << 24) // max(1, C * H * W))
    for n0 in range(0, N, block):
        n1 = min(N, n0 + block)
        x[n0:n1] = box_blur3(_normal(rng, (n1 - n0, C, H, W)))
    x += chan[None, :, None, None]
    return x


def upstream_gradient(shape, seed: int, tag: int = TAG_DY) -> np.ndarray:
    """dy ~ N(0,1), fp32."""
    return _normal(stream(seed, tag), tuple(shape))


def affine_parameters(C: int, seed: int):
    """gamma ~ U(0.5,1.5), beta ~ N(0, std 0.1), fp32 [C] each."""
    gamma = stream(seed, TAG_GAMMA).uniform(0.5, 1.5, size=C).astype(np.float32)
    beta = _normal(stream(seed, TAG_BETA), (C,), std=0.1)
    return gamma, beta


def virtual_samples(nv: int, C: int, H: int, W: int, seed: int) -> np.ndarray:
    """Virtual samples V ~ N(0,1), fp32 [nv,C,H,W] (Algorithm 3 draws N(mu,sigma) of a dataset;
    with no dataset here the standard normal stands in)."""
    return _normal(stream(seed, TAG_XV), (nv, C, H, W))


# ----------------------------------------------------------------------------- index sets
def batch_sample_indices(N: int, k: int, seed: int, contiguous: bool) -> np.ndarray:
    """int32 [k] sample indices for Batch Sampling.

    ``contiguous=True`` is the paper's rule (Algorithm 1): ``begin = randint(0, N-k)`` with both
    ends included, samples ``begin .. begin+k-1``.  ``contiguous=False`` draws k distinct samples
    without replacement and returns them sorted.
    """
    rng = stream(seed, TAG_INDEX)
    if contiguous:
        begin = int(rng.integers(0, N - k, endpoint=True))
        return np.arange(begin, begin + k, dtype=np.int32)
    return np.sort(rng.choice(N, size=k, replace=False)).astype(np.int32)


OFFSETS_SHARED, OFFSETS_PER_SAMPLE, OFFSETS_PER_MAP = 0, 1, 2


def patch_offsets(N: int, C: int, H: int, W: int, ph: int, pw: int, mode: int, seed: int) -> np.ndarray:
    """int32 (oh, ow) pairs for Feature Sampling: shape [1,2] (one location for the whole layer,
    Algorithm 2), [N,2] (one per sample) or [N*C,2] (one per feature map).  Each coordinate is
    uniform on [0, H-ph] x [0, W-pw], both ends included, so the patch always fits."""
    rng = stream(seed, TAG_INDEX)
    count = {OFFSETS_SHARED: 1, OFFSETS_PER_SAMPLE: N, OFFSETS_PER_MAP: N * C}[mode]
    oh = rng.integers(0, H - ph, size=count, endpoint=True)
    ow = rng.integers(0, W - pw, size=count, endpoint=True)
    return np.stack([oh, ow], axis=1).astype(np.int32)


# ----------------------------------------------------------------------------- workload shapes
def resnet50_bn_layers():
    """The 53 BN layers of ResNet-50 as (C, H) with H = W, for a 224x224 input.

    Bottleneck blocks [3,4,6,3] with widths 64/128/256/512 and x4 expansion; a stem BN at
    112x112; a projection BN in the first block of every stage; the stride of a down-sampling
    block sits on its 3x3 convolution, so the first BN of such a block still sees the larger map.
    """
    layers = [(64, 112)]
    size = 56
    for stage, (width, blocks) in enumerate(zip((64, 128, 256, 512), (3, 4, 6, 3))):
        for b in range(blocks):
            strided = stage > 0 and b == 0
            in_size = size
            if strided:
                size //= 2
            layers.append((width, in_size))       # after the 1x1 reduce
            layers.append((width, size))          # after the 3x3 (carries the stride)
            layers.append((4 * width, size))      # after the 1x1 expand
            if b == 0:
                layers.append((4 * width, size))  # projection shortcut
    return layers


def cifar_resnet_layers():
    """(C, H) of the three stages of a CIFAR ResNet-20/56 (H = W)."""
    return [(16, 32), (32, 16), (64, 8)]
