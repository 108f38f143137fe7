"""Seeded synthetic inputs shaped like the paper's ViT / LLM workloads.

This module only draws random numbers and names shapes.  It contains none of
the method's arithmetic (no quantizer, no matmul, no CWAC fit): both the CUDA
path and the CPU oracle receive the arrays produced here as inputs.

The paper evaluates on ImageNet / COCO / DiT / LLaMA activations of trained
networks (Section 4, Appendix A).  Those are not available offline, so the
generators below take the *shapes*, calibration-set sizes and the value
structure (outlier-heavy transformer activations, small-std weights) of those
workloads and stand in for them.

Two back ends with the same recipes:
  * ``host_*``  : numpy ``Generator(Philox(key))`` -> identical bytes on every
    machine; used by the parity tests (the oracle and the GPU see these bytes).
  * ``device_*``: ``torch.Generator`` on a CUDA device for arrays that are too
    large to draw on the host; whoever needs them on the host copies them back.
"""
from __future__ import annotations

import dataclasses
import zlib
from typing import Dict, List, Optional, Tuple

import numpy as np

TOKENS_PER_IMAGE = 197  # ViT patch tokens + class token at 224x224 / 16


@dataclasses.dataclass(frozen=True)
class LayerSpec:
    """One quantized linear layer of a workload (all sizes in elements)."""
    name: str
    M: int                 # tokens of one inference batch
    K: int                 # input features
    N: int                 # output features / channels
    w_bits: int            # 8 or 4 (4 = packed two per byte)
    out: str               # "int8" (per-token requant) or "bf16"
    act: str               # activation recipe: "sparse_outlier" | "lognormal_channel" | "channel_outlier"
    calib_rows: int        # calibration tokens used to fit CWAC for this layer
    planted: bool = False  # config 4: CWAC (a, b) is planted and refit

    @property
    def ops(self) -> int:
        return 2 * self.M * self.N * self.K


def _vit_block(prefix: str, M: int, dim: int, mlp: int, w_bits: int, out: str, calib_rows: int) -> List[LayerSpec]:
    shapes = [("qkv", dim, 3 * dim), ("proj", dim, dim), ("fc1", dim, mlp), ("fc2", mlp, dim)]
    return [LayerSpec(f"{prefix}.{n}", M, k, nn, w_bits, out, "lognormal_channel", calib_rows) for n, k, nn in shapes]


def config_layers(cfg: int, full: bool = True) -> List[LayerSpec]:
    """Layer list of workload ``cfg`` (1-based, numbering of the benchmark configs).

    cfg 1: one W8A8 layer 788x384 -> 1536, CWAC fit on 32 images.
    cfg 2: DeiT-S W8A8 stack, 12 blocks, batch 64 images, CWAC fit on 512 images.
    cfg 3: ViT-B W4A8 stack, 12 blocks, batch 128 images, BF16 out, CWAC fit on 1024 images.
    cfg 4: LLaMA-7B shaped W8A8 layers at M=2048 and 8192, CWAC planted and refit
           from 128 x 2048 calibration tokens.
    ``full=False`` returns one block (cfg 2, 3) instead of twelve.
    """
    T = TOKENS_PER_IMAGE
    if cfg == 1:
        return [LayerSpec("cfg1.fc1", 4 * T, 384, 1536, 8, "int8", "sparse_outlier", 32 * T)]
    if cfg == 2:
        nblk = 12 if full else 1
        out: List[LayerSpec] = []
        for b in range(nblk):
            out += _vit_block(f"deit_s.{b}", 64 * T, 384, 1536, 8, "int8", 512 * T)
        return out
    if cfg == 3:
        nblk = 12 if full else 1
        out = []
        for b in range(nblk):
            out += _vit_block(f"vit_b.{b}", 128 * T, 768, 3072, 4, "bf16", 1024 * T)
        return out
    if cfg == 4:
        out = []
        for M in (2048, 8192):
            for n, k, nn in [("q", 4096, 4096), ("k", 4096, 4096), ("v", 4096, 4096), ("o", 4096, 4096),
                             ("gate", 4096, 11008), ("up", 4096, 11008), ("down", 11008, 4096)]:
                out.append(LayerSpec(f"llama7b.M{M}.{n}", M, k, nn, 8, "int8", "channel_outlier", 128 * 2048, True))
        return out
    raise ValueError(f"no forward layers for config {cfg}")


def resnet50_pointwise_layers(batch: int = 32, calib_images: int = 32) -> List[LayerSpec]:
    """ResNet-50 shaped 1x1 convolutions (the paper also places CWAC after every quantized convolution, Section 3.3
    and Table 1).  In NHWC layout a 1x1 convolution over a B x H x W x C_in activation IS this linear layer with
    M = B*H*W tokens, K = C_in, N = C_out, so no new kernel is involved: these shapes only widen the workload set
    (first and last pointwise convolution of a bottleneck in each of the four stages)."""
    out: List[LayerSpec] = []
    for stage, (hw, cin, mid, cout) in enumerate([(56, 256, 64, 256), (28, 512, 128, 512), (14, 1024, 256, 1024),
                                                  (7, 2048, 512, 2048)]):
        M, R = batch * hw * hw, calib_images * hw * hw
        out.append(LayerSpec(f"resnet50.s{stage}.reduce", M, cin, mid, 8, "int8", "lognormal_channel", R))
        out.append(LayerSpec(f"resnet50.s{stage}.expand", M, mid, cout, 8, "int8", "lognormal_channel", R))
    return out


CALIB_SWEEP_ROWS = 2048 * TOKENS_PER_IMAGE   # config 5: 403,456 rows
CALIB_SWEEP_WIDTHS = (768, 2304, 3072)
CALIB_SWEEP_BITS = (8, 4)


def _key(seed: int, *tags) -> int:
    """Stable 64-bit stream key from (seed, tags)."""
    h = zlib.crc32(repr(tags).encode())
    return ((seed & 0xFFFFFFFF) << 32) | h


def host_rng(seed: int, *tags) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=_key(seed, *tags)))


# --------------------------------------------------------------------------- host (numpy) generators

def host_activations(recipe: str, rows: int, K: int, seed: int, tag: str) -> np.ndarray:
    """FP32 activations [rows, K] following ``recipe``.

    sparse_outlier    : N(0,1), each element x20 with probability 0.01      (config 1)
    lognormal_channel : N(0,1) x g_k, g_k ~ LogNormal(0,1) per input channel  (configs 2, 3;
                        the per-channel factors depend on (seed, layer) only, so a layer's
                        calibration tokens and inference tokens share them)
    channel_outlier   : N(0,1), round(0.001 K) input channels x50             (config 4)
    """
    layer = tag.split("|")[0]
    rng = host_rng(seed, "act", tag)
    X = rng.standard_normal((rows, K), dtype=np.float32)
    if recipe == "sparse_outlier":
        mask = rng.random((rows, K), dtype=np.float32) < np.float32(0.01)
        X[mask] *= np.float32(20.0)
    elif recipe == "lognormal_channel":
        g = host_rng(seed, "act_chan", layer).lognormal(0.0, 1.0, size=K).astype(np.float32)
        X *= g[None, :]
    elif recipe == "channel_outlier":
        n_out = int(round(0.001 * K))
        idx = host_rng(seed, "act_chan", layer).choice(K, size=n_out, replace=False)
        X[:, idx] *= np.float32(50.0)
    elif recipe == "normal":
        pass
    else:
        raise ValueError(recipe)
    return X


def host_weights(N: int, K: int, seed: int, tag: str, std: float = 0.02) -> np.ndarray:
    """FP32 weights [N, K] ~ N(0, std) (std = 0.02, the usual ViT / LLM init)."""
    rng = host_rng(seed, "w", tag)
    return (rng.standard_normal((N, K), dtype=np.float32) * np.float32(std)).astype(np.float32)


def host_bias(N: int, seed: int, tag: str, std: float = 0.01) -> np.ndarray:
    rng = host_rng(seed, "bias", tag)
    return (rng.standard_normal(N, dtype=np.float32) * np.float32(std)).astype(np.float32)


def host_planted_cwac(N: int, seed: int, tag: str) -> Tuple[np.ndarray, np.ndarray]:
    """Config 4: planted a ~ N(1, 0.05), b ~ N(0, 0.02)."""
    rng = host_rng(seed, "planted", tag)
    a = (1.0 + 0.05 * rng.standard_normal(N)).astype(np.float32)
    b = (0.02 * rng.standard_normal(N)).astype(np.float32)
    return a, b


def host_layer_inputs(spec: LayerSpec, seed: int = 0, rows: Optional[int] = None,
                      calib_rows: Optional[int] = None) -> Dict[str, np.ndarray]:
    """All FP32 inputs of one layer: inference tokens X, calibration tokens Xc, W, bias."""
    rows = spec.M if rows is None else rows
    calib_rows = spec.calib_rows if calib_rows is None else calib_rows
    d = {
        "X": host_activations(spec.act, rows, spec.K, seed, spec.name + "|infer"),
        "Xc": host_activations(spec.act, calib_rows, spec.K, seed, spec.name + "|calib"),
        "W": host_weights(spec.N, spec.K, seed, spec.name),
        "bias": host_bias(spec.N, seed, spec.name),
    }
    if spec.planted:
        d["a_star"], d["b_star"] = host_planted_cwac(spec.N, seed, spec.name)
    return d


def host_calib_pair(rows: int, C: int, bits: int, seed: int = 0, ld: Optional[int] = None
                    ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Config 5 pair (fp_out, q_out), both FP32 [rows, C] (leading dimension ``ld`` >= C).

    fp_out = N(0,1) x sigma_c with sigma_c ~ LogNormal(0, 0.5);
    q_out  = fp_out + U(-D_c/2, D_c/2),  D_c = 8 sigma_c / (2^bits - 1)
    (a range of +-4 sigma_c divided into 2^bits - 1 uniform steps).
    Returns (fp_out, q_out, sigma).
    """
    ld = C if ld is None else ld
    sig = host_rng(seed, "calib_sigma", C, bits).lognormal(0.0, 0.5, size=C).astype(np.float32)
    rng = host_rng(seed, "calib", rows, C, bits)
    fp = np.zeros((rows, ld), dtype=np.float32)
    q = np.zeros((rows, ld), dtype=np.float32)
    fp[:, :C] = rng.standard_normal((rows, C), dtype=np.float32) * sig[None, :]
    delta = (np.float32(8.0) * sig / np.float32(2 ** bits - 1)).astype(np.float32)
    u = rng.random((rows, C), dtype=np.float32) - np.float32(0.5)
    q[:, :C] = fp[:, :C] + u * delta[None, :]
    return fp, q, sig


# --------------------------------------------------------------------------- device (torch) generators

def device_activations(recipe: str, rows: int, K: int, seed: int, tag: str, device="cuda"):
    """Same recipes as :func:`host_activations`, drawn on ``device`` (different bytes, same law)."""
    import torch
    layer = tag.split("|")[0]
    g = torch.Generator(device=device)
    g.manual_seed(_key(seed, "act", tag) & 0x7FFFFFFFFFFFFFFF)
    X = torch.randn((rows, K), generator=g, device=device, dtype=torch.float32)
    if recipe == "sparse_outlier":
        mask = torch.rand((rows, K), generator=g, device=device) < 0.01
        X = torch.where(mask, X * 20.0, X)
    elif recipe == "lognormal_channel":
        gk = host_rng(seed, "act_chan", layer).lognormal(0.0, 1.0, size=K).astype(np.float32)
        X *= torch.from_numpy(gk).to(device)[None, :]
    elif recipe == "channel_outlier":
        n_out = int(round(0.001 * K))
        idx = host_rng(seed, "act_chan", layer).choice(K, size=n_out, replace=False)
        X[:, torch.from_numpy(idx).to(device)] *= 50.0
    elif recipe == "normal":
        pass
    else:
        raise ValueError(recipe)
    return X


def device_weights(N: int, K: int, seed: int, tag: str, std: float = 0.02, device="cuda"):
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(_key(seed, "w", tag) & 0x7FFFFFFFFFFFFFFF)
    return torch.randn((N, K), generator=g, device=device, dtype=torch.float32) * std


def device_calib_pair(rows: int, C: int, bits: int, seed: int = 0, device="cuda"):
    """Config 5 pair drawn on the device (same law as :func:`host_calib_pair`)."""
    import torch
    sig = host_rng(seed, "calib_sigma", C, bits).lognormal(0.0, 0.5, size=C).astype(np.float32)
    sig_d = torch.from_numpy(sig).to(device)
    g = torch.Generator(device=device)
    g.manual_seed(_key(seed, "calib", rows, C, bits) & 0x7FFFFFFFFFFFFFFF)
    fp = torch.randn((rows, C), generator=g, device=device, dtype=torch.float32)
    fp *= sig_d[None, :]
    q = torch.rand((rows, C), generator=g, device=device, dtype=torch.float32)
    q -= 0.5
    q *= (8.0 * sig_d / float(2 ** bits - 1))[None, :]
    q += fp
    return fp, q, sig
