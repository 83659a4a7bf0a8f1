"""Seeded synthetic layer workloads: shapes and input generators only.

This module holds none of the method's arithmetic.  It names the layer shapes
(ResNet-style 3x3 blocks, a MobileNetV2 inverted-residual block, a
DeepLabV3/UPerNet decoder conv, a ResNet-34-like stage, and the seven layers of
the paper's on-device test table) and draws x, g_y and W for them from a seeded
generator.  The same bits feed the CUDA path and the CPU checker; for bf16 runs
the tensors are rounded to bf16 here, once, so that input rounding is not
counted as error on either side.

Value recipes:
  x    "normal"  N(0,1);  "relu" max(N(0,1),0);  "relu6" clamp(N(0,1),0,6)
  g_y  N(0, gy_std)  (gy_std is a standard deviation)
  W    Kaiming-normal, std = sqrt(2 / (C_in/groups * KH * KW))
Seeds: 1000 * config + tensor id (0 = x, 1 = g_y, 2 = W) + 10 * layer index.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class Layer:
    name: str
    config: int          # 1..5 headline configs, 6 = on-device table, 0 = ad hoc
    index: int           # layer index inside the config (seeding)
    N: int
    C_in: int
    C_out: int
    H: int
    W: int
    K: int
    groups: int
    r: int
    dtype: str           # "f32" | "bf16"
    x_dist: str = "normal"
    gy_std: float = 1.0

    @property
    def pad(self) -> int:
        return (self.K - 1) // 2

    @property
    def C_ig(self) -> int:
        return self.C_in // self.groups

    @property
    def Hp(self) -> int:
        return -(-self.H // self.r)

    @property
    def Wp(self) -> int:
        return -(-self.W // self.r)

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def with_(self, **kw) -> "Layer":
        return replace(self, **kw)

    # ---- byte / flop accounting of one layer backward (shapes only) ----
    def numel_x(self) -> int:
        return self.N * self.C_in * self.H * self.W

    def numel_gy(self) -> int:
        return self.N * self.C_out * self.H * self.W

    def numel_w(self) -> int:
        return self.C_out * self.C_ig * self.K * self.K

    def numel_stash(self) -> int:
        if self.r == 1:
            return self.numel_x()
        return self.N * self.C_in * self.Hp * self.Wp

    def backward_bytes(self) -> int:
        """Bytes the method itself must move: read g_y, stash, W once; write
        g_X and g_W (fp32) once."""
        e = self.elem_bytes
        return e * (self.numel_gy() + self.numel_x() + self.numel_stash() + self.numel_w()) \
            + 4 * self.numel_w()

    def stash_bytes_moved(self) -> int:
        e = self.elem_bytes
        return e * (self.numel_x() + self.numel_stash())

    def reduced_flops(self) -> int:
        """2 M C_out C_in/groups for each of the two reduced contractions."""
        M = self.N * self.Hp * self.Wp
        return 2 * 2 * M * self.C_out * self.C_ig


def torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


def _draw(shape, seed: int) -> torch.Tensor:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    return torch.randn(shape, generator=g, dtype=torch.float32)


def make_inputs(L: Layer) -> tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """(x, g_y, W) on the CPU in L.dtype, drawn in fp32 and rounded once."""
    base = 1000 * L.config + 10 * L.index
    if L.config == 1:
        base = 0
    x = _draw((L.N, L.C_in, L.H, L.W), base + 0)
    if L.x_dist == "relu":
        x = x.clamp_(min=0.0)
    elif L.x_dist == "relu6":
        x = x.clamp_(min=0.0, max=6.0)
    elif L.x_dist != "normal":
        raise ValueError(L.x_dist)
    gy = _draw((L.N, L.C_out, L.H, L.W), base + 1) * L.gy_std
    w = _draw((L.C_out, L.C_ig, L.K, L.K), base + 2) * math.sqrt(2.0 / (L.C_ig * L.K * L.K))
    dt = torch_dtype(L.dtype)
    return x.to(dt).contiguous(), gy.to(dt).contiguous(), w.to(dt).contiguous()


# ---------------------------------------------------------------------------
# The five headline configurations
# ---------------------------------------------------------------------------

def config1(r: int = 2) -> list[Layer]:
    return [Layer("cfg1_conv3x3", 1, 0, 2, 16, 16, 32, 32, 3, 1, r, "f32", "normal", 1.0)]


def config2() -> list[Layer]:
    return [Layer("cfg2_resnet3x3", 2, 0, 64, 256, 256, 28, 28, 3, 1, 2, "bf16", "relu", 1e-2)]


def config3(r: int = 2) -> list[Layer]:
    return [
        Layer("cfg3a_pw_96_576", 3, 0, 128, 96, 576, 28, 28, 1, 1, r, "f32", "relu6", 1e-2),
        Layer("cfg3b_dw_576", 3, 1, 128, 576, 576, 28, 28, 3, 576, r, "f32", "relu6", 1e-2),
        Layer("cfg3c_pw_576_96", 3, 2, 128, 576, 96, 28, 28, 1, 1, r, "f32", "relu6", 1e-2),
    ]


def config4() -> list[Layer]:
    return [Layer("cfg4_decoder3x3", 4, 0, 8, 512, 256, 128, 128, 3, 1, 4, "bf16", "relu", 1e-3)]


def config5(r: int = 2, dtype: str = "f32") -> list[Layer]:
    return [
        Layer("cfg5a_res34_3x3", 5, 0, 256, 512, 512, 16, 16, 3, 1, r, dtype, "relu", 1e-2),
        Layer("cfg5b_pw_512_2048", 5, 1, 256, 512, 2048, 16, 16, 1, 1, r, dtype, "relu", 1e-2),
    ]


def all_headline_layers() -> list[Layer]:
    out = config1(2) + config1(1) + config2() + config3(2) + config3(4) + config4()
    for dt in ("f32", "bf16"):
        for r in (2, 4, 8):
            out += config5(r, dt)
    return out


# The paper's on-device latency test cases (Table "Layer configuration for test
# cases"): batch 32, 3x3, stride 1, pad 1; (C_in, C_out, width, height).
_ONDEVICE = [(128, 128, 120, 160), (256, 256, 60, 80), (512, 512, 30, 40),
             (512, 512, 14, 14), (256, 256, 14, 14), (128, 128, 28, 28), (64, 64, 56, 56)]


def ondevice_table(r: int = 2, dtype: str = "f32", N: int = 32) -> list[Layer]:
    return [Layer(f"ondevice{i}_{ci}x{h}x{w}", 6, i, N, ci, co, h, w, 3, 1, r, dtype, "relu", 1e-2)
            for i, (ci, co, w, h) in enumerate(_ONDEVICE)]
