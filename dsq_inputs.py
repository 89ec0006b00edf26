"""Seeded synthetic inputs and workload shapes for the DSQ low-bit conv path.

This module serves both the CPU oracle and the CUDA library and therefore
holds none of the method's arithmetic: it draws random fp32 tensors and random
integer codes, and it lists layer shapes.  Quantising, packing and convolving
are done by whoever consumes these arrays.

Five workloads (seed = 190805033*10 + workload id):
  1  one 3x3 conv, 64x56x56 -> 64, 4-bit (the first row of the paper's
     Table 8)
  2  plain GEMM, M=N=K in {1024, 4096, 8192}, b in {2, 3, 4}
  3  ResNet-18-shaped stack, 4-bit, batch 64 (the network of Table 9)
  4  MobileNetV2-shaped stack, 4-bit, batch 64
  5  VGG-16-shaped stack, 2-bit, batch 32
The ImageNet images and trained weights the paper used are replaced by random
tensors of the same shapes; the first and last layers of every network stay
outside the quantised path, as in the paper's Sec. 4.1.
"""
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

SEED_BASE = 190805033 * 10


def rng_for(workload_id: int, stream: int = 0) -> np.random.Generator:
    return np.random.default_rng([SEED_BASE + workload_id, stream])


def relu_normal(rng, shape, cap: Optional[float] = None) -> np.ndarray:
    """max(N(0,1), 0), optionally capped (ReLU6-like), fp32."""
    x = rng.standard_normal(shape, dtype=np.float32)
    np.maximum(x, 0.0, out=x)
    if cap is not None:
        np.minimum(x, np.float32(cap), out=x)
    return x


def normal(rng, shape, std: float) -> np.ndarray:
    return (rng.standard_normal(shape, dtype=np.float32)
            * np.float32(std)).astype(np.float32)


def uniform_codes(rng, shape, lo: int, hi: int) -> np.ndarray:
    """Integer codes uniform on [lo, hi] inclusive, int8."""
    return rng.integers(lo, hi + 1, size=shape, dtype=np.int8)


# --------------------------------------------------------------------------
# workload 1: single 3x3 convolution
# --------------------------------------------------------------------------
def conv3x3_case(workload_id=1, N=1, H=56, W=56, Cin=64, Cout=64, bits=4,
                 ksize=3, stride=1, pad=1, act_hi=2.0, w_std=0.05,
                 w_clip=0.1):
    rng = rng_for(workload_id)
    return dict(
        x=relu_normal(rng, (N, H, W, Cin)),
        w=normal(rng, (Cout, ksize, ksize, Cin), w_std),
        scale=normal(rng, (Cout,), 0.1),
        bias=normal(rng, (Cout,), 0.1),
        bits=bits, act_lo=0.0, act_hi=act_hi, w_lo=-w_clip, w_hi=w_clip,
        stride=stride, pad=pad)


# --------------------------------------------------------------------------
# workload 2: plain low-bit GEMM
# --------------------------------------------------------------------------
def gemm_case(M, N, K, bits, workload_id=2):
    """A [M,K] signed codes over the full b-bit range, B [N,K] unsigned codes
    over the full range, row_scale [M] ~ U(0.5,1.5) * 2^-10."""
    rng = rng_for(workload_id, stream=M * 31 + N * 17 + K * 7 + bits)
    half = 1 << (bits - 1)
    A = uniform_codes(rng, (M, K), -half, half - 1)
    B = uniform_codes(rng, (N, K), 0, 2 * half - 1)
    row_scale = (rng.uniform(0.5, 1.5, size=M) * 2.0 ** -10).astype(np.float32)
    return A, B, row_scale


def binary_gemm_case(M, N, K, workload_id=2):
    """Bit rows (0/1, uniform) of a binary GEMM and row_scale [M]."""
    rng = rng_for(workload_id, stream=M * 29 + N * 13 + K * 5 + 1)
    A = rng.integers(0, 2, size=(M, K)).astype(np.int8)
    B = rng.integers(0, 2, size=(N, K)).astype(np.int8)
    row_scale = (rng.uniform(0.5, 1.5, size=M) * 2.0 ** -10).astype(np.float32)
    return A, B, row_scale


def weight_only_case(M, N, K, bits, workload_id=2):
    """Weight-only linear layer: activations X [M,K] ~ N(0,1) rounded to
    bfloat16 (returned as float32 holding bf16 values), unsigned weight codes
    [N,K] uniform over the full range, per-channel clip u ~ U(0.05, 0.3) on
    [-u, u], bias ~ N(0, 0.1)."""
    rng = rng_for(workload_id, stream=M * 23 + N * 11 + K * 3 + bits)
    x = rng.standard_normal((M, K)).astype(np.float32)
    xi = x.view(np.uint32)
    xi = ((xi + 0x7FFF + ((xi >> 16) & 1)) & 0xFFFF0000).astype(np.uint32)   # round to nearest even
    x = xi.view(np.float32)
    q = rng.integers(0, 2 ** bits, size=(N, K)).astype(np.int8)
    u = rng.uniform(0.05, 0.3, size=N).astype(np.float32)
    bias = (rng.standard_normal(N) * 0.1).astype(np.float32)
    return x, q, u, bias


# --------------------------------------------------------------------------
# workloads 3-5: layer stacks.  A stack is a list of Layer records over named
# code tensors; each tensor has one quantiser range (bits, lo, hi).
# --------------------------------------------------------------------------
@dataclass
class Layer:
    name: str
    kind: str                 # "conv" | "dw" | "pool"
    src: str                  # input code tensor
    dst: str                  # output code tensor
    cin: int = 0
    cout: int = 0
    ksize: int = 1
    stride: int = 1
    pad: int = 0
    residual: Optional[str] = None   # code tensor added before requantising
    out_lo: float = 0.0       # requantiser range of dst
    out_hi: float = 1.0
    w_per_channel: bool = False


@dataclass
class Stack:
    name: str
    bits: int
    batch: int
    in_shape: tuple           # (H, W, C) of the synthesised input tensor
    in_lo: float
    in_hi: float
    in_cap: Optional[float]   # cap of the ReLU-normal input (ReLU6-like)
    layers: List[Layer] = field(default_factory=list)
    out: str = ""

    def macs_per_image(self) -> int:
        """Multiply-accumulates of the quantised layers for one image."""
        shapes = {"in": self.in_shape}
        total = 0
        for L in self.layers:
            H, W, _ = shapes[L.src]
            if L.kind == "pool":
                shapes[L.dst] = (H // 2, W // 2, shapes[L.src][2])
                continue
            Ho = (H + 2 * L.pad - L.ksize) // L.stride + 1
            Wo = (W + 2 * L.pad - L.ksize) // L.stride + 1
            shapes[L.dst] = (Ho, Wo, L.cout)
            per_out = L.ksize * L.ksize * (1 if L.kind == "dw" else L.cin)
            total += Ho * Wo * L.cout * per_out
        return total

    def tensor_shapes(self):
        shapes = {"in": self.in_shape}
        for L in self.layers:
            H, W, Cc = shapes[L.src]
            if L.kind == "pool":
                shapes[L.dst] = (H // 2, W // 2, Cc)
            else:
                Ho = (H + 2 * L.pad - L.ksize) // L.stride + 1
                Wo = (W + 2 * L.pad - L.ksize) // L.stride + 1
                shapes[L.dst] = (Ho, Wo, L.cout)
        return shapes


def resnet18_stack(batch=64, bits=4, workload_id=3, hw=56) -> Stack:
    """The 19 quantised convolutions of ResNet-18 behind the fp32 stem: four
    stages of two basic blocks; stages 2-4 open with a stride-2 block whose
    shortcut is a 1x1 stride-2 convolution.  Clip range of every ReLU output
    u ~ U(1,4), l = 0; shortcut convolutions (no ReLU) use [-u, u]."""
    rng = rng_for(workload_id, stream=1)
    st = Stack("resnet18", bits, batch, (hw, hw, 64), 0.0,
               float(rng.uniform(1, 4)), None)
    cur, cin = "in", 64
    for stage, cout in enumerate((64, 128, 256, 512), start=1):
        for blk in range(2):
            stride = 2 if (stage > 1 and blk == 0) else 1
            p = f"l{stage}b{blk}"
            ident = cur
            if stride != 1 or cin != cout:
                u = float(rng.uniform(1, 4))
                st.layers.append(Layer(p + "ds", "conv", cur, p + "ds", cin,
                                       cout, 1, stride, 0, None, -u, u))
                ident = p + "ds"
            st.layers.append(Layer(p + "c1", "conv", cur, p + "c1", cin, cout,
                                   3, stride, 1, None, 0.0,
                                   float(rng.uniform(1, 4))))
            st.layers.append(Layer(p + "c2", "conv", p + "c1", p + "c2", cout,
                                   cout, 3, 1, 1, ident, 0.0,
                                   float(rng.uniform(1, 4))))
            cur, cin = p + "c2", cout
    st.out = cur
    return st


def mobilenetv2_stack(batch=64, bits=4, workload_id=4, hw=112) -> Stack:
    """The 17 inverted-residual blocks of MobileNetV2 behind the fp32 stem
    (32 channels at 112x112) plus the final 1x1 320->1280.  Expansion 6
    (1 in the first block); every tensor requantised to [0, 6]."""
    st = Stack("mobilenetv2", bits, batch, (hw, hw, 32), 0.0, 6.0, 6.0)
    cfg = [(1, 16, 1, 1), (6, 24, 2, 2), (6, 32, 3, 2), (6, 64, 4, 2),
           (6, 96, 3, 1), (6, 160, 3, 2), (6, 320, 1, 1)]
    cur, cin, b = "in", 32, 0
    for t, c, n, s in cfg:
        for i in range(n):
            stride = s if i == 0 else 1
            p = f"b{b}"
            x, mid = cur, cin * t
            if t != 1:
                st.layers.append(Layer(p + "e", "conv", x, p + "e", cin, mid,
                                       1, 1, 0, None, 0.0, 6.0, True))
                x = p + "e"
            st.layers.append(Layer(p + "d", "dw", x, p + "d", mid, mid, 3,
                                   stride, 1, None, 0.0, 6.0, True))
            res = cur if (stride == 1 and cin == c) else None
            st.layers.append(Layer(p + "p", "conv", p + "d", p + "p", mid, c,
                                   1, 1, 0, res, 0.0, 6.0, True))
            cur, cin, b = p + "p", c, b + 1
    st.layers.append(Layer("last", "conv", cur, "last", cin, 1280, 1, 1, 0,
                           None, 0.0, 6.0, True))
    st.out = "last"
    return st


def vgg16_stack(batch=32, bits=2, workload_id=5, hw=224) -> Stack:
    """The 12 quantised 3x3 convolutions of VGG-16 behind the fp32 first
    convolution (64 channels at 224x224), with the four 2x2 max-pools that
    sit between them."""
    rng = rng_for(workload_id, stream=1)
    st = Stack("vgg16", bits, batch, (hw, hw, 64), 0.0,
               float(rng.uniform(1, 4)), None)
    plan = [64, "P", 128, 128, "P", 256, 256, 256, "P", 512, 512, 512, "P",
            512, 512, 512]
    cur, cin, i = "in", 64, 0
    for item in plan:
        if item == "P":
            st.layers.append(Layer(f"pool{i}", "pool", cur, f"pool{i}"))
            cur = f"pool{i}"
            continue
        i += 1
        st.layers.append(Layer(f"conv{i}", "conv", cur, f"conv{i}", cin, item,
                               3, 1, 1, None, 0.0, float(rng.uniform(1, 4))))
        cur, cin = f"conv{i}", item
    st.out = cur
    return st


def tiny_stack(bits=4, batch=2, workload_id=9) -> Stack:
    """A few layers of every kind on an 8x8 image: conv3x3, strided conv with
    a 1x1 shortcut and residual, depthwise, pool.  For fast parity tests."""
    st = Stack("tiny", bits, batch, (8, 8, 32), 0.0, 2.0, None)
    st.layers = [
        Layer("c1", "conv", "in", "c1", 32, 32, 3, 1, 1, None, 0.0, 2.5),
        Layer("ds", "conv", "c1", "ds", 32, 64, 1, 2, 0, None, -3.0, 3.0),
        Layer("c2", "conv", "c1", "c2", 32, 64, 3, 2, 1, None, 0.0, 3.0),
        Layer("c3", "conv", "c2", "c3", 64, 64, 3, 1, 1, "ds", 0.0, 2.0),
        Layer("dw", "dw", "c3", "dw", 64, 64, 3, 1, 1, None, 0.0, 6.0, True),
        Layer("pj", "conv", "dw", "pj", 64, 24, 1, 1, 0, None, 0.0, 6.0,
              True),
        Layer("pool", "pool", "pj", "pool"),
    ]
    st.out = "pool"
    return st


def stack_input(st: Stack, batch: Optional[int] = None,
                workload_id: int = 0) -> np.ndarray:
    """fp32 NHWC input of a stack: ReLU(N(0,1)), capped where the stack says
    so."""
    rng = rng_for(workload_id, stream=2)
    n = st.batch if batch is None else batch
    return relu_normal(rng, (n,) + tuple(st.in_shape), st.in_cap)


def stack_params(st: Stack, workload_id: int = 0):
    """Random-init fp32 parameters of every conv / depthwise layer:
      w     ~ N(0, var = 2/fan_in), fan_in = k*k*Cin (k*k for depthwise)
      w_lo, w_hi  clip at +-3 sigma: nominal sigma per layer, or the
                  empirical per-output-channel sigma when w_per_channel
      bias  ~ N(0, std 0.1)
    The dequantisation scale is not drawn: it is Delta_a * Delta_w and is
    derived by the consumer from the ranges."""
    rng = rng_for(workload_id, stream=3)
    params = {}
    for L in st.layers:
        if L.kind == "pool":
            continue
        if L.kind == "dw":
            shape, fan_in = (L.cout, L.ksize, L.ksize), L.ksize * L.ksize
        else:
            shape = (L.cout, L.ksize, L.ksize, L.cin)
            fan_in = L.ksize * L.ksize * L.cin
        sigma = float(np.sqrt(2.0 / fan_in))
        w = normal(rng, shape, sigma)
        if L.w_per_channel:
            s = w.reshape(L.cout, -1).std(axis=1).astype(np.float32)
            s = np.maximum(s, np.float32(1e-3))
            w_hi = (3.0 * s).astype(np.float32)
        else:
            w_hi = np.full((1,), 3.0 * sigma, np.float32)
        params[L.name] = dict(w=w, w_lo=-w_hi, w_hi=w_hi,
                              bias=normal(rng, (L.cout,), 0.1))
    return params
