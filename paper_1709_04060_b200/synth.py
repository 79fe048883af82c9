"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds none of the method's arithmetic: it only draws logical
integer tensors (numpy int32, one element per value) and sorted integer
thresholds.  Both the CPU oracle's tests and the CUDA path's tests/benchmarks
take their inputs from here, so that the two sides see identical data.

Encodings: UNSIGNED b bits -> [0, 2^b - 1]; SIGNED -> [-2^(b-1), 2^(b-1) - 1];
BIPOLAR (1 bit) -> {-1, +1}.  8-bit operands use the same rule with b = 8.
"""
from dataclasses import dataclass, field
import numpy as np

UNSIGNED, SIGNED, BIPOLAR = 0, 1, 2
BASE_SEED = 170904060


def value_range(bits: int, enc: int):
    if enc == BIPOLAR:
        return -1, 1
    if enc == SIGNED:
        return -(1 << (bits - 1)), (1 << (bits - 1)) - 1
    return 0, (1 << bits) - 1


def draw_operand(rng, shape, bits: int, enc: int) -> np.ndarray:
    """Uniform over the encoding's value set."""
    if enc == BIPOLAR:
        return (2 * rng.integers(0, 2, size=shape, dtype=np.int32) - 1).astype(np.int32)
    lo, hi = value_range(bits, enc)
    return rng.integers(lo, hi + 1, size=shape, dtype=np.int32)


def _moments(bits: int, enc: int):
    lo, hi = value_range(bits, enc)
    vals = np.array([-1, 1] if enc == BIPOLAR else list(range(lo, hi + 1)), dtype=np.float64)
    return float(vals.mean()), float((vals ** 2).mean())


def acc_stats(K: int, w_bits, w_enc, a_bits, a_enc):
    """Mean and standard deviation of a depth-K accumulator of uniform operands."""
    ew, ew2 = _moments(w_bits, w_enc)
    ea, ea2 = _moments(a_bits, a_enc)
    mu = K * ew * ea
    var = K * (ew2 * ea2 - (ew * ea) ** 2)
    return mu, float(np.sqrt(max(var, 1.0)))


def draw_thresholds(rng, rows: int, n_thr: int, mu: float, sigma: float,
                    spread: float = 3.0) -> np.ndarray:
    """Per-row sorted int32 thresholds, uniform in [mu - spread*sigma, mu + spread*sigma]."""
    lo = int(np.floor(mu - spread * sigma))
    hi = int(np.ceil(mu + spread * sigma))
    t = rng.integers(lo, hi + 1, size=(rows, n_thr), dtype=np.int64)
    t.sort(axis=1)
    return t.astype(np.int32)


@dataclass
class GemmCase:
    M: int
    N: int
    K: int
    w_bits: int
    a_bits: int
    w_enc: int
    a_enc: int
    out_bits: int
    W: np.ndarray      # int32 [M][K]
    At: np.ndarray     # int32 [N][K]  (activations, depth contiguous)
    thr: np.ndarray    # int32 [M][2^out_bits - 1], sorted per row


def gemm_case(seed: int, M, N, K, w_bits, a_bits, w_enc=None, a_enc=UNSIGNED,
              out_bits=None, spread: float = 3.0) -> GemmCase:
    """One fused GEMM+threshold problem.  Weights default to BIPOLAR for
    w_bits == 1 and SIGNED otherwise, as in the paper-shaped configurations."""
    if w_enc is None:
        w_enc = BIPOLAR if w_bits == 1 else SIGNED
    if out_bits is None:
        out_bits = min(a_bits, 4)
    ss = np.random.SeedSequence([BASE_SEED, seed])
    r_w, r_a, r_t = (np.random.default_rng(s) for s in ss.spawn(3))
    W = draw_operand(r_w, (M, K), w_bits, w_enc)
    At = draw_operand(r_a, (N, K), a_bits, a_enc)
    mu, sigma = acc_stats(K, w_bits, w_enc, a_bits, a_enc)
    thr = draw_thresholds(r_t, M, (1 << out_bits) - 1, mu, sigma, spread)
    return GemmCase(M, N, K, w_bits, a_bits, w_enc, a_enc, out_bits, W, At, thr)


@dataclass
class ConvCase:
    B: int
    H: int
    Wd: int
    C: int
    OC: int
    KH: int
    KW: int
    stride: int
    pad: int
    w_bits: int
    a_bits: int
    w_enc: int
    a_enc: int
    out_bits: int
    In: np.ndarray     # int32 [B][H][W][C]  channels-last
    Wt: np.ndarray     # int32 [OC][KH][KW][C]
    thr: np.ndarray    # int32 [OC][2^out_bits - 1]

    @property
    def OH(self):
        return (self.H + 2 * self.pad - self.KH) // self.stride + 1

    @property
    def OW(self):
        return (self.Wd + 2 * self.pad - self.KW) // self.stride + 1


def conv_case(seed: int, B, H, Wd, C, OC, KH, KW, stride, pad, w_bits, a_bits,
              w_enc=None, a_enc=UNSIGNED, out_bits=2, spread: float = 3.0) -> ConvCase:
    if w_enc is None:
        w_enc = BIPOLAR if w_bits == 1 else SIGNED
    ss = np.random.SeedSequence([BASE_SEED, seed])
    r_w, r_a, r_t = (np.random.default_rng(s) for s in ss.spawn(3))
    Wt = draw_operand(r_w, (OC, KH, KW, C), w_bits, w_enc)
    In = draw_operand(r_a, (B, H, Wd, C), a_bits, a_enc)
    mu, sigma = acc_stats(KH * KW * C, w_bits, w_enc, a_bits, a_enc)
    thr = draw_thresholds(r_t, OC, (1 << out_bits) - 1, mu, sigma, spread)
    return ConvCase(B, H, Wd, C, OC, KH, KW, stride, pad, w_bits, a_bits, w_enc,
                    a_enc, out_bits, In, Wt, thr)


def conv2_alexnet_case(B: int, seed: int = 3) -> ConvCase:
    """AlexNet conv2-shaped W1A2 layer: 27x27x96 input, 256 5x5 filters, pad 2
    (lowered GEMM rows 256, depth 2400, cols 729 per image; Table 3)."""
    return conv_case(seed, B, 27, 27, 96, 256, 5, 5, 1, 2, 1, 2)


# --- AlexNet-shaped streamlined W1A2 network (Section 4.2, Table 3 shapes) ---

@dataclass
class LayerSpec:
    name: str
    kind: str              # "conv" | "fc"
    OC: int
    KH: int = 1
    KW: int = 1
    stride: int = 1
    pad: int = 0
    w_bits: int = 1
    w_enc: int = BIPOLAR
    a_bits: int = 2        # bit width of this layer's INPUT activations
    out_bits: int = 2      # 0 -> raw int32 accumulators (last layer)
    pool: bool = False     # 3x3 stride-2 max-pool after the threshold


ALEXNET_LAYERS = (
    LayerSpec("conv1", "conv", 96, 11, 11, 4, 0, 8, SIGNED, 8, 2, True),
    LayerSpec("conv2", "conv", 256, 5, 5, 1, 2, 1, BIPOLAR, 2, 2, True),
    LayerSpec("conv3", "conv", 384, 3, 3, 1, 1, 1, BIPOLAR, 2, 2, False),
    LayerSpec("conv4", "conv", 384, 3, 3, 1, 1, 1, BIPOLAR, 2, 2, False),
    LayerSpec("conv5", "conv", 256, 3, 3, 1, 1, 1, BIPOLAR, 2, 2, True),
    LayerSpec("fc6", "fc", 4096, a_bits=2, out_bits=2),
    LayerSpec("fc7", "fc", 4096, a_bits=2, out_bits=2),
    LayerSpec("fc8", "fc", 1000, w_bits=8, w_enc=SIGNED, a_bits=2, out_bits=0),
)


@dataclass
class NetCase:
    B: int
    image: np.ndarray                      # int32 [B][227][227][3], values 0..255
    layers: tuple = ALEXNET_LAYERS
    weights: dict = field(default_factory=dict)   # name -> int32 [OC][KH][KW][C] or [OC][K]
    thr: dict = field(default_factory=dict)       # name -> int32 [OC][3]


def alexnet_case(B: int, seed: int = 4, hw: int = 227) -> NetCase:
    """Random-init AlexNet-shaped network and a batch of uint8 images.

    Thresholds of each layer are sorted integers drawn uniformly within one
    standard deviation of the mean of that layer's accumulator, with the moments
    computed for uniformly distributed input codes; any sorted integers are
    legal thresholds, this choice only keeps all four codes populated."""
    ss = np.random.SeedSequence([BASE_SEED, seed])
    streams = ss.spawn(1 + 2 * len(ALEXNET_LAYERS))
    image = draw_operand(np.random.default_rng(streams[0]), (B, hw, hw, 3), 8, UNSIGNED)
    case = NetCase(B=B, image=image)
    H, C = hw, 3
    flat = None
    for li, L in enumerate(ALEXNET_LAYERS):
        r_w = np.random.default_rng(streams[1 + 2 * li])
        r_t = np.random.default_rng(streams[2 + 2 * li])
        if L.kind == "conv":
            K = L.KH * L.KW * C
            case.weights[L.name] = draw_operand(r_w, (L.OC, L.KH, L.KW, C), L.w_bits, L.w_enc)
            H = (H + 2 * L.pad - L.KH) // L.stride + 1
            if L.pool:
                H = (H - 3) // 2 + 1
            C = L.OC
            flat = H * H * C
        else:
            K = flat
            case.weights[L.name] = draw_operand(r_w, (L.OC, K), L.w_bits, L.w_enc)
            flat = L.OC
        if L.out_bits:
            mu, sigma = acc_stats(K, L.w_bits, L.w_enc, L.a_bits, UNSIGNED)
            case.thr[L.name] = draw_thresholds(r_t, L.OC, (1 << L.out_bits) - 1,
                                               mu, sigma, spread=1.0)
    return case
