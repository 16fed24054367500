"""Shape bookkeeping: layer lists of the benchmark workloads and their operation counts.

GEMM view of a convolution (Section 1: the convolution lowers to a matrix-matrix
product): M = B*OH*OW output pixels, N = C_out, K = kh*kw*C_in.  One binary MAC is
one multiply and one add, so ops = 2*M*N*K.

``paper_table1_binary_counts`` recomputes the binary parameter and binary MAC totals
of the paper's own network from its configuration table (Table 1) and is checked
against the totals the paper prints (Table 2); it guards the counting rules used for
every throughput figure.
"""
from __future__ import annotations

from dataclasses import dataclass, asdict


@dataclass(frozen=True)
class ConvLayer:
    name: str
    H: int
    W: int
    C_in: int
    C_out: int
    k: int
    stride: int
    pad: int

    @property
    def OH(self) -> int:
        return (self.H + 2 * self.pad - self.k) // self.stride + 1

    @property
    def OW(self) -> int:
        return (self.W + 2 * self.pad - self.k) // self.stride + 1

    @property
    def K(self) -> int:
        return self.k * self.k * self.C_in

    def M(self, B: int) -> int:
        return B * self.OH * self.OW

    def macs(self, B: int = 1) -> int:
        return self.M(B) * self.C_out * self.K

    def ops(self, B: int = 1) -> int:
        return 2 * self.macs(B)

    def in_bytes(self, B: int) -> int:
        return B * self.H * self.W * self.C_in // 8

    def w_bytes(self) -> int:
        return self.C_out * self.K // 8

    def out_bits_bytes(self, B: int) -> int:
        return self.M(B) * self.C_out // 8

    def as_dict(self):
        return asdict(self)


def conv_out(H: int, k: int, stride: int, pad: int) -> int:
    return (H + 2 * pad - k) // stride + 1


# Single 3x3 layer: batch 1, 32x32x128 -> 32x32x128, stride 1, pad 1 (K = 1152).
SINGLE_3X3 = ConvLayer("single3x3", 32, 32, 128, 128, 3, 1, 1)
SINGLE_3X3_BATCH = 1

# GEMM sweep: M = N, K in bits.
GEMM_SWEEP_MN = (1024, 4096, 16384)
GEMM_SWEEP_K = (512, 2304, 4608, 9216)

# Stem / down-sampling shaped layers at batch 64.
STEM_DOWN = (
    ConvLayer("down112to56", 112, 112, 32, 64, 3, 2, 1),
    ConvLayer("down56to28", 56, 56, 64, 128, 3, 2, 1),
)
STEM_DOWN_BATCH = 64

# ResNet-style block stack at batch 128.
BLOCK_STACK = (
    ConvLayer("b1_1x1_256to128", 28, 28, 256, 128, 1, 1, 0),
    ConvLayer("b2_3x3_128", 28, 28, 128, 128, 3, 1, 1),
    ConvLayer("b3_1x1_128to512", 28, 28, 128, 512, 1, 1, 0),
    ConvLayer("b4_3x3s2_512", 28, 28, 512, 512, 3, 2, 1),
)
BLOCK_STACK_BATCH = 128


def _backbone18():
    L = []
    L.append(ConvLayer("L1_1x1_32", 224, 224, 32, 32, 1, 1, 0))       # the paper's stem shape (Table 1)
    L.append(ConvLayer("L2_3x3s2_32", 224, 224, 32, 32, 3, 2, 1))      # -> 112
    L.append(ConvLayer("L3_3x3s2_32to64", 112, 112, 32, 64, 3, 2, 1))  # -> 56
    L.append(ConvLayer("L4_3x3_64", 56, 56, 64, 64, 3, 1, 1))
    L.append(ConvLayer("L5_1x1_64", 56, 56, 64, 64, 1, 1, 0))
    L.append(ConvLayer("L6_3x3_64", 56, 56, 64, 64, 3, 1, 1))
    h, c = 56, 64
    n = 7
    for _ in range(3):
        L.append(ConvLayer(f"L{n}_3x3s2_{c}to{2*c}", h, h, c, 2 * c, 3, 2, 1))
        h //= 2
        c *= 2
        L.append(ConvLayer(f"L{n+1}_3x3_{c}", h, h, c, c, 3, 1, 1))
        L.append(ConvLayer(f"L{n+2}_1x1_{c}", h, h, c, c, 1, 1, 0))
        L.append(ConvLayer(f"L{n+3}_3x3_{c}", h, h, c, c, 3, 1, 1))
        n += 4
    return tuple(L)


# Backbone-shaped sequence at batch 256: 224x224 input binarized to 32 channels, 18 layers.
BACKBONE18 = _backbone18()
BACKBONE18_BATCH = 256
BACKBONE18_INPUT = (224, 224, 4, 8)   # H, W, real channels, replication R (4 * 8 = 32 sign channels)


def chain_macs(layers, B: int = 1) -> int:
    return sum(l.macs(B) for l in layers)


def chain_ops(layers, B: int = 1) -> int:
    return 2 * chain_macs(layers, B)


def gemm_ops(M: int, N: int, K: int) -> int:
    return 2 * M * N * K


# ---- the paper's own network (Table 1), for the bookkeeping pin ----------------------------------
# rows: (name, blocks, S, R, channels after replication, output resolution)
PAPER_TABLE1 = (
    ("stem replicate", 1, 1, 8, 32, 224),
    ("stem normal", 0, 1, 1, 32, 224),
    ("level1 down", 1, 2, 2, 64, 112),
    ("level1 normal", 0, 1, 1, 64, 112),
    ("level2 down", 1, 2, 2, 128, 56),
    ("level2 normal", 0, 1, 1, 128, 56),
    ("level3 down", 1, 2, 2, 256, 28),
    ("level3 normal", 1, 1, 1, 256, 28),
    ("level4 down", 1, 2, 2, 512, 14),
    ("level4 normal", 5, 1, 1, 512, 14),
    ("level5 down", 1, 2, 2, 1024, 7),
    ("level5 normal", 1, 1, 1, 1024, 7),
)


def paper_table1_binary_counts(P: int = 1):
    """(binary parameters, binary MACs per image) of the network of Table 1.

    Each building block (Section 4.2) has two binary 1x1 convolution modules on the
    residual path; a block configured for replication or down-sampling has a third
    one on its identity path (Section 4.2.3).  Every binary 1x1 conv is C x C after
    replication.  In a down-sampling block the first residual 1x1 runs before the
    strided depth-wise 3x3, i.e. at the input resolution S*H; the other convs run at
    the output resolution H.  P parallel branches multiply both totals by P.
    """
    params = 0
    macs = 0
    for _name, blocks, S, R, C, res in PAPER_TABLE1:
        special = (R > 1) or (S > 1)
        for _ in range(blocks):
            hw_out = res * res
            hw_in = (res * S) * (res * S)
            params += 2 * C * C
            macs += hw_in * C * C + hw_out * C * C
            if special:
                params += C * C
                macs += hw_out * C * C
    return P * params, P * macs


def paper_binary_1x1_convs(P: int = 1):
    """The binary 1x1 convolutions of the network of Table 1 as (ConvLayer, count) pairs, in network order.

    Same rules as ``paper_table1_binary_counts``: per block one C x C conv at the block's input resolution
    (S * res) and one at its output resolution, plus one more at the output resolution on the identity
    path of a replicate / down-sampling block; P parallel branches repeat every conv P times
    (Section 4.2.1).  Their MACs add up to the paper's 2.41e9 (4.83e9 for P = 2) per image.
    """
    out = []
    for name, blocks, S, R, C, res in PAPER_TABLE1:
        if blocks == 0:
            continue
        special = (R > 1) or (S > 1)
        tag = name.replace(" ", "_")
        if S > 1:
            out.append((ConvLayer(f"{tag}_in{res * S}_c{C}", res * S, res * S, C, C, 1, 1, 0), P * blocks))
            out.append((ConvLayer(f"{tag}_out{res}_c{C}", res, res, C, C, 1, 1, 0), P * blocks * (2 if special else 1)))
        else:
            out.append((ConvLayer(f"{tag}_{res}_c{C}", res, res, C, C, 1, 1, 0), P * blocks * (3 if special else 2)))
    return out
