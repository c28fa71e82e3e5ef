"""Workload definitions: parameter lists shaped like the paper's models (Section 5: ResNet-56 on
CIFAR-100, ResNet-50 on ImageNet) plus a small ResNet-20 and a 12-layer transformer encoder, and the
five benchmark configurations built on them.  Shapes only -- no weights, no data, no arithmetic of the
method.  Every tensor of a list is its own compression segment (Section 5: compression is layer-wise).
"""
from dataclasses import dataclass, field
from typing import List

IDENTITY, SIGN, TOPK = 0, 1, 2
EF, SAEF = 0, 1


def resnet_cifar_sizes(n_blocks: int, num_classes: int) -> List[int]:
    """CIFAR ResNet-(6n+2): 3x3 stem 3->16, three stages of n basic blocks at 16/32/64 channels with
    parameter-free shortcuts, a BN (scale, bias) pair after every conv, FC 64 x classes + bias."""
    sizes = [3 * 16 * 9, 16, 16]
    cin = 16
    for cout in (16, 32, 64):
        for _ in range(n_blocks):
            sizes += [cin * cout * 9, cout, cout, cout * cout * 9, cout, cout]
            cin = cout
    sizes += [64 * num_classes, num_classes]
    return sizes


def resnet50_sizes() -> List[int]:
    """ResNet-50: 7x7 stem, bottleneck stages (3,4,6,3) at planes 64/128/256/512 (expansion 4), a 1x1
    downsample conv + BN in the first block of each stage, BN pair after every conv, FC 2048x1000 + bias."""
    sizes = [7 * 7 * 3 * 64, 64, 64]
    cin = 64
    for planes, blocks in ((64, 3), (128, 4), (256, 6), (512, 3)):
        for b in range(blocks):
            cout = planes * 4
            sizes += [cin * planes, planes, planes, planes * planes * 9, planes, planes, planes * cout, cout, cout]
            if b == 0:
                sizes += [cin * cout, cout, cout]
            cin = cout
    sizes += [2048 * 1000, 1000]
    return sizes


def encoder_sizes(layers: int = 12, hidden: int = 768, ffn: int = 3072, vocab: int = 30522,
                  positions: int = 512) -> List[int]:
    """Transformer encoder: word/position/type embeddings + LayerNorm; per layer four hidden x hidden
    projections with biases, LayerNorm, FFN up/down with biases, LayerNorm; pooler."""
    sizes = [vocab * hidden, positions * hidden, 2 * hidden, hidden, hidden]
    for _ in range(layers):
        sizes += [hidden * hidden, hidden] * 4 + [hidden, hidden]
        sizes += [hidden * ffn, ffn, ffn * hidden, hidden, hidden, hidden]
    sizes += [hidden * hidden, hidden]
    return sizes


def blockwise_sizes(tensor_sizes: List[int], block: int) -> List[int]:
    """Block-wise compression (the block-wise scaled sign of the related work, Section 2): every tensor is
    cut into consecutive segments of `block` elements (the last one of a tensor may be shorter) and each
    segment is compressed on its own.  To the library a segment is simply a tensor of the list."""
    if block < 1:
        raise ValueError("block must be >= 1")
    out: List[int] = []
    for n in tensor_sizes:
        full, rest = divmod(n, block)
        out += [block] * full
        if rest:
            out.append(rest)
    return out


@dataclass
class Workload:
    name: str
    num_workers: int
    tensor_sizes: List[int]
    compressor: int
    iterations: int
    momentum: float = 0.9
    lr: float = 0.1
    weight_decay: float = 0.0
    topk_num: int = 1
    topk_den: int = 100
    log10_scale_lo: float = -4.0       # per-tensor gradient scale s_j = 10^(lo + (hi-lo) u_j)
    log10_scale_hi: float = -1.0
    outlier_per_65536: int = 0         # entries whose hash lane falls below this are multiplied ...
    outlier_mult: float = 1.0          # ... by this factor (heavy tail)
    avg_period_paper: int = 20         # the one finite averaging period the paper uses (Section 5)
    server_compress: int = 1
    mode: int = SAEF
    extra: dict = field(default_factory=dict)

    @property
    def d(self) -> int:
        return sum(self.tensor_sizes)

    @property
    def num_tensors(self) -> int:
        return len(self.tensor_sizes)


def workload(index: int) -> Workload:
    if index == 0:
        return Workload("cfg0_resnet20_sign_w4", 4, resnet_cifar_sizes(3, 10), SIGN, 10, avg_period_paper=5)
    if index == 1:
        return Workload("cfg1_resnet56_sign_w8_wd", 8, resnet_cifar_sizes(9, 100), SIGN, 200, weight_decay=1e-4,
                        outlier_per_65536=655, outlier_mult=50.0)
    if index == 2:
        return Workload("cfg2_resnet50_sign_w16", 16, resnet50_sizes(), SIGN, 100)
    if index == 3:
        return Workload("cfg3_resnet50_topk1pct_w8", 8, resnet50_sizes(), TOPK, 100, outlier_per_65536=66,
                        outlier_mult=100.0)
    if index == 4:
        return Workload("cfg4_encoder110m_sign_w32", 32, encoder_sizes(), SIGN, 50, log10_scale_lo=-5.0,
                        log10_scale_hi=-2.0)
    raise ValueError("workload index must be 0..4")


NUM_WORKLOADS = 5
