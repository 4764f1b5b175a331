"""Tensor shapes of the synthetic training jobs and the block cutter.

Only shapes: no weights, no data, none of the aggregation arithmetic.  Tensors
are listed in FORWARD layer order; backward produces them in reverse.  The
architectures are the published ones (AlexNet, VGG-16, ResNet-50, BERT) plus a
3-layer LSTM language model sized to a 33278-word vocabulary with a 400-wide
embedding and 800-wide hidden layers (24,240,478 parameters).
"""
from __future__ import annotations

from dataclasses import dataclass
from math import prod

BLOCK_ELEMS = 1 << 20   # "1M-elem blocks" read as 2**20


@dataclass(frozen=True)
class Tensor:
    name: str
    shape: tuple
    layer: int          # forward position (0 = first layer)
    row_sparse: bool = False

    @property
    def nelem(self) -> int:
        return prod(self.shape)


@dataclass(frozen=True)
class Block:
    block: int          # dense block id within the job
    tensor: int         # index into the job's tensor list
    offset: int         # element offset inside the tensor
    nelem: int
    layer: int
    job_offset: int     # element offset inside the job's flat parameter vector


def alexnet() -> list[Tensor]:
    spec = [("conv1", (64, 3, 11, 11)), ("conv2", (192, 64, 5, 5)), ("conv3", (384, 192, 3, 3)),
            ("conv4", (256, 384, 3, 3)), ("conv5", (256, 256, 3, 3)),
            ("fc6", (4096, 9216)), ("fc7", (4096, 4096)), ("fc8", (1000, 4096))]
    out = []
    for i, (n, s) in enumerate(spec):
        out += [Tensor(n + ".weight", s, i), Tensor(n + ".bias", (s[0],), i)]
    return out


def vgg16() -> list[Tensor]:
    cfg = [(64, 3), (64, 64), (128, 64), (128, 128), (256, 128), (256, 256), (256, 256),
           (512, 256), (512, 512), (512, 512), (512, 512), (512, 512), (512, 512)]
    out = []
    for i, (co, ci) in enumerate(cfg):
        out += [Tensor("conv%d.weight" % (i + 1), (co, ci, 3, 3), i), Tensor("conv%d.bias" % (i + 1), (co,), i)]
    for j, (o, k) in enumerate([(4096, 25088), (4096, 4096), (1000, 4096)]):
        out += [Tensor("fc%d.weight" % (6 + j), (o, k), 13 + j), Tensor("fc%d.bias" % (6 + j), (o,), 13 + j)]
    return out


def resnet50() -> list[Tensor]:
    out: list[Tensor] = []
    layer = 0

    def conv_bn(name, co, ci, k):
        nonlocal layer
        out.append(Tensor(name + ".conv.weight", (co, ci, k, k), layer))
        out.append(Tensor(name + ".bn.weight", (co,), layer))
        out.append(Tensor(name + ".bn.bias", (co,), layer))
        layer += 1

    conv_bn("stem", 64, 3, 7)
    cin = 64
    for s, (nblk, width) in enumerate([(3, 64), (4, 128), (6, 256), (3, 512)]):
        for b in range(nblk):
            name = "layer%d.%d" % (s + 1, b)
            conv_bn(name + ".a", width, cin, 1)
            conv_bn(name + ".b", width, width, 3)
            conv_bn(name + ".c", width * 4, width, 1)
            if b == 0:
                conv_bn(name + ".down", width * 4, cin, 1)
            cin = width * 4
    out.append(Tensor("fc.weight", (1000, 2048), layer))
    out.append(Tensor("fc.bias", (1000,), layer))
    return out


def awd_lm() -> list[Tensor]:
    vocab, emb, hid = 33278, 400, 800
    out = [Tensor("encoder.weight", (vocab, emb), 0, row_sparse=True)]
    dims = [(emb, hid), (hid, hid), (hid, emb)]
    for l, (i, h) in enumerate(dims):
        out += [Tensor("rnn%d.weight_ih" % l, (4 * h, i), 1 + l), Tensor("rnn%d.weight_hh" % l, (4 * h, h), 1 + l),
                Tensor("rnn%d.bias_ih" % l, (4 * h,), 1 + l), Tensor("rnn%d.bias_hh" % l, (4 * h,), 1 + l)]
    out.append(Tensor("decoder.bias", (vocab,), 4))   # decoder weight is tied to the encoder
    return out


def bert(layers: int, hidden: int, ffn: int, classifier: int = 0,
         vocab: int = 30522, positions: int = 512) -> list[Tensor]:
    out = [Tensor("emb.word", (vocab, hidden), 0), Tensor("emb.position", (positions, hidden), 0),
           Tensor("emb.type", (2, hidden), 0), Tensor("emb.ln.weight", (hidden,), 0),
           Tensor("emb.ln.bias", (hidden,), 0)]
    for l in range(layers):
        n = "layer%d." % l
        for a in ("q", "k", "v", "o"):
            out += [Tensor(n + a + ".weight", (hidden, hidden), 1 + l), Tensor(n + a + ".bias", (hidden,), 1 + l)]
        out += [Tensor(n + "ln1.weight", (hidden,), 1 + l), Tensor(n + "ln1.bias", (hidden,), 1 + l)]
        out += [Tensor(n + "ffn1.weight", (ffn, hidden), 1 + l), Tensor(n + "ffn1.bias", (ffn,), 1 + l)]
        out += [Tensor(n + "ffn2.weight", (hidden, ffn), 1 + l), Tensor(n + "ffn2.bias", (hidden,), 1 + l)]
        out += [Tensor(n + "ln2.weight", (hidden,), 1 + l), Tensor(n + "ln2.bias", (hidden,), 1 + l)]
    out += [Tensor("pooler.weight", (hidden, hidden), layers + 1), Tensor("pooler.bias", (hidden,), layers + 1)]
    if classifier:
        out += [Tensor("cls.weight", (classifier, hidden), layers + 2), Tensor("cls.bias", (classifier,), layers + 2)]
    return out


def bert_base() -> list[Tensor]:
    return bert(12, 768, 3072)


def bert_large() -> list[Tensor]:
    return bert(24, 1024, 4096, classifier=2)


MODELS = {"alexnet": alexnet, "vgg16": vgg16, "resnet50": resnet50, "awd_lm": awd_lm,
          "bert_base": bert_base, "bert_large": bert_large}


def cut_blocks(tensors: list[Tensor], max_elems: int = BLOCK_ELEMS,
               keep_whole=lambda t: False) -> list[Block]:
    """A tensor of n elements becomes ceil(n / max_elems) blocks, all full but
    the last; tensors for which keep_whole(t) holds stay one block.  Row-sparse
    tensors (embedding tables) are cut at row boundaries, so that a block is a
    whole number of rows (the largest such block that fits max_elems)."""
    blocks: list[Block] = []
    job_off = 0
    for ti, t in enumerate(tensors):
        n = t.nelem
        step = n if keep_whole(t) else max_elems
        if t.row_sparse and not keep_whole(t):
            row_len = n // t.shape[0]
            step = max(1, max_elems // row_len) * row_len
        off = 0
        while off < n:
            m = min(step, n - off)
            blocks.append(Block(len(blocks), ti, off, m, t.layer, job_off + off))
            off += m
        job_off += n
    return blocks


def num_params(tensors: list[Tensor]) -> int:
    return sum(t.nelem for t in tensors)
