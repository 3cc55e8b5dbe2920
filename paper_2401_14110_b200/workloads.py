"""Layer shape lists and a forward harness for the benchmark configurations.

The hot path is the LBA contraction; this module only says which contractions a network consists of
(standard ResNet-18/50 and BERT-base shapes) and strings them together with plain PyTorch glue (ReLU,
max-pool, residual add, global average pool, re-quantisation to E4M3) so that every contraction sees
inputs with the value distribution of a real forward pass.  BatchNorm at fresh-initialised evaluation
state is the identity and is left out.  Weights are He-normal, quantised per output channel; activations
are quantised per tensor before every convolution and the final linear layer.
"""
from dataclasses import dataclass
from typing import List, Optional

import torch
import torch.nn.functional as F

from . import synth


@dataclass
class ConvSpec:
    name: str
    c_in: int
    c_out: int
    k: int
    stride: int
    pad: int
    h_in: int          # input height = width
    src: str           # name of the tensor it reads ("image", or a block-level activation)

    @property
    def h_out(self):
        return (self.h_in + 2 * self.pad - self.k) // self.stride + 1

    def gemm_shape(self, batch):
        """(M, N, K) of the implicit GEMM."""
        return batch * self.h_out * self.h_out, self.c_out, self.k * self.k * self.c_in

    def macs(self, batch):
        m, n, k = self.gemm_shape(batch)
        return m * n * k


def resnet18_convs() -> List[ConvSpec]:
    """The 20 convolutions of the standard ResNet-18 at 224x224 input (the 512->1000 linear layer is separate)."""
    specs = [ConvSpec("conv1", 3, 64, 7, 2, 3, 224, "image")]
    h, c = 56, 64
    for stage, (c_out, stride) in enumerate([(64, 1), (128, 2), (256, 2), (512, 2)], start=1):
        for block in range(2):
            s = stride if block == 0 else 1
            cin = c if block == 0 else c_out
            hin = h if block == 0 else h // stride
            specs.append(ConvSpec(f"layer{stage}.{block}.conv1", cin, c_out, 3, s, 1, hin, "block_in"))
            specs.append(ConvSpec(f"layer{stage}.{block}.conv2", c_out, c_out, 3, 1, 1, hin // s, "mid"))
            if block == 0 and (s != 1 or cin != c_out):
                specs.append(ConvSpec(f"layer{stage}.{block}.downsample", cin, c_out, 1, s, 0, hin, "block_in"))
        h, c = h // stride, c_out
    return specs


def resnet50_convs() -> List[ConvSpec]:
    """The 53 convolutions of the standard ResNet-50 (stride on the 3x3, as in torchvision)."""
    specs = [ConvSpec("conv1", 3, 64, 7, 2, 3, 224, "image")]
    h, c = 56, 64
    for stage, (width, blocks, stride) in enumerate([(64, 3, 1), (128, 4, 2), (256, 6, 2), (512, 3, 2)], start=1):
        c_out = width * 4
        for block in range(blocks):
            s = stride if block == 0 else 1
            cin = c if block == 0 else c_out
            hin = h if block == 0 else h // stride
            specs.append(ConvSpec(f"layer{stage}.{block}.conv1", cin, width, 1, 1, 0, hin, "block_in"))
            specs.append(ConvSpec(f"layer{stage}.{block}.conv2", width, width, 3, s, 1, hin, "mid"))
            specs.append(ConvSpec(f"layer{stage}.{block}.conv3", width, c_out, 1, 1, 0, hin // s, "mid2"))
            if block == 0:
                specs.append(ConvSpec(f"layer{stage}.{block}.downsample", cin, c_out, 1, s, 0, hin, "block_in"))
        h, c = h // stride, c_out
    return specs


def bert_base_linears(tokens: int = 4096):
    """(name, M, N, K) of the linear layers of one BERT-base encoder layer."""
    return [("query", tokens, 768, 768), ("key", tokens, 768, 768), ("value", tokens, 768, 768),
            ("attn_out", tokens, 768, 768), ("ffn_in", tokens, 3072, 768), ("ffn_out", tokens, 768, 3072)]


@dataclass
class LbaCall:
    """One contraction of a network, with its operands resident on a device (or pinned on the host)."""
    name: str
    kind: str                      # "conv" or "gemm"
    x: torch.Tensor                # conv: [B][H][W][Cin] codes; gemm: [M][K] codes
    w: torch.Tensor                # conv: [Cout][KH][KW][Cin] codes; gemm: [N][K] codes
    sx: torch.Tensor
    sw: torch.Tensor
    stride: tuple = (1, 1)
    pad: tuple = (0, 0)
    out: Optional[torch.Tensor] = None

    @property
    def gemm_shape(self):
        if self.kind == "bgemm":        # per problem; macs counts all of them
            return self.x.shape[1], self.w.shape[1], self.x.shape[2]
        if self.kind in ("gemm", "ste"):   # "ste": the mask re-computation pass of the same GEMM
            return self.x.shape[0], self.w.shape[0], self.x.shape[1]
        b, h, wd, cin = self.x.shape
        cout, kh, kw, _ = self.w.shape
        ho = (h + 2 * self.pad[0] - kh) // self.stride[0] + 1
        wo = (wd + 2 * self.pad[1] - kw) // self.stride[1] + 1
        return b * ho * wo, cout, kh * kw * cin

    @property
    def macs(self):
        m, n, k = self.gemm_shape
        return m * n * k * (self.x.shape[0] if self.kind == "bgemm" else 1)


def _quant_act(t_nhwc: torch.Tensor, wa_format: str = "e4m3"):
    if wa_format == "m4e3":
        codes, scale = synth.quantise_m4e3_per_tensor(t_nhwc)
        return codes.to(t_nhwc.device).contiguous(), scale.to(t_nhwc.device)
    codes, scale = synth.quantise_per_tensor(t_nhwc)
    return codes.contiguous(), scale.to(t_nhwc.device)


def _quant_weight(w: torch.Tensor, wa_format: str = "e4m3"):
    if wa_format == "m4e3":      # the paper's flex-bias: one power-of-two scale per tensor (Sec. 3.1)
        return synth.quantise_m4e3_per_tensor(w)
    return synth.quantise_per_channel(w)


def build_resnet_calls(arch: str, batch: int, config: int, device, conv_fn, gemm_fn, image_hw: int = 224,
                       wa_format: str = "e4m3"):
    """Run one forward pass of ResNet-18/50 through ``conv_fn``/``gemm_fn`` and record every LBA call.

    conv_fn(x, w, sx, sw, stride, pad) -> float32 NHWC output; gemm_fn(a, b, sa, sb) -> float32 [M][N].
    ``wa_format``: "e4m3" (OCP E4M3 bytes, per-tensor activation and per-channel weight scales) or "m4e3" (the paper's
    own W/A bytes with one power-of-two flex-bias scale per tensor, Sec. 3.1).
    Returns the list of LbaCall (operands on ``device``) and the logits.
    """
    specs = {"resnet18": resnet18_convs, "resnet50": resnet50_convs}[arch]()
    # the recorded calls take their spatial sizes from the tensors themselves, so a smaller image
    # (used by the tests) needs no change to the shape list
    calls: List[LbaCall] = []
    index = 0

    def weights(spec):
        nonlocal index
        index += 1
        w = synth.he_normal((spec.c_out, spec.k, spec.k, spec.c_in), spec.k * spec.k * spec.c_in,
                            synth.seed_for(config, 100 + index))
        codes, scale = _quant_weight(w, wa_format)
        return codes.to(device), scale.to(device)

    def run_conv(spec, act):
        xc, sx = _quant_act(act, wa_format)
        wc, sw = weights(spec)
        call = LbaCall(spec.name, "conv", xc, wc, sx, sw, (spec.stride, spec.stride), (spec.pad, spec.pad))
        calls.append(call)
        return conv_fn(xc, wc, sx, sw, call.stride, call.pad)

    image = synth.gaussian((batch, image_hw, image_hw, 3), synth.seed_for(config, 0)).to(device)
    it = iter(specs)
    act = run_conv(next(it), image).relu_()
    act = F.max_pool2d(act.permute(0, 3, 1, 2), 3, 2, 1).permute(0, 2, 3, 1).contiguous()
    per_block = 2 if arch == "resnet18" else 3
    pending = list(it)
    i = 0
    while i < len(pending):
        block_in = act
        y = block_in
        for j in range(per_block):
            y = run_conv(pending[i + j], y)
            if j + 1 < per_block:
                y = y.relu_()
        i += per_block
        identity = block_in
        if i < len(pending) and pending[i].name.endswith("downsample"):
            identity = run_conv(pending[i], block_in)
            i += 1
        act = (y + identity).relu_()
    pooled = act.mean(dim=(1, 2))                                  # [B][C]
    c = pooled.shape[1]
    fc_w = synth.gaussian((1000, c), synth.seed_for(config, 99), std=float((1.0 / c) ** 0.5))
    wc, sw = _quant_weight(fc_w, wa_format)
    xc, sx = _quant_act(pooled, wa_format)
    call = LbaCall("fc", "gemm", xc, wc.to(device), sx, sw.to(device))
    calls.append(call)
    logits = gemm_fn(xc, call.w, sx, call.sw)
    return calls, logits


def build_bert_calls(tokens: int, config: int, device):
    """Operands of the six linear layers of one BERT-base encoder layer (Gaussian activations with a seeded
    1 % of outlier feature columns x20, N(0, 0.02^2) weights)."""
    calls = []
    for idx, (name, m, n, k) in enumerate(bert_base_linears(tokens)):
        a = synth.with_outlier_columns(synth.gaussian((m, k), synth.seed_for(config, 10 * idx)),
                                       synth.seed_for(config, 10 * idx + 1))
        w = synth.gaussian((n, k), synth.seed_for(config, 10 * idx + 2), std=0.02)
        ac, sa = synth.quantise_per_tensor(a)
        wc, sw = synth.quantise_per_channel(w)
        calls.append(LbaCall(name, "gemm", ac.to(device), wc.to(device), sa.to(device), sw.to(device)))
    return calls
