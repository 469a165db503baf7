"""Seeded synthetic inputs for the ResNet-50-shaped CNN workload (config 5).  Like nm_inputs, this
module holds no arithmetic of the forward pass: it draws images, He-normal convolution weights and
BatchNorm statistics, folds the (inference-time, constant) BatchNorm into each convolution's weight
and bias -- an offline re-parameterisation of the inputs, W' = W*g/sqrt(var+eps), b' = beta - mean*g/
sqrt(var+eps) -- rounds to fp16, and hands the same folded tensors to the oracle and to the CUDA library.

Stand-in for the ImageNet-class inputs and trained weights the paper evaluates with, which are not
available and are not reproduced; only the ResNet-50 layer shapes are used.

Draw order (numpy default_rng(seed)): images, then per convolution in network order its weight and
(when random_bn) gamma, beta, mean, var; last the FC weight and bias."""
from __future__ import annotations

import numpy as np

from nm_inputs import round_to

STAGE_BLOCKS = (3, 4, 6, 3)
STAGE_WIDTH = (64, 128, 256, 512)


def resnet_conv_specs(blocks=STAGE_BLOCKS, base_width=64):
    """(Cin, Cout, k, stride, pad) of the convolutions of a bottleneck ResNet in network order: conv1, then
    per block conv_a (1x1), conv_b (3x3, carries the stride), conv_c (1x1) and, in the first block of a stage,
    the 1x1 projection shortcut.  blocks: bottleneck blocks per stage; base_width: inner width of stage 1
    (stage s: base_width << s).  (3, 4, 6, 3) and 64 give ResNet-50's 53 convolutions."""
    specs = [(3, base_width, 7, 2, 3)]
    cin = base_width
    for st, nb in enumerate(blocks):
        width = base_width << st
        for b in range(nb):
            stride = 2 if (b == 0 and st > 0) else 1
            specs.append((cin, width, 1, 1, 0))
            specs.append((width, width, 3, stride, 1))
            specs.append((width, 4 * width, 1, 1, 0))
            if b == 0:
                specs.append((cin, 4 * width, 1, stride, 0))
            cin = 4 * width
    return specs


def resnet50_conv_specs():
    specs = resnet_conv_specs()
    assert len(specs) == 53
    return specs


def resnet50_inputs(batch, seed=0, random_bn=False, num_classes=1000, image=224, dtype="f16", blocks=STAGE_BLOCKS,
                    base_width=64):
    """Returns (x [batch,image,image,3] fp32 holding dtype-rounded values in [0,1),
    convs: list of dicts {w [Cout,k,k,Cin], b [Cout], spec}, fc_w [classes, 32 base_width], fc_b [classes]).
    blocks / base_width: the depth and width variants of the network (defaults: ResNet-50)."""
    rng = np.random.default_rng(seed)
    x = round_to(rng.random((batch, image, image, 3), dtype=np.float32), dtype)
    convs = []
    feat = 32 * base_width
    for (cin, cout, k, stride, pad) in resnet_conv_specs(blocks, base_width):
        fan_in = cin * k * k
        w = (np.sqrt(2.0 / fan_in) * rng.standard_normal((cout, k, k, cin), dtype=np.float32)).astype(np.float32)
        if random_bn:
            g = (1.0 + 0.1 * rng.standard_normal(cout)).astype(np.float32)
            beta = (0.1 * rng.standard_normal(cout)).astype(np.float32)
            mean = (0.1 * rng.standard_normal(cout)).astype(np.float32)
            var = rng.uniform(0.8, 1.25, cout).astype(np.float32)
            s = g / np.sqrt(var + np.float32(1e-5))
            w = w * s[:, None, None, None]
            b = (beta - mean * s).astype(np.float32)
        else:
            b = np.zeros(cout, np.float32)
        convs.append({"w": round_to(w, dtype), "b": b, "spec": (cin, cout, k, stride, pad)})
    fc_w = round_to((np.sqrt(1.0 / feat) * rng.standard_normal((num_classes, feat), dtype=np.float32)), dtype)
    fc_b = (0.01 * rng.standard_normal(num_classes)).astype(np.float32)
    return x, convs, fc_w, fc_b
