"""Oracle of the ResNet-50-shaped CNN (TEST INFRASTRUCTURE): a composition, in the order of the
network, of the fp64 routines of nm_oracle.c -- direct convolution (Section 3.1), ReLU as a
2-segment PWL table (Section 3: ReLU is already piecewise linear), plain max for the max-pool,
mean for the average pool, a linear operator for the classifier."""
from __future__ import annotations

import numpy as np

from . import Table, conv2d_nhwc, maxpool_nhwc, avgpool_nhwc, linear, pwl_eval

STAGE_BLOCKS = (3, 4, 6, 3)


def resnet50(x, convs, fc_w, fc_b, relu: Table, collect=None, blocks=STAGE_BLOCKS):
    """x [N,H,W,3]; convs: dicts with 'w', 'b', 'spec' = (Cin, Cout, k, stride, pad) in network
    order (conv1; per block conv_a, conv_b, conv_c, and the projection in a stage's first block): 53 for
    ResNet-50.  `blocks`: bottleneck blocks per stage, for the depth variants Section 5 compares (the widths
    are those of the weights).  Returns logits [N, classes].  `collect`, if a list, receives the output of
    every block."""
    it = iter(convs)

    def conv(inp, c, table, residual=None):
        _, _, _, stride, pad = c["spec"]
        return conv2d_nhwc(inp, c["w"], stride, pad, c["b"], residual, table)

    y = conv(x, next(it), relu)
    y = maxpool_nhwc(y, 3, 2, 1)
    for st, nb in enumerate(blocks):
        for b in range(nb):
            ca, cb, cc = next(it), next(it), next(it)
            t = conv(y, ca, relu)
            t = conv(t, cb, relu)
            shortcut = conv(y, next(it), None) if b == 0 else y
            z = conv(t, cc, None, residual=shortcut)        # conv + bias + shortcut
            y = pwl_eval(relu, z)[0]                        # ReLU after the add
            if collect is not None:
                collect.append(y)
    assert next(it, None) is None, "more convolutions than the block counts use"
    pooled = avgpool_nhwc(y)
    return linear(pooled, fc_w, fc_b)
