"""AlexNet-shaped streamlined W1A2 chain on the CPU oracle (TEST INFRASTRUCTURE ONLY).

Section 4.2 / Table 3 of the paper: conv1 and fc8 are 8-bit layers, every other
matrix layer is W1A2 followed by the per-channel threshold activation; 3x3
stride-2 max-pools follow conv1, conv2 and conv5 and act on the integer codes.
Each layer is evaluated by its plain definition (direct convolution / integer
matrix product, then T(x, t), then max-pool); no lowering is used here.

The network description is passed in by the caller (any object with
``image``, ``layers``, ``weights``, ``thr``); nothing is imported from the CUDA
package.  Every intermediate tensor is returned so that a mismatch can be
localised to the layer that produced it.
"""
import numpy as np

from . import oracle as orc


def forward(net, keep_intermediates: bool = True):
    """Returns (logits int64 [B][n_classes], {layer name: codes after that layer})."""
    x = np.ascontiguousarray(net.image, dtype=np.int32)     # [B][H][W][C]
    inter = {}
    for L in net.layers:
        Wt = net.weights[L.name]
        thr = net.thr.get(L.name)
        if L.kind == "conv":
            y = orc.qconv(x, Wt, thr, L.stride, L.pad)
            if L.pool:
                y = orc.maxpool(y, 3, 2)
        else:
            if x.ndim == 4:                                  # flatten in (h, w, c) order
                x = x.reshape(x.shape[0], -1)
            y = orc.qgemm(Wt, x, thr)                        # [OC][B]
            y = np.ascontiguousarray(y.T)                    # -> [B][OC]
        if keep_intermediates:
            inter[L.name] = y
        x = y
    return x, inter
