"""AlexNet-shaped streamlined W1A2 inference as a sequence of C-ABI calls.

Section 4.2 / Table 3 of the paper: conv1 and fc8 are 8-bit layers, the other
matrix layers are W1A2 with per-channel threshold activations, 3x3 stride-2
max-pools follow conv1, conv2 and conv5.  This module only sequences the calls
(qnn_qconv, qnn_maxpool, qnn_qgemm) and owns the device buffers; all
arithmetic runs in the library's kernels.

``mode`` selects the operand format of the W1A2 layers' activations/weights:
  "tensor"     8-bit containers everywhere  (tcgen05 path for every layer)
  "bitserial"  bit planes for the W1A2 layers (bit-serial path; conv1 writes bit
               planes directly from its epilogue, fc7 writes 8-bit codes for fc8)
  "auto"       per layer, as Section 4.1 of the paper suggests choosing the engine
               by shape: 8-bit containers (tensor cores) for the convolutions,
               and, at batch <= 16, bit planes for the fully connected W1A2
               layers, whose packed weights are streamed once by the few-column
               bit-serial kernel; at larger batch the same as "tensor"
"""
import numpy as np
import torch

from . import binding as qb

BITPLANES, INT8 = qb.QNN_FMT_BITPLANES, qb.QNN_FMT_INT8


def _round_up(x, m):
    return (x + m - 1) // m * m


class AlexNetPlan:
    def __init__(self, net, B: int, mode: str = "auto", hw: int = 227):
        assert mode in ("tensor", "bitserial", "auto")
        self.B, self.mode, self.layers, self.hw = B, mode, list(net.layers), hw
        self.steps = []          # (kind, desc, tensors...)
        self.names = []
        H, C = hw, 3
        fmt_in = INT8            # the image is uint8, pixel pitch 3
        in_pitch = 3
        flat = None
        ws_bytes = 16
        n_layers = len(self.layers)
        def planes(L):
            if L.w_bits == 8:
                return False
            return mode == "bitserial" or (mode == "auto" and L.kind == "fc" and B <= 16)

        for li, L in enumerate(self.layers):
            fmt = BITPLANES if planes(L) else INT8
            assert fmt == fmt_in, "layer input format must match the producer's output format"
            # output format = what the next matrix layer consumes
            nxt = self.layers[li + 1] if li + 1 < n_layers else None
            out_fmt = BITPLANES if (nxt is not None and planes(nxt)) else INT8
            thr = net.thr.get(L.name)
            thr_d = torch.from_numpy(np.ascontiguousarray(thr)).cuda() if thr is not None else None
            Wl = np.asarray(net.weights[L.name])
            if L.kind == "conv":
                d = qb.qnn_conv_desc(B, H, H, C, in_pitch if fmt == INT8 else 0, L.OC, L.KH, L.KW,
                                     L.stride, L.pad, L.w_bits, L.a_bits, max(L.out_bits, 1),
                                     L.w_enc, qb.QNN_ENC_UNSIGNED, fmt, out_fmt, qb.QNN_PATH_AUTO)
                Wflat = qb.conv_weight_rows(d, Wl)
                Wp = qb.pack(qb.to_device_logical(Wflat, L.w_enc), L.w_bits, L.w_enc, fmt)
                out = torch.empty(qb.qnn_conv_out_bytes(d, thr is not None), dtype=torch.uint8, device="cuda")
                ws_bytes = max(ws_bytes, qb.qnn_conv_workspace_bytes(d))
                OH = qb.qnn_conv_out_h(d)
                self.steps.append(("conv", d, Wp, thr_d, out))
                self.names.append(L.name)
                H, C = OH, L.OC
                if L.pool:
                    pd = qb.qnn_pool_desc(B, H, H, C, 3, 2, L.out_bits, out_fmt)
                    PH = (H - 3) // 2 + 1
                    nbytes = (B * PH * PH * _round_up(C, 16) if out_fmt == INT8
                              else L.out_bits * B * PH * PH * ((C + 31) // 32) * 4)
                    pout = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
                    self.steps.append(("pool", pd, None, None, pout))
                    self.names.append(L.name + "_pool")
                    H = PH
                in_pitch = _round_up(C, 16)
                flat = H * H * C
                assert C % 32 == 0 or out_fmt == INT8
            else:
                K = flat
                out_bits = max(L.out_bits, 1)
                d = qb.gemm_desc(L.OC, B, K, L.w_bits, L.a_bits, out_bits, L.w_enc,
                                 qb.QNN_ENC_UNSIGNED, fmt, out_fmt)
                Wp = qb.pack(qb.to_device_logical(Wl.reshape(L.OC, K), L.w_enc), L.w_bits, L.w_enc, fmt)
                out = torch.empty(max(qb.qnn_gemm_out_bytes(d, thr is not None), 16),
                                  dtype=torch.uint8, device="cuda")
                self.steps.append(("fc", d, Wp, thr_d, out))
                self.names.append(L.name)
                flat = L.OC
            fmt_in = out_fmt
        self.workspace = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
        self.n_classes = self.layers[-1].OC

    def forward(self, image: torch.Tensor, stream=None):
        """image: uint8 device tensor [B][H][W][3].  Returns int32 logits [B][n_classes]
        (a view of the plan's last buffer).  Enqueues only; does not synchronise."""
        x = image
        for kind, d, Wp, thr, out in self.steps:
            if kind == "conv":
                qb.check(qb.qnn_qconv(d, Wp, x, thr, out, self.workspace, self.workspace.numel(), stream))
            elif kind == "pool":
                qb.check(qb.qnn_maxpool(d, x, out, stream))
            else:
                qb.check(qb.qnn_qgemm(d, Wp, x, thr, out, None, 0, stream))
            x = out
        return x[: self.B * self.n_classes * 4].view(torch.int32).view(self.B, self.n_classes)

    def capture(self, image: torch.Tensor):
        """Record one forward pass into a CUDA graph (the chain at small batch is bound by
        launch overhead, 16 kernels of a few microseconds each).  Returns (graph, logits):
        ``graph.replay()`` re-runs the chain on the current contents of ``image`` and
        refreshes ``logits`` in place.  One eager pass runs first so that every one-time
        set-up of the library happens outside the capture."""
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            self.forward(image)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            logits = self.forward(image)
        return graph, logits

    def intermediates(self):
        """{step name: (output buffer, descriptor kind, descriptor)} for tests."""
        return {n: (s[4], s[0], s[1]) for n, s in zip(self.names, self.steps)}

    def launches_per_forward(self) -> int:
        """Kernels one forward pass launches (counted by the library on a dry call)."""
        if getattr(self, "_launches", None) is None:
            img = torch.zeros(self.B, self.hw, self.hw, 3, dtype=torch.uint8, device="cuda")
            n0 = qb.qnn_launch_count()
            self.forward(img)
            torch.cuda.synchronize()
            self._launches = qb.qnn_launch_count() - n0
        return self._launches
