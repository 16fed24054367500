"""Sequencing helper: a chain of fused binary convolutions with device-resident packed activations.

Holds the packed weights, thresholds and the ping-pong activation buffers on the device
and enqueues, through the C ABI, one ``bcnn_pack`` followed by one
``bcnn_conv2d_b1_fused`` per layer.  It contains no arithmetic of its own.  The launch
sequence can be captured once into a CUDA graph and replayed.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding
from .workloads import ConvLayer


class FusedChain:
    def __init__(self, layers, batch: int, w_bits_list, thr_list, real_input_shape=None, bias=None,
                 replicate: int = 1, engine: int = binding.ENGINE_AUTO, keep_all: bool = False,
                 device="cuda"):
        """layers: sequence of ConvLayer; w_bits_list[i]: uint8 numpy [C_out, k, k, C_in/8];
        thr_list[i]: int32 numpy [C_out].  real_input_shape = (H, W, C_real) enables the pack
        stage (fp32 NHWC input, optional per-channel bias, replication factor).
        keep_all keeps one output buffer per layer (for checking) instead of two ping-pong buffers."""
        self.layers = list(layers)
        self.batch = int(batch)
        self.engine = engine
        self.device = torch.device(device)
        self.w = [torch.from_numpy(np.ascontiguousarray(w)).to(self.device) for w in w_bits_list]
        self.thr = [torch.from_numpy(np.ascontiguousarray(t, dtype=np.int32)).to(self.device) for t in thr_list]
        l0 = self.layers[0]
        self.in_bits = torch.empty(self.batch * l0.H * l0.W * l0.C_in // 8, dtype=torch.uint8, device=self.device)
        self.real_input_shape = real_input_shape
        self.replicate = replicate
        self.bias = None if bias is None else torch.from_numpy(np.ascontiguousarray(bias, dtype=np.float32)).to(self.device)
        self.x_real = None
        if real_input_shape is not None:
            H, W, C = real_input_shape
            assert (H, W, C * replicate) == (l0.H, l0.W, l0.C_in)
            self.x_real = torch.empty(self.batch * H * W * C, dtype=torch.float32, device=self.device)
        sizes = [l.out_bits_bytes(self.batch) for l in self.layers]
        if keep_all:
            self.outs = [torch.empty(s, dtype=torch.uint8, device=self.device) for s in sizes]
        else:
            ping = torch.empty(max(sizes[0::2]), dtype=torch.uint8, device=self.device)
            pong = torch.empty(max(sizes[1::2]) if len(sizes) > 1 else 16, dtype=torch.uint8, device=self.device)
            self.outs = [(ping if i % 2 == 0 else pong)[:s] for i, s in enumerate(sizes)]
        self.graph = None
        self.launches_per_run = len(self.layers) + (1 if real_input_shape is not None else 0)

    def enqueue(self):
        """Enqueue the whole sequence on the current stream; returns the last layer's packed output."""
        if self.x_real is not None:
            H, W, C = self.real_input_shape
            binding.bcnn_pack(self.x_real, self.bias, self.in_bits, self.batch, H, W, C, self.replicate)
        cur = self.in_bits
        for l, w, t, o in zip(self.layers, self.w, self.thr, self.outs):
            binding.bcnn_conv2d_b1_fused(cur, w, t, o, self.batch, l.H, l.W, l.C_in, l.C_out, l.k, l.k,
                                         l.stride, l.pad, engine=self.engine)
            cur = o
        return cur

    def capture(self):
        """Record the sequence once into a CUDA graph (after a warm-up run on a side stream)."""
        s = torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s):
            self.enqueue()
        torch.cuda.current_stream().wait_stream(s)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            self.enqueue()
        self.graph = g
        return g

    def run(self):
        if self.graph is not None:
            self.graph.replay()
        else:
            self.enqueue()
        return self.outs[-1]
