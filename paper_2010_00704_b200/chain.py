"""Sequencing helper: a chain of fused binary convolutions with device-resident packed activations.

Holds the packed weights, thresholds and the ping-pong activation buffers on the device
and enqueues, through the C ABI, one ``bcnn_pack`` followed by one
``bcnn_conv2d_b1_fused`` per layer (``bcnn_stem_fused`` replaces the pack and the first layer when the
shapes are the stem's: 4 real channels x 8 replicas, 1x1 to 32 channels).  It contains no arithmetic of its own.  The launch
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
                 device="cuda", fuse_stem=None, prepare_weights=None):
        """layers: sequence of ConvLayer; w_bits_list[i]: uint8 numpy [C_out, k, k, C_in/8];
        thr_list[i]: int32 numpy [C_out].  real_input_shape = (H, W, C_real) enables the pack
        stage (fp32 NHWC input, optional per-channel bias, replication factor).
        keep_all keeps one output buffer per layer (for checking) instead of two ping-pong buffers.
        fuse_stem: run pack + first layer as one ``bcnn_stem_fused`` call (the packed input is then never
        written); default: whenever the shapes allow it and keep_all is off.
        prepare_weights: expand the weights of wide / long-K layers once (``bcnn_prepare_weights``) and run those layers
        through ``bcnn_conv2d_b1_prepared``; default: with the AUTO engine."""
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
        self.layers_graph = None
        can_fuse = (real_input_shape is not None and real_input_shape[2] == 4 and replicate == 8
                    and (l0.k, l0.stride, l0.pad, l0.C_in, l0.C_out) == (1, 1, 0, 32, 32)
                    and engine == binding.ENGINE_AUTO)
        self.fuse_stem = (can_fuse and not keep_all) if fuse_stem is None else bool(fuse_stem)
        if self.fuse_stem and not can_fuse:
            raise ValueError("fuse_stem needs a 4-channel real input replicated 8x and a first 1x1 layer 32 -> 32")
        self.launches_per_run = len(self.layers) + (1 if real_input_shape is not None and not self.fuse_stem else 0)
        # wide layers / long K: the layer's weights are expanded once, here, into a buffer this object owns, and the
        # *_prepared call streams them by TMA (bit-identical results); everything else takes the plain fused call
        self.prepared = [None] * len(self.layers)
        if prepare_weights is None:
            prepare_weights = engine == binding.ENGINE_AUTO
        if prepare_weights:
            for i, l in enumerate(self.layers):
                if binding.bcnn_prepared_preferred(self.batch, l.H, l.W, l.C_in, l.C_out, l.k, l.k, l.stride, l.pad):
                    buf = torch.empty(binding.bcnn_prepared_weights_bytes(l.C_out, l.K), dtype=torch.uint8, device=self.device)
                    binding.bcnn_prepare_weights(self.w[i], buf, l.C_out, l.K)
                    self.prepared[i] = buf
            torch.cuda.synchronize()

    def enqueue_pack(self, x_real):
        H, W, C = self.real_input_shape
        if self.fuse_stem:
            binding.bcnn_stem_fused(x_real, self.bias, self.w[0], self.thr[0], self.outs[0], self.batch, H, W, C,
                                    self.replicate, self.layers[0].C_out)
        else:
            binding.bcnn_pack(x_real, self.bias, self.in_bits, self.batch, H, W, C, self.replicate)

    def enqueue_layer(self, i: int, cur):
        """Enqueue layer i (input ``cur``, output ``self.outs[i]``): the prepared call where its weights were prepared,
        else the plain fused call."""
        l, o = self.layers[i], self.outs[i]
        if self.prepared[i] is not None:
            binding.bcnn_conv2d_b1_prepared(cur, self.prepared[i], self.thr[i], o, self.batch, l.H, l.W, l.C_in, l.C_out,
                                            l.k, l.k, l.stride, l.pad)
        else:
            binding.bcnn_conv2d_b1_fused(cur, self.w[i], self.thr[i], o, self.batch, l.H, l.W, l.C_in, l.C_out, l.k, l.k,
                                         l.stride, l.pad, engine=self.engine)
        return o

    def engine_name(self, i: int) -> str:
        """Name of the engine layer i runs on."""
        l = self.layers[i]
        if i == 0 and self.fuse_stem:
            return "stem"
        if self.prepared[i] is not None:
            return "tc_pre"
        if self.engine != binding.ENGINE_AUTO:
            return {v: k for k, v in binding.ENGINES.items()}[self.engine]
        return binding.bcnn_auto_engine(self.batch, l.H, l.W, l.C_in, l.C_out, l.k, l.k, l.stride, l.pad)

    def enqueue(self, include_pack: bool = True):
        """Enqueue the whole sequence on the current stream; returns the last layer's packed output."""
        if self.x_real is not None and include_pack:
            self.enqueue_pack(self.x_real)
        cur = self.in_bits
        for i, (l, w, t, o) in enumerate(zip(self.layers, self.w, self.thr, self.outs)):
            if i == 0 and self.fuse_stem:        # done by enqueue_pack
                cur = o
                continue
            cur = self.enqueue_layer(i, cur)
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
        if self.x_real is not None:
            # the layers alone, for the host-input pipeline below (its pack stage alternates input buffers)
            gl = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gl):
                self.enqueue(include_pack=False)
            self.layers_graph = gl
        return g

    def run_from_host(self, x_host: torch.Tensor, out_host: torch.Tensor):
        """One step from a pinned fp32 host tensor to a pinned host copy of the last layer's packed output.

        Double-buffered: the host-to-device copy of this call's input runs on a copy stream and overlaps
        the kernels of the previous call (which read the other input buffer).  Everything is enqueued
        asynchronously; synchronise the device before reading ``out_host``."""
        if not hasattr(self, "_pipe"):
            self._pipe = {"stream": torch.cuda.Stream(), "bufs": [self.x_real, torch.empty_like(self.x_real)],
                          "copied": [torch.cuda.Event(), torch.cuda.Event()],
                          "consumed": [torch.cuda.Event(), torch.cuda.Event()], "n": 0}
            for ev in self._pipe["consumed"]:
                ev.record()
        pp = self._pipe
        b = pp["n"] & 1
        pp["n"] += 1
        main = torch.cuda.current_stream()
        with torch.cuda.stream(pp["stream"]):
            pp["stream"].wait_event(pp["consumed"][b])      # the pack that last read this buffer is done
            pp["bufs"][b].copy_(x_host, non_blocking=True)
            pp["copied"][b].record()
        main.wait_event(pp["copied"][b])
        self.enqueue_pack(pp["bufs"][b])
        pp["consumed"][b].record()
        if getattr(self, "layers_graph", None) is not None:
            self.layers_graph.replay()
        else:
            self.enqueue(include_pack=False)
        out_host.copy_(self.outs[-1], non_blocking=True)
        return out_host

    def run(self):
        if self.graph is not None:
            self.graph.replay()
        else:
            self.enqueue()
        return self.outs[-1]
