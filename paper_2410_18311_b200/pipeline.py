"""Buffer management around the C-ABI calls for one model: per-layer core sets, compacted
weights and workspaces, allocated once with torch and reused.  No arithmetic here: selection,
compaction and decoding all run in the library's kernels."""
from __future__ import annotations

import torch

from . import binding as B
from .workloads import Config


class CoreSparseStack:
    """Core-sparse FFN stack of `cfg.L` layers (Section 4.2): `prefill()` fixes each layer's
    sentence-wise core set from its pre-fill activations and compacts the weights;
    `decode()` then pushes one token through all layers in one launch."""

    def __init__(self, cfg: Config, device="cuda", alpha=None, beta=None):
        self.cfg = cfg
        self.alpha = cfg.alpha if alpha is None else alpha
        self.beta = cfg.beta if beta is None else beta
        self.kind = B.FFN_RELU_GATED if cfg.gated else B.FFN_RELU
        self.K = B.coreinfer_count(self.beta, cfg.d_ff)
        dt, d, K, L = cfg.torch_dtype, cfg.d_model, self.K, cfg.L
        new = lambda *s, dtype=dt: torch.empty(s, dtype=dtype, device=device)
        self.core_idx = [new(K, dtype=torch.int32) for _ in range(L)]
        self.w_up_c = [new(K, d) for _ in range(L)]
        self.w_gate_c = [new(K, d) if cfg.gated else None for _ in range(L)]
        self.w_downT_c = [new(K, d) for _ in range(L)]
        self.select_ws = None
        self._side = None               # side stream and events of prefill(), created on first use
        self._events = None
        self.stack_ws = new(B.coreinfer_ffn_decode_stack_workspace_bytes(L, 1, d, K), dtype=torch.uint8)
        self.layer_ws = new(B.coreinfer_ffn_decode_workspace_bytes(B.MAX_BATCH, d, K), dtype=torch.uint8)
        self.layers = B.make_layers([(self.w_up_c[l], self.w_gate_c[l], self.w_downT_c[l], None, None)
                                     for l in range(L)])

    # kernels launched by one prefill() per layer / one decode() call, for launch accounting
    SELECT_KERNELS_PER_LAYER = 3
    COMPACT_KERNELS_PER_LAYER = 2
    DECODE_KERNELS_PER_TOKEN = 1

    def compacted_bytes_per_token(self) -> int:
        c = self.cfg
        return c.L * c.n_mat * self.K * c.d_model * c.esize

    def select_layer(self, l: int, act: torch.Tensor, counts_out=None, stream=None):
        need = B.coreinfer_select_workspace_bytes(act.shape[0], act.shape[1])
        if self.select_ws is None or self.select_ws.numel() < need:
            self.select_ws = torch.empty(need, dtype=torch.uint8, device=act.device)
        B.coreinfer_select_core(act, self.alpha, self.beta, self.core_idx[l], counts_out, self.select_ws, stream)

    def compact_layer(self, l: int, w_up, w_gate, w_down, stream=None):
        B.coreinfer_compact(w_up, w_gate, w_down, None, self.core_idx[l], self.K, self.w_up_c[l],
                            self.w_gate_c[l], self.w_downT_c[l], None, stream)

    def prefill(self, acts, weights, stream=None, overlap=True):
        """acts[l]: [T, d_ff] fp32 activations of layer l; weights[l] = (w_up, w_gate | None, w_down).

        Selection is a chain of small latency-bound kernels, compaction is bandwidth-bound: with
        `overlap` the compaction of layer l runs on a side stream while `stream` goes on with the
        selection of layer l + 1.  On return `stream` has been made to wait for the side stream."""
        main = torch.cuda.current_stream() if stream is None else stream
        if not overlap:
            for l in range(self.cfg.L):
                self.select_layer(l, acts[l], None, main)
                self.compact_layer(l, *weights[l], stream=main)
            return
        if self._side is None:
            self._side = torch.cuda.Stream(device=self.core_idx[0].device)
            self._events = [torch.cuda.Event() for _ in range(self.cfg.L + 2)]
        side, ev = self._side, self._events
        ev[-2].record(main)                 # earlier work on `stream` may still read the compacted buffers
        side.wait_event(ev[-2])
        for l in range(self.cfg.L):
            self.select_layer(l, acts[l], None, main)
            ev[l].record(main)
            side.wait_event(ev[l])
            self.compact_layer(l, *weights[l], stream=side)
        ev[-1].record(side)
        main.wait_event(ev[-1])

    def decode(self, x0, y_last, y_layers=None, x_layers=None, stream=None):
        """x0 [1, d] -> y_last [1, d] fp32 (FFN output of the last layer)."""
        B.coreinfer_ffn_decode_stack(self.layers, x0, self.kind, y_last, y_layers, x_layers, self.stack_ws, stream)

    def decode_layer(self, l: int, x, y, stream=None):
        """One layer, any batch 1..8."""
        B.coreinfer_ffn_decode(x, self.kind, self.w_up_c[l], self.w_gate_c[l], self.w_downT_c[l], None, None,
                               y, self.layer_ws, stream)

    def check(self, stream=None):
        B.coreinfer_workspace_status(self.stack_ws, stream)
