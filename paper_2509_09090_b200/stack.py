"""Call sequence of the 32-layer W4A4 linear stack for one observation (prefill, pruning between two layers,
single-token decode steps), issued through the C ABI. Argument marshalling only: every step runs in the
library's kernels. Used by the bench (timing) and by the parity tests (every output kept for comparison).

Data flow of a layer (attention, norms and residuals are not part of the W4A4 path, so stand-ins connect the
four linears): qkv = L_qkv(x) with the Hadamard rotation; o = L_o(V third of qkv); h = SwiGLU(L_gate(o), L_up(o));
d = L_down(h). Every layer takes the same token matrix x (the rows that survive the pruning from the prune
layer on) and writes its own d.
"""
from __future__ import annotations

from . import workloads as wl


class Stack:
    def __init__(self, torch, B, device, layers, rows=wl.ROWS, keep=128, k_attn=64, ring_radius=1, prune_after=2,
                 n_decode=7, keep_intermediates=False):
        """layers: list of dicts of packed weight handles with keys qkv, o, gate, up, down.
        keep_intermediates: give every layer (and decode step) its own qkv / o / h buffers instead of one shared
        set, so that each linear's input and output can be read back afterwards."""
        t = torch
        self.t, self.B, self.dev, self.layers = t, B, device, layers
        self.rows, self.keep, self.prune_after, self.n_decode = rows, keep, prune_after, n_decode
        self.rows_kept = rows - wl.N_VISUAL + keep
        H, F, Q = wl.HIDDEN, wl.FFN, wl.QKV
        nl = len(layers)
        f16, i32 = t.float16, t.int32
        ni = nl if keep_intermediates else 1
        self.qkv = t.empty(ni, rows, Q, dtype=f16, device=device)
        self.o = t.empty(ni, rows, H, dtype=f16, device=device)
        self.h = t.empty(ni, rows, F, dtype=f16, device=device)
        self.d = t.empty(nl, rows, H, dtype=f16, device=device)
        nd = n_decode * nl if keep_intermediates else 1
        self.qkv_dec = t.empty(nd, 1, Q, dtype=f16, device=device)
        self.o_dec = t.empty(nd, 1, H, dtype=f16, device=device)
        self.h_dec = t.empty(nd, 1, F, dtype=f16, device=device)
        self.d_dec = t.empty(n_decode, nl, 1, H, dtype=f16, device=device)
        self.row_index = t.empty(self.rows_kept, dtype=i32, device=device)   # the kept rows, as source rows of x
        self.kept = t.empty(1, rows, dtype=i32, device=device)
        self.nkept = t.empty(1, dtype=i32, device=device)
        self.prune_params = wl.prune_params(1, rows, wl.VISUAL_START, wl.N_VISUAL, wl.GRID, wl.GRID, 32, k_attn, keep,
                                            ring_radius=ring_radius)
        self.ws_bytes = B.sqap_quantize_linear_workspace_bytes(rows, Q, F)
        self.ws = t.empty(self.ws_bytes, dtype=t.uint8, device=device)
        self.keep_intermediates = keep_intermediates

    def _lin(self, x_ptr, m, ldx, w, w_up, out, rotate=False, row_index=None):
        B = self.B
        B.sqap_quantize_linear(x_ptr, m, ldx, row_index, B.SQAP_Q_ROTATE if rotate else 0, w, w_up, out, out.shape[-1],
                               B.SQAP_FP16, 0, self.ws, self.ws_bytes)

    def _layer(self, x, m, L, qkv, o, h, d, row_index=None):
        H = wl.HIDDEN
        self._lin(x.data_ptr(), m, H, L["qkv"], None, qkv, rotate=True, row_index=row_index)
        self._lin(qkv.data_ptr() + 2 * 2 * H, m, wl.QKV, L["o"], None, o)      # the V third of the fused output
        self._lin(o.data_ptr(), m, H, L["gate"], L["up"], h)
        self._lin(h.data_ptr(), m, wl.FFN, L["down"], None, d)

    def prefill(self, x, scores, centers):
        """x: fp16 [rows, HIDDEN]; scores: fp16 [1, 32, N_VISUAL]; centers: int32 [1, 2] (device tensors).
        From the prune layer on, the first linear of a layer reads the surviving rows of x in place, through the row
        list the criterion wrote (no gathered copy is made)."""
        for li, L in enumerate(self.layers):
            if li == self.prune_after:
                self.B.sqap_prune_select(self.prune_params, scores, centers, self.rows_kept, self.kept, self.nkept,
                                         self.row_index)
            pruned = li >= self.prune_after
            i = li if self.keep_intermediates else 0
            self._layer(x, self.rows_kept if pruned else self.rows, L, self.qkv[i], self.o[i], self.h[i], self.d[li],
                        row_index=self.row_index if pruned else None)

    def decode(self, xdec):
        """xdec: fp16 [n_decode, HIDDEN]: one new token per step through every layer."""
        nl = len(self.layers)
        for step in range(self.n_decode):
            for li, L in enumerate(self.layers):
                i = step * nl + li if self.keep_intermediates else 0
                self._layer(xdec[step:step + 1], 1, L, self.qkv_dec[i], self.o_dec[i], self.h_dec[i],
                            self.d_dec[step, li])
