"""Driver for a stack of SSD layers under Multi-Axis Gradient Checkpointing.

Algorithm 1 (forward): segments outer, layers inner; along the layer axis only the INPUT x_j of every
`layer_interval`-th layer is kept (L_ckpt), along the sequence axis the state entering every segment
of every layer (S_ckpt).  Algorithm 2 (backward): segments right to left (outer), blocks of
`layer_interval` layers top to bottom (inner); each grid cell (one block x one segment) is restored
from (x_j slice of its lowest layer, the states entering it): the inputs of its upper layers are
recomputed into `layer_interval - 1` segment-long buffers (the l*s term of Eq. 4), then the cell is
back-propagated layer by layer and hands dx down the stack and dh to the segment on its left.

Layer j: y_j = SSD_j(x_j), x_{j+1} = W (y_j + x_j).  B, C, dt are shared by the layers; A, D are per layer.
This module only marshals: every arithmetic step is a libssd call (ssd_fwd, ssd_bwd_segmented with
one segment per call and the skip-branch gradient folded in, ssd_glue_*).  torch allocates the buffers.
"""
import torch

from . import libssd


class LayerStack:
    def __init__(self, x0, dt, Bm, Cm, A_list, D_list, W, *, chunk, seg, flags=0, layer_interval=1):
        self.layers = len(A_list)
        self.interval = int(layer_interval)
        assert 1 <= self.interval <= self.layers
        self.dt, self.Bm, self.Cm, self.A, self.D, self.W = dt, Bm, Cm, A_list, D_list, W
        self.chunk, self.seg, self.flags = int(chunk), int(seg), int(flags)
        B, L, H, P = x0.shape
        N = Bm.shape[3]
        assert B == 1, "the per-cell slicing below passes pointer offsets: batch 1 (as in the benchmark)"
        assert L % self.seg == 0 and self.seg % self.chunk == 0
        self.B, self.L, self.H, self.P, self.N = B, L, H, P, N
        self.nseg = L // self.seg
        dev = x0.device
        # layer checkpoints: the input of every `interval`-th layer (x[0] is the caller's) and the stack
        # output; None for the layers whose input is recomputed inside a cell
        self.x = [x0] + [torch.empty_like(x0) if (j % self.interval == 0 or j == self.layers) else None
                         for j in range(1, self.layers + 1)]
        # sequence checkpoints: state entering segment k of layer j at [j][k]; [j][nseg] = final state
        self.bnd = torch.zeros(self.layers, self.nseg + 1, B, H, P, N, dtype=torch.float32, device=dev)
        # per-cell scratch
        self.y = torch.empty(B, self.seg, H, P, dtype=x0.dtype, device=dev)
        self.g = [torch.empty(B, self.seg, H, P, dtype=x0.dtype, device=dev) for _ in range(2)]
        self.dz = torch.empty(B, self.seg, H, P, dtype=x0.dtype, device=dev)
        # inputs of the upper layers of a block, one segment long: forward passes through them, the
        # backward recomputes them per cell
        self.cx = [torch.empty(B, self.seg, H, P, dtype=x0.dtype, device=dev) for _ in range(self.interval - 1)]
        self.h_scratch = torch.empty(B, H, P, N, dtype=torch.float32, device=dev) if self.interval > 1 else None
        cell = libssd.SSDShape(B, self.seg, H, P, N, Bm.shape[2], self.chunk, self.seg, libssd.SSD_DTYPE_BF16
                               if x0.dtype == torch.bfloat16 else libssd.SSD_DTYPE_F32, self.flags, 0, 0, 0)
        self.ws_f = libssd.alloc_workspace(cell, libssd.SSD_OP_FWD, dev)
        self.ws_b = libssd.alloc_workspace(cell, libssd.SSD_OP_BWD_SEG, dev)
        self.dh = torch.zeros(self.layers, 2, B, H, P, N, dtype=torch.float32, device=dev)
        # the slices every cell call takes (views; made once, the loops below are launch-bound otherwise)
        ns = self.nseg
        self._xs = [[self._sl(t, k) if t is not None else self.cx[j % self.interval - 1] for k in range(ns)]
                    for j, t in enumerate(self.x)]
        self._dts = [self._sl(dt, k) for k in range(ns)]
        self._Bs = [self._sl(Bm, k) for k in range(ns)]
        self._Cs = [self._sl(Cm, k) for k in range(ns)]
        self._bin = [[self.bnd[j, k:k + 1].reshape(B, 1, H, P, N) for k in range(ns)] for j in range(self.layers)]

    def set_h0(self, layer, h0):
        self.bnd[layer, 0].copy_(h0)

    def _sl(self, t, k):
        return t[:, k * self.seg:(k + 1) * self.seg]

    def forward(self):
        """Algorithm 1.  Returns the stack output x[layers] (a kept buffer)."""
        for k in range(self.nseg):
            for j in range(self.layers):
                xs = self._xs[j][k]
                libssd.ssd_fwd(xs, self._dts[k], self.A[j], self._Bs[k], self._Cs[k],
                               self.D[j], self.bnd[j, k], chunk=self.chunk, seg=self.seg, flags=self.flags,
                               y=self.y, h_final=self.bnd[j, k + 1], ws=self.ws_f)
                libssd.ssd_glue_fwd(xs, self.y, self.W, self._xs[j + 1][k])
        return self.x[self.layers]

    def backward(self, g_top, dh_final=None, out=None, on_cell=None):
        """Algorithm 2.  g_top [B,L,H,P]: gradient of the stack output; dh_final: optional list of
        per-layer final-state gradients.  `out`: dict with dx0 [B,L,H,P], dA/dD [layers,H] (zero-filled
        by the caller or here), and per-cell scratch ddt/dB/dC (one segment long) unless `on_cell`
        wants them kept; on_cell(layer, seg_index, cell_outputs) is called after every cell."""
        dev = g_top.device
        H = self.H
        if out is None:
            out = {}
        out.setdefault("dx0", torch.empty_like(self.x[0]))
        out.setdefault("dA", torch.zeros(self.layers, H, dtype=torch.float32, device=dev))
        out.setdefault("dD", torch.zeros(self.layers, H, dtype=torch.float32, device=dev))
        ddt = torch.empty(self.B, self.seg, H, dtype=torch.float32, device=dev)
        dB = torch.empty(self.B, self.seg, self.Bm.shape[2], self.N, dtype=self.Bm.dtype, device=dev)
        dC = torch.empty_like(dB)
        self.dh.zero_()
        if dh_final is not None:
            for j, t in enumerate(dh_final):
                if t is not None:
                    self.dh[j, 0].copy_(t)
        # dx of a layer = (SSD backward of dz) + dz, the skip branch: the dx kernel adds it itself
        flags = self.flags | libssd.SSD_FLAG_ACCUM_PARAM_GRADS | libssd.SSD_FLAG_SKIP_GRAD
        for k in range(self.nseg - 1, -1, -1):
            cur = (self.nseg - 1 - k) & 1              # dh[j, cur] enters from the right, dh[j, 1-cur] leaves
            g_in = self._sl(g_top, k)
            for j in range(self.layers - 1, -1, -1):
                if self.interval > 1 and (j % self.interval == self.interval - 1 or j == self.layers - 1):
                    self._restore_cell(j - j % self.interval, j, k)
                xs = self._xs[j][k]
                libssd.ssd_glue_bwd(g_in, self.W, self.dz)
                dx = self._sl(out["dx0"], k) if j == 0 else self.g[j & 1]
                cell = dict(dx=dx, ddt=ddt, dA=out["dA"][j], dB=dB, dC=dC, dD=out["dD"][j], dh0=self.dh[j, 1 - cur])
                libssd.ssd_bwd_segmented(xs, self._dts[k], self.A[j], self._Bs[k],
                                         self._Cs[k], self.D[j], self._bin[j][k], self.dz, self.dh[j, cur],
                                         chunk=self.chunk, seg=self.seg, flags=flags, out=cell, ws=self.ws_b)
                if on_cell is not None:
                    on_cell(j, k, dict(cell, dy=self.dz))
                g_in = dx
        last = (self.nseg) & 1                          # buffer holding dh0 of segment 0
        out["dh0"] = [self.dh[j, last] for j in range(self.layers)]
        return out

    def _restore_cell(self, j0, j1, k):
        """Recompute the inputs of layers j0+1..j1 on segment k from the kept x[j0] and the stored states."""
        for j in range(j0, j1):
            xs = self._xs[j][k]
            libssd.ssd_fwd(xs, self._dts[k], self.A[j], self._Bs[k], self._Cs[k], self.D[j], self.bnd[j, k],
                           chunk=self.chunk, seg=self.seg, flags=self.flags, y=self.y, h_final=self.h_scratch,
                           ws=self.ws_f)
            libssd.ssd_glue_fwd(xs, self.y, self.W, self._xs[j + 1][k])

    def checkpoint_bytes(self):
        layer_inputs = sum(t.numel() * t.element_size() for t in self.x if t is not None)
        boundary = self.bnd.numel() * 4
        scratch = self.ws_f.numel() + self.ws_b.numel() + sum(
            t.numel() * t.element_size() for t in [self.y, self.dz, self.g[0], self.g[1]] + self.cx)
        return dict(layer_inputs=layer_inputs, boundary_states=boundary, per_cell_scratch=scratch)
