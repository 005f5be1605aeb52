"""Whole-network EfQAT step over a stack of quantized layers: host-side scheduling only.

Algorithm 1 runs the layer step over every layer of the network; Section 3.2 ("Freezing
Frequency") re-ranks the channels only once per f processed samples and keeps the frozen set
in between.  This module owns that schedule and the per-layer argument lists; every
computation is a call into the C library (selection, network forward / backward with the
fused SGD update of the unfrozen rows, Adam on the quantization parameters, refresh of the
weight-operand caches).  Nothing here touches tensor values.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch

from . import binding as B


class FreezeSchedule:
    """Re-selection once per `f_samples` processed training samples (Section 3.2).  The first
    step always selects; f_samples <= batch_samples means every step."""

    def __init__(self, f_samples: int, batch_samples: int):
        if batch_samples < 1:
            raise ValueError("batch_samples must be positive")
        self.f = max(int(f_samples), 1)
        self.batch = int(batch_samples)
        self.since = None          # samples processed since the last selection; None: never selected
        self.selections = 0
        self.steps = 0

    def due(self) -> bool:
        return self.since is None or self.since >= self.f

    def selected(self):
        self.since = 0
        self.selections += 1

    def advance(self):
        self.since += self.batch
        self.steps += 1


class LayerState:
    """Device tensors of one layer of the stack (all caller-owned device memory)."""

    def __init__(self, case, W, X, dY, bias=None):
        self.case, self.W, self.X, self.dY, self.bias = case, W, X, dY, bias
        self.s_w = self.s_x = self.z_x = self.mom = None


class EfqatNetwork:
    """A stack of fake-quantized linear layers trained with EfQAT.

    mode / budget: efqat_select_channels' mode and k (CWPL: list of per-layer counts; CWPN: one
    channel budget; LWPN: number of layers).  f_samples / batch_samples: the freezing frequency.
    use_cache: keep a weight-operand cache per layer and refresh only the stepped rows.
    sgd = (lr, momentum, weight_decay) enables the fused update of the unfrozen rows;
    adam = dict(lr=..., log2_scale=...) enables the optimizer of the quantization parameters.
    alternate_ws: two workspaces taken in turn (a launch less per layer in the backward) instead of one.
    """

    def __init__(self, ctx: B.Context, layers: Sequence[LayerState], mode: int, budget, f_samples: int,
                 batch_samples: int, use_cache: bool = True, sgd=None, adam: Optional[dict] = None,
                 share_outputs: bool = True, want_db: bool = True, alternate_ws: bool = True):
        self.ctx, self.layers, self.mode = ctx, list(layers), mode
        self.schedule = FreezeSchedule(f_samples, batch_samples)
        self.use_cache = use_cache
        dev = self.layers[0].W.device
        # quantizer parameters: MinMax start (the paper's PTQ initialisation)
        for st in self.layers:
            c = st.case
            if st.s_w is None:
                st.s_w = B.init_weight_scales(ctx, st.W, c.w_bits)
            if st.s_x is None:
                st.s_x, st.z_x = B.init_act_qparams(ctx, st.X, c.x_bits, c.x_symmetric)
        self.L = len(self.layers)
        self.N = [int(st.W.shape[0]) for st in self.layers]
        total = sum(self.N)
        if mode == B.CWPL:
            ks = [int(v) for v in budget]
        else:
            ks = [int(budget)] + [0] * (self.L - 1)
        self._select_plans = {}
        self.select_plan = None
        self.use_selection(mode, ks if mode == B.CWPL else ks[0])
        self.offsets_host = [0] * (self.L + 1)
        # plans: one workspace for the whole stack, output tensors shared per layer shape
        k_max = [n for n in self.N]          # any layer may end up fully unfrozen (LWPN, CWPN)
        descs = []
        ws_need = 0

        def geom(c):
            return B.ConvGeom(c.B, c.H, c.Wd, c.Cin, c.R, c.S, c.stride, c.pad) if c.conv else None

        for st, km in zip(self.layers, k_max):
            c = st.case
            d = B.layer_desc(c.M, c.N, c.K, B.F32 if c.act_dtype == torch.float32 else B.BF16, geom(c))
            spec = B.QSpec(c.w_bits, c.x_bits, 1 if c.x_symmetric else 0)
            ws_need = max(ws_need, B.workspace_bytes(d, spec, km))
            descs.append((d, spec))
        # two workspaces, taken in turn: neighbouring layers then never share one, which lets the library put
        # a layer's finalize work into the next layer's prepare launch (see efqat_network_bwd)
        self.ws = [B.alloc_workspace(ws_need, dev) for _ in range(2 if alternate_ws else 1)]
        self.plans: List[B.LayerPlan] = []
        by_shape = {}
        self.sgds = []
        entries = []
        self.qopts = []
        for li, (st, km) in enumerate(zip(self.layers, k_max)):
            c = st.case
            key = (c.M, c.N, c.K, c.act_dtype, c.conv, c.R, c.stride)
            plan = B.LayerPlan(ctx, c.M, c.N, c.K, c.act_dtype, c.w_bits, c.x_bits, c.x_symmetric, km, dev,
                               conv=geom(c), x_shape=tuple(st.X.shape), y_shape=tuple(st.dY.shape),
                               with_cache=use_cache, ws=self.ws[li % len(self.ws)],
                               outputs=by_shape.get(key) if share_outputs else None)
            by_shape.setdefault(key, plan)
            self.plans.append(plan)
            opt = None
            if sgd is not None:
                st.mom = torch.zeros_like(st.W) if st.mom is None else st.mom
                opt = B.make_sgd(sgd[0], sgd[1], sgd[2], st.W, st.mom)
            self.sgds.append(opt)
            entries.append(plan.net_layer(st.X, st.W, st.s_w, st.s_x, st.z_x, st.bias, st.dY, sgd=opt,
                                          want_db=want_db, use_cache=use_cache))
            if adam is not None:
                self.qopts.append(B.QParamOptimizer(ctx, st.s_w, st.s_x, None if c.x_symmetric else st.z_x, **adam))
        self.net = B.NetworkPlan(ctx, entries, keep=self.sgds)
        if use_cache:
            for st, plan in zip(self.layers, self.plans):
                plan.cache_update(st.W, st.s_w)

    # ------------------------------------------------------------------------------------
    def use_selection(self, mode: int, budget):
        """Switches the selection mode / budget used from the next re-selection on."""
        key = (mode, tuple(budget) if mode == B.CWPL else int(budget))
        if key not in self._select_plans:
            ks = [int(v) for v in budget] if mode == B.CWPL else [int(budget)] + [0] * (self.L - 1)
            self._select_plans[key] = B.SelectPlan(self.ctx, mode, [st.W for st in self.layers], ks)
        self.mode = mode
        self.select_plan = self._select_plans[key]

    def reselect(self):
        """Importance + Top-K over the stack, then the per-layer counts come to the host (the one
        synchronisation of the schedule: the backward's grids are sized by them)."""
        idx, offsets, _ = self.select_plan.run()
        self.offsets_host = offsets.cpu().tolist()
        self.net.set_selection(idx, self.offsets_host)
        self.schedule.selected()

    def counts(self):
        return [self.offsets_host[l + 1] - self.offsets_host[l] for l in range(self.L)]

    def forward(self):
        self.net.fwd()

    def backward(self):
        self.net.bwd()

    def optimizer_tail(self):
        """Adam on the quantization parameters of every layer, then the cache rows of the channels
        whose weights or scales have just moved."""
        if self.qopts:
            self.net.qparam_adam(self.qopts)
        if self.use_cache:
            self.net.cache_update()

    def train_step(self):
        if self.schedule.due():
            self.reselect()
        self.forward()
        self.backward()
        self.optimizer_tail()
        self.schedule.advance()
