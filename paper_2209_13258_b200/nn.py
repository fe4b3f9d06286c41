"""torch.nn front end of the split linear layer: a module whose forward and backward are the library's
calls (Section 3.3: the operator is processed as k sequential slices), so that a model can swap an
``nn.Linear`` for it the way the paper's wrapper replaces FSDP's.

Only argument marshalling and autograd bookkeeping happen here; every product, sum and activation runs in
the CUDA kernels behind ``osdp_split_linear_fwd`` / ``osdp_split_linear_bwd``.  CUDA only: there is no CPU path.
"""
from __future__ import annotations

import torch

from . import binding as B


class _SplitLinearFn(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, weight, bias, layer):
        M = x.numel() // layer.in_features
        x2 = x.reshape(M, layer.in_features)
        if not x2.is_contiguous():
            x2 = x2.contiguous()
        N, K, k = layer.out_features, layer.in_features, layer.k_split
        out = torch.empty(M, N, dtype=torch.bfloat16, device=x.device)
        # any gradient of an activated layer, the bias gradient included, is taken through act'(Z)
        need_z = layer.act != B.ACT_NONE and (x.requires_grad or weight.requires_grad or
                                              (bias is not None and bias.requires_grad))
        z = torch.empty(M, N, dtype=torch.bfloat16, device=x.device) if need_z else None
        ws = layer._workspace(M)
        # the parameter is read in place from the flat buffer it lives in (element offset of the view)
        B.osdp_split_linear_fwd(x2, layer.flat, layer.w_offset, bias, M, N, K, k, layer.split_dim, layer.act, out, z, ws,
                                check=True, flags=layer.flags)
        ctx.layer, ctx.M = layer, M
        ctx.save_for_backward(x2, z if z is not None else torch.empty(0, device=x.device), weight)
        ctx.x_shape = x.shape
        ctx.has_bias = bias is not None
        return out.reshape(*x.shape[:-1], N)

    @staticmethod
    def backward(ctx, dy):
        layer, M = ctx.layer, ctx.M
        x2, z, weight = ctx.saved_tensors
        N, K, k = layer.out_features, layer.in_features, layer.k_split
        dy2 = dy.reshape(M, N)
        if not dy2.is_contiguous():
            dy2 = dy2.contiguous()
        need_dx, need_dw, need_db = ctx.needs_input_grad[0], ctx.needs_input_grad[1], ctx.has_bias and ctx.needs_input_grad[2]
        dx = torch.empty(M, K, dtype=torch.bfloat16, device=dy.device) if need_dx else None
        dw = torch.empty(N, K, dtype=torch.bfloat16, device=dy.device) if need_dw else None
        db = torch.empty(N, dtype=torch.float32, device=dy.device) if need_db else None
        ws = layer._workspace(M)
        B.osdp_split_linear_bwd(dy2, x2, layer.flat, layer.w_offset, z if z.numel() else None, M, N, K, k,
                                layer.split_dim, layer.act, dx, dw, 0, B.DTYPE_BF16, layer.flags & B.FLAG_CARRY_BF16,
                                db, ws, check=True)
        return (dx.reshape(ctx.x_shape) if need_dx else None), dw, db, None


class SplitLinear(torch.nn.Module):
    """y = act(x W^T + b), computed as `k_split` sequential slices of W along `split_dim`
    (SPLIT_OUT: rows of W, SPLIT_RED: columns of W and x).  bf16 activations and weight, fp32 bias.

    `flat` (optional): a 1-D bf16 parameter buffer that already holds W [out_features, in_features] row-major
    at element offset `w_offset` (a multiple of 8); the module's `weight` is then a view of it and nothing is
    copied, which is how a flat-parameter wrapper stores its layers.  Without it the module owns its buffer.
    """

    def __init__(self, in_features, out_features, bias=True, k_split=1, split_dim=B.SPLIT_OUT, act=B.ACT_NONE,
                 flags=0, flat=None, w_offset=0, device="cuda"):
        super().__init__()
        if in_features % 8 or out_features % 8:
            raise ValueError("in_features and out_features must be multiples of 8")
        self.in_features, self.out_features = int(in_features), int(out_features)
        self.k_split, self.split_dim, self.act, self.flags = int(k_split), int(split_dim), int(act), int(flags)
        n = self.in_features * self.out_features
        if flat is None:
            w = torch.empty(n, dtype=torch.bfloat16, device=device)
            torch.nn.init.normal_(w, std=0.02)
            self.flat_param = torch.nn.Parameter(w)
            self._flat_owner, self.w_offset = None, 0
        else:
            if flat.dtype != torch.bfloat16 or flat.dim() != 1 or w_offset % 8 or w_offset + n > flat.numel():
                raise ValueError("flat must be a 1-D bf16 buffer holding W at a multiple-of-8 element offset")
            self.flat_param = None
            self._flat_owner, self.w_offset = flat, int(w_offset)
        self.bias = torch.nn.Parameter(torch.zeros(self.out_features, dtype=torch.float32, device=device)) if bias else None
        self._ws = None
        rc, _ = B.osdp_split_linear_workspace_bytes(1, self.out_features, self.in_features, self.k_split, self.split_dim,
                                                    self.act, B.OP_LINEAR_FWD, self.flags)
        if rc:
            raise B.OsdpError(rc, "SplitLinear")

    @property
    def flat(self):
        return self.flat_param if self._flat_owner is None else self._flat_owner

    @property
    def weight(self):
        n = self.in_features * self.out_features
        return self.flat[self.w_offset:self.w_offset + n].view(self.out_features, self.in_features)

    def _workspace(self, M):
        need = 0
        for op in (B.OP_LINEAR_FWD, B.OP_LINEAR_BWD):
            rc, n = B.osdp_split_linear_workspace_bytes(M, self.out_features, self.in_features, self.k_split,
                                                        self.split_dim, self.act, op, self.flags)
            if rc:
                raise B.OsdpError(rc, "osdp_split_linear_workspace_bytes")
            need = max(need, n)
        if self._ws is None or self._ws.numel() < need or self._ws.device != self.flat.device:
            self._ws = B.new_workspace(need, device=self.flat.device)
        return self._ws

    def forward(self, x):
        if not x.is_cuda:
            raise RuntimeError("SplitLinear runs on CUDA only: there is no CPU path")
        if x.dtype != torch.bfloat16:
            raise TypeError("SplitLinear takes bf16 activations")
        return _SplitLinearFn.apply(x, self.weight, self.bias, self)


class _SplitMLPFn(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, flat, b1, b2, layer):
        H, F, k = layer.hidden, layer.ffn, layer.k_split
        M = x.numel() // H
        x2 = x.reshape(M, H)
        if not x2.is_contiguous():
            x2 = x2.contiguous()
        out = torch.empty(M, H, dtype=torch.bfloat16, device=x.device)
        need_grad = x.requires_grad or flat.requires_grad
        # with recomputation no [M, ffn] activation is kept between forward and backward
        z1 = torch.empty(M, F, dtype=torch.bfloat16, device=x.device) if need_grad and not layer.recompute else None
        ws = layer._workspace(M)
        B.osdp_split_mlp_fwd(x2, layer.flat, layer.off_w1, b1, layer.off_w2, b2, M, H, F, k, layer.act, out, z1, ws,
                             check=True, flags=layer.flags & B.FLAG_CARRY_BF16)
        ctx.layer, ctx.M, ctx.x_shape = layer, M, x.shape
        ctx.has_b = (b1 is not None, b2 is not None)
        empty = torch.empty(0, device=x.device)
        ctx.save_for_backward(x2, z1 if z1 is not None else empty, b1 if b1 is not None else empty)
        return out.reshape(*x.shape[:-1], H)

    @staticmethod
    def backward(ctx, dy):
        layer, M = ctx.layer, ctx.M
        H, F, k = layer.hidden, layer.ffn, layer.k_split
        x2, z1, b1 = ctx.saved_tensors
        dy2 = dy.reshape(M, H)
        if not dy2.is_contiguous():
            dy2 = dy2.contiguous()
        need_dx, need_dw = ctx.needs_input_grad[0], ctx.needs_input_grad[1]
        dx = torch.empty(M, H, dtype=torch.bfloat16, device=dy.device) if need_dx else None
        # the gradient of the flat parameter buffer, laid out like it: dW1 and dW2 at the offsets of W1 and W2
        dflat = torch.zeros_like(layer.flat) if need_dw else None
        db1 = torch.empty(F, dtype=torch.float32, device=dy.device) if ctx.has_b[0] and ctx.needs_input_grad[2] else None
        db2 = torch.empty(H, dtype=torch.float32, device=dy.device) if ctx.has_b[1] and ctx.needs_input_grad[3] else None
        flags = (layer.flags & B.FLAG_CARRY_BF16) | (B.FLAG_RECOMPUTE if layer.recompute else 0)
        ws = layer._workspace(M)
        B.osdp_split_mlp_bwd(dy2, x2, layer.flat, layer.off_w1, layer.off_w2, z1 if z1.numel() else None, M, H, F, k,
                             layer.act, dx, dflat, layer.off_w1, layer.off_w2, B.DTYPE_BF16, flags, db1, db2, ws,
                             check=True, b1=b1 if b1.numel() else None)
        return (dx.reshape(ctx.x_shape) if need_dx else None), dflat, db1, db2, None


class SplitMLP(torch.nn.Module):
    """y = act(x W1^T + b1) W2^T + b2, the transformer MLP block computed as `k_split` sequential slices of the
    ffn dimension (Section 3.3 applied to both MatMuls: the first layer's output slice feeds the second layer's
    reduction slice, so only an [M, ffn / k] intermediate exists at a time).  W1 [ffn, hidden] and W2 [hidden, ffn]
    live in one flat bf16 parameter buffer (`flat_param`, W1 first), biases are fp32.

    recompute=True is the activation-checkpointing setting of Section 2.3: the forward saves no [M, ffn]
    pre-activation and the backward recomputes it slice by slice.
    """

    def __init__(self, hidden, ffn, bias=True, k_split=1, act=B.ACT_GELU_TANH, recompute=False, flags=0, device="cuda"):
        super().__init__()
        if hidden % 8 or ffn % 8:
            raise ValueError("hidden and ffn must be multiples of 8")
        self.hidden, self.ffn, self.k_split, self.act = int(hidden), int(ffn), int(k_split), int(act)
        self.recompute, self.flags = bool(recompute), int(flags)
        self.off_w1, self.off_w2 = 0, self.hidden * self.ffn
        w = torch.empty(2 * self.hidden * self.ffn, dtype=torch.bfloat16, device=device)
        torch.nn.init.normal_(w, std=0.02)
        self.flat_param = torch.nn.Parameter(w)
        mk = lambda n: torch.nn.Parameter(torch.zeros(n, dtype=torch.float32, device=device)) if bias else None
        self.b1, self.b2 = mk(self.ffn), mk(self.hidden)
        self._ws = None
        rc, _ = B.osdp_split_linear_workspace_bytes(1, self.ffn, self.hidden, self.k_split, B.SPLIT_OUT, self.act,
                                                    B.OP_MLP_FWD, self.flags)
        if rc:
            raise B.OsdpError(rc, "SplitMLP")

    @property
    def flat(self):
        return self.flat_param

    @property
    def w1(self):
        return self.flat_param[:self.off_w2].view(self.ffn, self.hidden)

    @property
    def w2(self):
        return self.flat_param[self.off_w2:].view(self.hidden, self.ffn)

    def _workspace(self, M):
        need = 0
        for op, fl in ((B.OP_MLP_FWD, self.flags & B.FLAG_CARRY_BF16),
                       (B.OP_MLP_BWD, (self.flags & B.FLAG_CARRY_BF16) | (B.FLAG_RECOMPUTE if self.recompute else 0))):
            rc, n = B.osdp_split_linear_workspace_bytes(M, self.ffn, self.hidden, self.k_split, B.SPLIT_OUT, self.act,
                                                        op, fl)
            if rc:
                raise B.OsdpError(rc, "osdp_split_linear_workspace_bytes")
            need = max(need, n)
        if self._ws is None or self._ws.numel() < need or self._ws.device != self.flat.device:
            self._ws = B.new_workspace(need, device=self.flat.device)
        return self._ws

    def forward(self, x):
        if not x.is_cuda:
            raise RuntimeError("SplitMLP runs on CUDA only: there is no CPU path")
        if x.dtype != torch.bfloat16:
            raise TypeError("SplitMLP takes bf16 activations")
        return _SplitMLPFn.apply(x, self.flat_param, self.b1, self.b2, self)


class _ZdpLinearFn(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, shard, bias, layer, *dp_parts):
        impl = layer.impl
        M = x.numel() // impl.K
        x2 = x.reshape(M, impl.K)
        if not x2.is_contiguous():
            x2 = x2.contiguous()
        need_grad = any(ctx.needs_input_grad)
        z = torch.empty(M, impl.N, dtype=torch.bfloat16, device=x.device) if impl.act != B.ACT_NONE and need_grad else None
        out = impl.forward(x2, bias=bias, z_save=z)
        ctx.layer, ctx.M, ctx.x_shape, ctx.has_bias = layer, M, x.shape, bias is not None
        ctx.save_for_backward(x2, z if z is not None else torch.empty(0, device=x.device))
        return out.reshape(*x.shape[:-1], impl.N)

    @staticmethod
    def backward(ctx, dy):
        layer, M = ctx.layer, ctx.M
        impl = layer.impl
        x2, z = ctx.saved_tensors
        dy2 = dy.reshape(M, impl.N)
        if not dy2.is_contiguous():
            dy2 = dy2.contiguous()
        need_dx = ctx.needs_input_grad[0]
        need_db = ctx.has_bias and ctx.needs_input_grad[2]
        db = torch.empty(impl.N, dtype=torch.float32, device=dy.device) if need_db else None
        dx = impl.backward(dy2, x2, z_saved=z if z.numel() else None, dbias=db, need_dx=need_dx)
        if need_db:
            impl.comm.all_reduce(db, tag="bias")       # the bias is replicated: its gradient is summed over ranks
        # The loop leaves the summed gradients in its own buffers, which the next backward overwrites:
        # autograd gets copies (shard-sized for the ZDP slices, slice-sized for the DP ones).
        g_shard = impl.grad_shard.clone() if ctx.needs_input_grad[1] else None
        g_dp = [impl.dp_grad[s].clone() for s in layer._dp_order]
        return (dx.reshape(ctx.x_shape) if need_dx else None), g_shard, db, None, *g_dp


class ZdpLinear(torch.nn.Module):
    """The split linear layer with its weight sharded over the ranks of a process group, the counterpart of the
    paper's wrapper around a sharded module (Section 3.2, implementation; Section 3.3 for the slices): W is cut
    into `k_split` slices; a ZDP slice is stored as 1 / world of its elements per rank, gathered for use slice by
    slice in forward and backward, and its gradient reduce-scattered; a DP slice (`slice_modes`, e.g. from
    `zdp.slice_modes_from_plan`) is whole on every rank and has its gradient all-reduced.

    Parameters: `shard` (bf16, this rank's part of every ZDP slice), `dp_parts` (the DP slices' compact matrices),
    `bias` (fp32, replicated).  After backward their `.grad` hold this rank's part of the gradient summed over
    ranks (bf16 for the weights, fp32 for the bias), ready for a sharded optimiser step.  Every rank passes its
    own tokens.  Collectives run on the layer's communication stream, overlapped with the slice GEMMs.
    """

    def __init__(self, in_features, out_features, bias=True, k_split=1, split_dim=B.SPLIT_OUT, act=B.ACT_NONE,
                 slice_modes=None, comm=None, flags=0, device="cuda"):
        super().__init__()
        from .zdp import ZdpSplitLinear
        self.impl = ZdpSplitLinear(out_features, in_features, k_split, split_dim, act=act, dw_dtype=B.DTYPE_BF16, comm=comm,
                                   device=device, flags=flags, slice_modes=slice_modes)
        self.in_features, self.out_features = int(in_features), int(out_features)
        self.shard = torch.nn.Parameter(self.impl.param_shard)            # same storage: an optimiser step updates the loop's shard
        self._dp_order = sorted(self.impl.dp_weight)
        self.dp_parts = torch.nn.ParameterList([torch.nn.Parameter(self.impl.dp_weight[s]) for s in self._dp_order])
        self.bias = torch.nn.Parameter(torch.zeros(self.out_features, dtype=torch.float32, device=device)) if bias else None

    def load_full_weight(self, w_full):
        """Keeps this rank's part of a full [out_features, in_features] weight."""
        with torch.no_grad():
            self.impl.load_full_weight(w_full)

    def forward(self, x):
        if not x.is_cuda:
            raise RuntimeError("ZdpLinear runs on CUDA only: there is no CPU path")
        if x.dtype != torch.bfloat16:
            raise TypeError("ZdpLinear takes bf16 activations")
        return _ZdpLinearFn.apply(x, self.shard, self.bias, self, *self.dp_parts)
