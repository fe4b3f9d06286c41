"""Slice loop of a sharded (zero-redundancy data parallel) split linear layer, one process per GPU.

Section 3.3, last part: every rank keeps 1/world of each weight slice; slice s is all-gathered
into a slice-sized staging buffer while slice s-1 computes, and the slice's weight gradient is
reduce-scattered as soon as it exists, so the gathered weights (and gradients) live at
size(W)/k (two staging buffers each) instead of size(W).  Sections 2.2 / 3.1: ZDP needs two
all-gathers (forward, backward) and one reduce-scatter per operator; here they are issued per slice.

This module is plumbing only: shard bookkeeping (the layout comes from ``osdp_zdp_shard_layout``),
streams/events and ``torch.distributed`` collectives.  All arithmetic runs in the CUDA kernels
behind ``osdp_zdp_linear_fwd_slice`` / ``osdp_zdp_linear_bwd_slice``; there is no CPU fallback.
"""
from __future__ import annotations

from . import binding as B


class ShardLayout:
    """Per-slice shard table of one operator W [N, K] cut into k slices along `split_dim`."""

    def __init__(self, N, K, k_split, split_dim, world):
        self.N, self.K, self.split_dim, self.world = int(N), int(K), int(split_dim), int(world)
        self.k = max(1, int(k_split))
        self.slices = []   # (begin, end, slice_elems, shard_elems, shard_offset, ld)
        D = self.N if self.split_dim == B.SPLIT_OUT else self.K
        for s in range(self.k):
            rc, elems, shard, off, ld = B.osdp_zdp_shard_layout(N, K, self.k, split_dim, world, s)
            if rc:
                raise B.OsdpError(rc, "osdp_zdp_shard_layout")
            rc, b, e = B.osdp_slice_range(D, self.k, s)
            if rc:
                raise B.OsdpError(rc, "osdp_slice_range")
            self.slices.append((b, e, elems, shard, off, ld))
        rc, _, _, total, _ = B.osdp_zdp_shard_layout(N, K, self.k, split_dim, world, self.k)
        if rc:
            raise B.OsdpError(rc, "osdp_zdp_shard_layout")
        self.shard_total = total                                  # elements of a rank's shard buffer
        self.stage_elems = max(sl[3] for sl in self.slices) * self.world   # elements of one staging buffer

    def slice_matrix(self, full, s):
        """The slice's compact matrix cut out of a full [N, K] tensor (any device)."""
        b, e = self.slices[s][0], self.slices[s][1]
        return full[b:e, :] if self.split_dim == B.SPLIT_OUT else full[:, b:e]

    def shard_of(self, full, rank):
        """This rank's shard buffer (1-D, shard_total elements) of a full [N, K] tensor: copies only."""
        import torch
        out = torch.zeros(self.shard_total, dtype=full.dtype, device=full.device)
        for s, (_, _, elems, shard, off, _) in enumerate(self.slices):
            flat = self.slice_matrix(full, s).contiguous().reshape(-1)
            lo, hi = rank * shard, min((rank + 1) * shard, elems)
            if hi > lo:
                out[off:off + hi - lo] = flat[lo:hi]
        return out

    def unshard(self, shards):
        """Inverse of shard_of over all ranks' shard buffers: the full [N, K] tensor (copies only)."""
        import torch
        full = torch.empty(self.N, self.K, dtype=shards[0].dtype, device=shards[0].device)
        for s, (b, e, elems, shard, off, _) in enumerate(self.slices):
            flat = torch.cat([sh[off:off + shard] for sh in shards])[:elems]
            if self.split_dim == B.SPLIT_OUT:
                full[b:e, :] = flat.reshape(e - b, self.K)
            else:
                full[:, b:e] = flat.reshape(self.N, e - b)
        return full


class DistComm:
    """The two collectives of the loop over a torch.distributed process group (NCCL on GPUs)."""

    def __init__(self, group=None):
        import torch.distributed as dist
        if not dist.is_initialized():
            raise RuntimeError("torch.distributed is not initialised")
        self.group = group
        self.rank = dist.get_rank(group)
        self.world = dist.get_world_size(group)

    def all_gather_slice(self, dst, shard_buf, off, n):
        import torch.distributed as dist
        dist.all_gather_into_tensor(dst[:n * self.world], shard_buf[off:off + n], group=self.group)

    def reduce_scatter_slice(self, shard_buf, off, n, src):
        import torch.distributed as dist
        dist.reduce_scatter_tensor(shard_buf[off:off + n], src[:n * self.world], op=dist.ReduceOp.SUM,
                                   group=self.group)

    def all_reduce(self, t):
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=self.group)


class ZdpSplitLinear:
    """Y = act(X W^T + b) with W sharded over the ranks slice by slice; forward and backward gather one
    slice at a time.  `comm` supplies rank, world and the two slice collectives (DistComm by default).

    param_shard : bf16 [layout.shard_total]   this rank's part of W (slice-major)
    grad_shard  : dw_dtype, same length       this rank's part of sum over ranks of dW
    Tokens are sharded by the caller: every rank passes its own X / dY rows.
    """

    def __init__(self, N, K, k_split, split_dim, act=B.ACT_NONE, dw_dtype=B.DTYPE_FP32, comm=None, device="cuda",
                 flags=0):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("ZdpSplitLinear needs a CUDA device: there is no CPU path")
        self.comm = comm if comm is not None else DistComm()
        self.N, self.K, self.split_dim, self.act, self.dw_dtype = int(N), int(K), int(split_dim), int(act), int(dw_dtype)
        self.flags = int(flags)
        self.layout = ShardLayout(N, K, k_split, split_dim, self.comm.world)
        self.k = self.layout.k
        self.device = torch.device(device)
        gdt = torch.float32 if dw_dtype == B.DTYPE_FP32 else torch.bfloat16
        self.param_shard = torch.zeros(self.layout.shard_total, dtype=torch.bfloat16, device=self.device)
        self.grad_shard = torch.zeros(self.layout.shard_total, dtype=gdt, device=self.device)
        # Two staging buffers each for gathered weights and for weight gradients: slice s+1 is gathered
        # while slice s computes.  Their tails beyond a slice's elements are never written by the kernels.
        self.w_stage = [torch.zeros(self.layout.stage_elems, dtype=torch.bfloat16, device=self.device) for _ in range(min(2, self.k))]
        self.dw_stage = [torch.zeros(self.layout.stage_elems, dtype=gdt, device=self.device) for _ in range(min(2, self.k))]
        self.comm_stream = torch.cuda.Stream(device=self.device)
        self.side_stream = torch.cuda.Stream(device=self.device)
        self._ws = None
        self._ws_key = None

    # -- bookkeeping ------------------------------------------------------------------------------
    def load_full_weight(self, w_full):
        """Keeps this rank's shards of a full [N, K] bf16 weight (initialisation / checkpoint load)."""
        self.param_shard.copy_(self.layout.shard_of(w_full.to(self.device), self.comm.rank))

    def staging_bytes(self, M):
        """Bytes this layer holds besides its shards: weight and gradient staging plus the kernels' workspace."""
        _, f = B.osdp_split_linear_workspace_bytes(M, self.N, self.K, self.k, self.split_dim, self.act,
                                                   B.OP_LINEAR_FWD, self.flags & B.FLAG_CARRY_BF16)
        _, b = B.osdp_split_linear_workspace_bytes(M, self.N, self.K, self.k, self.split_dim, self.act,
                                                   B.OP_LINEAR_BWD, self.flags & B.FLAG_CARRY_BF16)
        stage = sum(t.numel() * t.element_size() for t in self.w_stage + self.dw_stage)
        wbytes = len(self.w_stage) * self.w_stage[0].numel() * 2
        return {"weight_staging": wbytes, "grad_staging": stage - wbytes, "workspace": max(f, b)}

    def _workspace(self, M):
        nbytes = self.staging_bytes(M)["workspace"]
        if self._ws is None or self._ws_key != nbytes:
            self._ws = B.new_workspace(nbytes, device=self.device)
            self._ws_key = nbytes
        return self._ws

    # -- the slice loops --------------------------------------------------------------------------
    # Slices whose outputs are concatenated (forward under OUT, dW always, dX under RED) do not depend on
    # one another, so consecutive ones are launched on two alternating streams: the next slice's CTAs
    # take over the SMs that the current slice's last, partly filled wave leaves idle.  Slices of a summed
    # output (forward under RED, dX under OUT) stay in order on the caller's stream.
    def _gather(self, s, free_events):
        """Issues the all-gather of slice s into its staging buffer on the communication stream."""
        import torch
        _, _, _, shard, off, _ = self.layout.slices[s]
        with torch.cuda.stream(self.comm_stream):
            for ev in free_events:
                self.comm_stream.wait_event(ev)             # the slice that last read this buffer is done
            self.comm.all_gather_slice(self.w_stage[s & 1], self.param_shard, off, shard)
            ready = torch.cuda.Event()
            ready.record(self.comm_stream)
        return ready

    @staticmethod
    def _mark(stream):
        import torch
        ev = torch.cuda.Event()
        ev.record(stream)
        return ev

    def forward(self, x, bias=None, out=None, z_save=None):
        import torch
        M = x.shape[0]
        cur = torch.cuda.current_stream(self.device)
        if out is None:
            out = torch.empty(M, self.N, dtype=torch.bfloat16, device=self.device)
        ws = self._workspace(M)
        self.comm_stream.wait_stream(cur)                   # shards may just have been updated on `cur`
        two = self.k > 1 and self.split_dim == B.SPLIT_OUT
        lanes = [cur, self.side_stream] if two else [cur, cur]
        if two:
            self.side_stream.wait_stream(cur)
        done = [[], []]
        ready = self._gather(0, [])
        for s in range(self.k):
            nxt = self._gather(s + 1, done[(s + 1) & 1]) if s + 1 < self.k else None
            st = lanes[s & 1]
            st.wait_event(ready)
            B.osdp_zdp_linear_fwd_slice(x, self.w_stage[s & 1], self.layout.slices[s][5], bias, M, self.N, self.K,
                                        self.k, self.split_dim, self.act, s, out, z_save, ws, stream=st, check=True,
                                        flags=self.flags & B.FLAG_CARRY_BF16)
            done[s & 1] = [self._mark(st)]
            ready = nxt
        if two:
            cur.wait_stream(self.side_stream)
        self.comm_stream.wait_stream(cur)
        return out

    def backward(self, dy, x, z_saved=None, dx=None, dbias=None, need_dx=True, accumulate=False):
        """Gathers W_s again (the second all-gather of ZDP), computes the slice's dX part, dW_s and db, and
        reduce-scatters dW_s into grad_shard (sum over ranks; `accumulate` adds to what is there).
        dbias (if given) is this rank's column sum; reduce it with comm.all_reduce where needed."""
        import torch
        M = x.shape[0]
        cur, side = torch.cuda.current_stream(self.device), self.side_stream
        if need_dx and dx is None:
            dx = torch.empty(M, self.K, dtype=torch.bfloat16, device=self.device)
        ws = self._workspace(M)
        self.comm_stream.wait_stream(cur)
        side.wait_stream(cur)
        out_split = self.split_dim == B.SPLIT_OUT
        # OUT: the dX chain on `cur`, the independent dW_s on `side` (not with an activation: its staged
        # G_s in the workspace serves one stream).  RED: whole slices alternate between the two streams.
        split_calls = self.k > 1 and out_split and self.act == B.ACT_NONE and need_dx
        alternate = self.k > 1 and not out_split
        flags = self.flags & B.FLAG_CARRY_BF16
        w_free = [[], []]
        dw_free = [None, None]
        tmp = torch.empty_like(self.dw_stage[0][:max(sl[3] for sl in self.layout.slices)]) if accumulate else None
        ready = self._gather(0, [])
        for s in range(self.k):
            b = s & 1
            nxt = self._gather(s + 1, w_free[(s + 1) & 1]) if s + 1 < self.k else None
            _, _, _, shard, off, ld = self.layout.slices[s]
            args = (dy, x, self.w_stage[b], ld, z_saved, M, self.N, self.K, self.k, self.split_dim, self.act, s)
            if split_calls:
                cur.wait_event(ready)
                B.osdp_zdp_linear_bwd_slice(*args, dx, None, 0, self.dw_dtype, flags, None, ws, stream=cur, check=True)
                side.wait_event(ready)
                if dw_free[b] is not None:
                    side.wait_event(dw_free[b])             # the reduce-scatter that read this buffer is done
                B.osdp_zdp_linear_bwd_slice(*args, None, self.dw_stage[b], ld, self.dw_dtype, 0, dbias, ws,
                                            stream=side, check=True)
                w_free[b] = [self._mark(cur), self._mark(side)]
                dw_done = w_free[b][1]
            else:
                st = (cur, side)[b] if alternate else cur
                if alternate and s == 1 and self.act != B.ACT_NONE:
                    st.wait_event(w_free[0][0])             # slice 0 stages G for every later slice
                st.wait_event(ready)
                if dw_free[b] is not None:
                    st.wait_event(dw_free[b])
                B.osdp_zdp_linear_bwd_slice(*args, dx if need_dx else None, self.dw_stage[b], ld, self.dw_dtype,
                                            flags, dbias, ws, stream=st, check=True)
                w_free[b] = [self._mark(st)]
                dw_done = w_free[b][0]
            with torch.cuda.stream(self.comm_stream):
                self.comm_stream.wait_event(dw_done)
                if accumulate:
                    self.comm.reduce_scatter_slice(tmp, 0, shard, self.dw_stage[b])
                    self.grad_shard[off:off + shard].add_(tmp[:shard])
                else:
                    self.comm.reduce_scatter_slice(self.grad_shard, off, shard, self.dw_stage[b])
                dw_free[b] = self._mark(self.comm_stream)
            ready = nxt
        cur.wait_stream(side)
        cur.wait_stream(self.comm_stream)                   # grad_shard is complete for whoever runs next on `cur`
        return dx
