"""Slice loop of a sharded (zero-redundancy data parallel) split linear layer, one process per GPU.

Section 3.3, last paragraph, is covered too: a slice may instead be kept in DP mode (replicated
weights, gradient all-reduced), so that one operator runs partly replicated and partly sharded, as
an execution plan from ``osdp_plan_search`` over the operator's slices prescribes.

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

    def all_reduce(self, t, tag=None):
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=self.group)

    def barrier(self):
        import torch.distributed as dist
        dist.barrier(group=self.group)

    def peer_buffers(self, numel, dtype, device):
        """One buffer of `numel` elements per rank, all addressable from this GPU: this rank's own and the
        peer-mapped ones of the other ranks (torch symmetric memory over the group).  Returns the list indexed
        by rank; entry [self.rank] is local memory."""
        import os
        import torch.distributed as dist
        # plain peer mappings are all that is needed: no NVLink multicast object is bound to these buffers
        os.environ.setdefault("TORCH_SYMM_MEM_DISABLE_MULTICAST", "1")
        try:
            import torch.distributed._symmetric_memory as symm
        except ImportError as e:   # pragma: no cover
            raise RuntimeError("peer-mapped buffers need torch.distributed._symmetric_memory") from e
        group = self.group if self.group is not None else dist.group.WORLD
        local = symm.empty(int(numel), dtype=dtype, device=device)
        handle = symm.rendezvous(local, group.group_name)
        self._symm_keep = getattr(self, "_symm_keep", []) + [(local, handle)]
        return [local if r == self.rank else handle.get_buffer(r, (int(numel),), dtype) for r in range(self.world)]


DP, ZDP = 0, 1


def slice_modes_from_plan(k, dp_slices):
    """Per-slice modes for `ZdpSplitLinear(slice_modes=...)` from the plan search's answer for one operator
    (`osdp_plan_search_granularity`: k slices, dp_slices of them replicated).  The slices are identical, so
    which ones stay replicated does not matter to the cost; the first dp_slices do."""
    k, dp_slices = int(k), int(dp_slices)
    if k < 1 or not 0 <= dp_slices <= k:
        raise ValueError("need k >= 1 and 0 <= dp_slices <= k")
    return [DP] * dp_slices + [ZDP] * (k - dp_slices)


class ZdpSplitLinear:
    """Y = act(X W^T + b) with W cut into k slices, each slice either sharded over the ranks (ZDP: gathered
    for use, gradient reduce-scattered) or replicated (DP: resident, gradient all-reduced).  `comm` supplies
    rank, world and the collectives (DistComm by default); `slice_modes` one mode per slice (default all ZDP).

    param_shard : bf16   this rank's parts of the ZDP slices, one after another
    grad_shard  : dw_dtype, same length: this rank's parts of sum over ranks of dW (ZDP slices)
    dp_weight[s], dp_grad[s] : the compact matrices of DP slice s (whole, on every rank)
    Tokens are sharded by the caller: every rank passes its own X / dY rows.
    """

    def __init__(self, N, K, k_split, split_dim, act=B.ACT_NONE, dw_dtype=B.DTYPE_FP32, comm=None, device="cuda",
                 flags=0, slice_modes=None, fused_scatter=False):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("ZdpSplitLinear needs a CUDA device: there is no CPU path")
        self.comm = comm if comm is not None else DistComm()
        self.N, self.K, self.split_dim, self.act, self.dw_dtype = int(N), int(K), int(split_dim), int(act), int(dw_dtype)
        self.flags = int(flags)
        self.layout = ShardLayout(N, K, k_split, split_dim, self.comm.world)
        self.k = self.layout.k
        self.modes = [ZDP] * self.k if slice_modes is None else [int(m) for m in slice_modes]
        if len(self.modes) != self.k or any(m not in (DP, ZDP) for m in self.modes):
            raise ValueError("slice_modes needs one mode (0 = DP, 1 = ZDP) per slice")
        self.device = torch.device(device)
        gdt = torch.float32 if dw_dtype == B.DTYPE_FP32 else torch.bfloat16
        self.zdp_slices = [s for s in range(self.k) if self.modes[s] == ZDP]
        self._zord = {s: i for i, s in enumerate(self.zdp_slices)}
        self._zoff, total = {}, 0                      # where slice s's part starts in this rank's shard buffers
        for s in self.zdp_slices:
            self._zoff[s] = total
            total += self.layout.slices[s][3]
        self.param_shard = torch.zeros(max(total, 8), dtype=torch.bfloat16, device=self.device)
        # fused_scatter: the backward GEMM's epilogue reduce-adds each slice's dW straight into the owners'
        # gradient shards, which therefore have to be addressable from every rank (comm.peer_buffers).  A step
        # is then: zero_grad() on every rank; comm.barrier() (no rank may add into a shard that its owner has
        # not zeroed yet); backward(); comm.barrier() (every rank's terms have arrived); read grad_shard.
        self.fused_scatter = bool(fused_scatter)
        if self.fused_scatter:
            self.peer_grad_shards = self.comm.peer_buffers(max(total, 8), gdt, self.device)
            self.grad_shard = self.peer_grad_shards[self.comm.rank]
            self.grad_shard.zero_()
        else:
            self.grad_shard = torch.zeros(max(total, 8), dtype=gdt, device=self.device)
        self.dp_weight = {s: torch.zeros(self.layout.slices[s][2], dtype=torch.bfloat16, device=self.device)
                          for s in range(self.k) if self.modes[s] == DP}
        self.dp_grad = {s: torch.zeros(self.layout.slices[s][2], dtype=gdt, device=self.device) for s in self.dp_weight}
        # Two staging buffers each for gathered weights and for weight gradients: the next slice is gathered
        # while this one computes.  Their tails beyond a slice's elements are never written by the kernels.
        wst = max([self.layout.slices[s][3] for s in self.zdp_slices] + [0]) * self.comm.world
        self.w_stage = [torch.zeros(wst, dtype=torch.bfloat16, device=self.device)
                        for _ in range(min(2, len(self.zdp_slices)))]
        # (gradient staging only if some slice goes through a collective: not when the epilogue scatters them all)
        need_dw_stage = any(self.modes[s] == ZDP and not self._scatter_ok(s) for s in range(self.k))
        self._gdt = gdt
        self.dw_stage = [torch.zeros(self.layout.stage_elems, dtype=gdt, device=self.device)
                         for _ in range(min(2, self.k) if need_dw_stage else 0)]
        self.comm_stream = torch.cuda.Stream(device=self.device)
        self.side_stream = torch.cuda.Stream(device=self.device)
        self._ws = None
        self._ws_key = None

    # -- bookkeeping ------------------------------------------------------------------------------
    def load_full_weight(self, w_full):
        """Keeps this rank's part of a full [N, K] bf16 weight (initialisation / checkpoint load): the rank's
        shard of every ZDP slice, the whole of every DP slice."""
        w_full = w_full.to(self.device)
        shard = self.layout.shard_of(w_full, self.comm.rank)
        for s in self.zdp_slices:
            _, _, _, n, off, _ = self.layout.slices[s]
            self.param_shard[self._zoff[s]:self._zoff[s] + n].copy_(shard[off:off + n])
        for s, t in self.dp_weight.items():
            t.copy_(self.layout.slice_matrix(w_full, s).contiguous().reshape(-1))

    def full_from_parts(self, shard_bufs, dp_parts):
        """A full [N, K] tensor from all ranks' shard buffers (laid out like param_shard / grad_shard) and the
        DP slices' compact tensors (checkpoint save; copies only)."""
        import torch
        ref = shard_bufs[0] if shard_bufs else next(iter(dp_parts.values()))
        full = torch.empty(self.N, self.K, dtype=ref.dtype, device=ref.device)
        for s, (b, e, elems, n, _, ld) in enumerate(self.layout.slices):
            if self.modes[s] == ZDP:
                o = self._zoff[s]
                flat = torch.cat([sh[o:o + n] for sh in shard_bufs])[:elems]
            else:
                flat = dp_parts[s][:elems]
            self.layout.slice_matrix(full, s).copy_(flat.reshape(-1, ld))
        return full

    def zero_grad(self):
        self.grad_shard.zero_()
        for t in self.dp_grad.values():
            t.zero_()

    def _scatter_ok(self, s):
        """Whether slice s can be reduce-scattered by the GEMM's epilogue (rows divisible by 32 * world)."""
        b, e = self.layout.slices[s][0], self.layout.slices[s][1]
        rows = (e - b) if self.split_dim == B.SPLIT_OUT else self.N
        return self.fused_scatter and self.modes[s] == ZDP and rows % (32 * self.comm.world) == 0

    def staging_bytes(self, M):
        """Bytes this layer holds besides its weights and gradients: staging plus the kernels' workspace."""
        _, f = B.osdp_split_linear_workspace_bytes(M, self.N, self.K, self.k, self.split_dim, self.act,
                                                   B.OP_LINEAR_FWD, (self.flags & B.FLAG_CARRY_BF16) | B.FLAG_SLICE_MAJOR)
        _, b = B.osdp_split_linear_workspace_bytes(M, self.N, self.K, self.k, self.split_dim, self.act,
                                                   B.OP_LINEAR_BWD, (self.flags & B.FLAG_CARRY_BF16) | B.FLAG_SLICE_MAJOR)
        nbytes = lambda ts: sum(t.numel() * t.element_size() for t in ts)
        return {"weight_staging": nbytes(self.w_stage), "grad_staging": nbytes(self.dw_stage), "workspace": max(f, b)}

    def state_bytes(self):
        """Bytes of weights and gradients resident on this rank (shards of ZDP slices, whole DP slices)."""
        nbytes = lambda ts: sum(t.numel() * t.element_size() for t in ts)
        return {"weights": nbytes([self.param_shard] + list(self.dp_weight.values())),
                "grads": nbytes([self.grad_shard] + list(self.dp_grad.values()))}

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
    @staticmethod
    def _mark(stream):
        import torch
        ev = torch.cuda.Event()
        ev.record(stream)
        return ev

    class _Gathers:
        """Issues the all-gathers of the ZDP slices in order, one slice ahead of the slice in use."""

        def __init__(self, layer):
            self.layer, self.issued, self.ready = layer, 0, {}
            self.free = [[], []]            # events after which weight staging buffer b may be overwritten

        def ensure(self, upto):
            import torch
            L = self.layer
            while self.issued <= upto and self.issued < len(L.zdp_slices):
                s = L.zdp_slices[self.issued]
                b = self.issued & 1
                n = L.layout.slices[s][3]
                with torch.cuda.stream(L.comm_stream):
                    for ev in self.free[b]:
                        L.comm_stream.wait_event(ev)        # the slice that last read this buffer is done
                    L.comm.all_gather_slice(L.w_stage[b], L.param_shard, L._zoff[s], n)
                    self.ready[s] = L._mark(L.comm_stream)
                self.issued += 1

        def weights(self, s, streams):
            """The compact weight matrix of slice s, valid on `streams` (gathered one slice ahead for ZDP)."""
            L = self.layer
            if L.modes[s] == DP:
                return L.dp_weight[s], None
            i = L._zord[s]
            self.ensure(i)
            for st in streams:
                st.wait_event(self.ready[s])
            self.ensure(i + 1)                              # buffer (i + 1) & 1 was last read by ordinal i - 1
            return L.w_stage[i & 1], i & 1

    def forward(self, x, bias=None, out=None, z_save=None):
        import torch
        M = x.shape[0]
        cur = torch.cuda.current_stream(self.device)
        if out is None:
            out = torch.empty(M, self.N, dtype=torch.bfloat16, device=self.device)
        ws = self._workspace(M)
        self.comm_stream.wait_stream(cur)                   # weights may just have been updated on `cur`
        two = self.k > 1 and self.split_dim == B.SPLIT_OUT
        lanes = [cur, self.side_stream] if two else [cur, cur]
        if two:
            self.side_stream.wait_stream(cur)
        g = self._Gathers(self)
        g.ensure(0)
        for s in range(self.k):
            st = lanes[s & 1]
            w, b = g.weights(s, [st])
            B.osdp_zdp_linear_fwd_slice(x, w, self.layout.slices[s][5], bias, M, self.N, self.K, self.k,
                                        self.split_dim, self.act, s, out, z_save, ws, stream=st, check=True,
                                        flags=self.flags & B.FLAG_CARRY_BF16)
            if b is not None:
                g.free[b] = [self._mark(st)]
        if two:
            cur.wait_stream(self.side_stream)
        cur.wait_stream(self.comm_stream)                   # join (also what a stream capture needs)
        return out

    def backward(self, dy, x, z_saved=None, dx=None, dbias=None, need_dx=True, accumulate=False):
        """Per slice: W_s (gathered again for ZDP slices: the second all-gather of ZDP), the slice's dX part,
        dW_s and db; then dW_s is reduce-scattered into grad_shard (ZDP) or all-reduced into dp_grad[s] (DP),
        summed over ranks; `accumulate` adds to what is there.  dbias (if given) is this rank's column sum;
        reduce it with comm.all_reduce where needed."""
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
        g = self._Gathers(self)
        g.ensure(0)
        dw_free = [None, None]
        first_done = None
        for s in range(self.k):
            _, _, elems, shard, _, ld = self.layout.slices[s]
            zdp = self.modes[s] == ZDP
            j = s & 1                                       # gradient staging buffer of this slice
            if self._scatter_ok(s):
                # the slice's dW goes from the GEMM's epilogue straight into the owners' shards (always added)
                o = self._zoff[s]
                peers = [int(t.data_ptr()) + o * t.element_size() for t in self.peer_grad_shards]
                st = side if (self.k > 1 and out_split and self.act == B.ACT_NONE and need_dx) else \
                    ((cur, side)[s & 1] if alternate else cur)
                if alternate and s == 1 and self.act != B.ACT_NONE:
                    st.wait_event(first_done)               # slice 0 stages G for every later slice
                split_here = st is side and not alternate    # dX on `cur`, dW (+ db) on `side`
                w, b = g.weights(s, [cur, st] if split_here else [st])
                if split_here:
                    B.osdp_zdp_linear_bwd_slice(dy, x, w, ld, z_saved, M, self.N, self.K, self.k, self.split_dim,
                                                self.act, s, dx, None, 0, self.dw_dtype, flags, None, ws, stream=cur,
                                                check=True)
                    B.osdp_zdp_linear_bwd_slice_scatter(dy, x, w, ld, z_saved, M, self.N, self.K, self.k,
                                                        self.split_dim, self.act, s, None, peers, self.dw_dtype, 0,
                                                        dbias, ws, stream=st, check=True)
                    done = [self._mark(cur), self._mark(st)]
                else:
                    B.osdp_zdp_linear_bwd_slice_scatter(dy, x, w, ld, z_saved, M, self.N, self.K, self.k,
                                                        self.split_dim, self.act, s, dx if need_dx else None, peers,
                                                        self.dw_dtype, flags, dbias, ws, stream=st, check=True)
                    done = [self._mark(st)]
                if s == 0:
                    first_done = done[0]
                if b is not None:
                    g.free[b] = done
                continue
            direct = not zdp and not accumulate             # DP: the kernel writes dp_grad[s] itself
            if not direct and len(self.dw_stage) <= j:      # first use (a DP slice accumulating through staging)
                import torch as _t
                while len(self.dw_stage) <= j:
                    self.dw_stage.append(_t.zeros(self.layout.stage_elems, dtype=self._gdt, device=self.device))
            dw_dst = self.dp_grad[s] if direct else self.dw_stage[j]
            if split_calls:
                w, b = g.weights(s, [cur, side])
                args = (dy, x, w, ld, z_saved, M, self.N, self.K, self.k, self.split_dim, self.act, s)
                B.osdp_zdp_linear_bwd_slice(*args, dx, None, 0, self.dw_dtype, flags, None, ws, stream=cur, check=True)
                if not direct and dw_free[j] is not None:
                    side.wait_event(dw_free[j])             # the collective that read this buffer is done
                B.osdp_zdp_linear_bwd_slice(*args, None, dw_dst, ld, self.dw_dtype, 0, dbias, ws, stream=side,
                                            check=True)
                done = [self._mark(cur), self._mark(side)]
                dw_done = done[1]
            else:
                st = (cur, side)[s & 1] if alternate else cur
                if alternate and s == 1 and self.act != B.ACT_NONE:
                    st.wait_event(first_done)               # slice 0 stages G for every later slice
                w, b = g.weights(s, [st])
                if not direct and dw_free[j] is not None:
                    st.wait_event(dw_free[j])
                B.osdp_zdp_linear_bwd_slice(dy, x, w, ld, z_saved, M, self.N, self.K, self.k, self.split_dim,
                                            self.act, s, dx if need_dx else None, dw_dst, ld, self.dw_dtype, flags,
                                            dbias, ws, stream=st, check=True)
                done = [self._mark(st)]
                dw_done = done[0]
            if s == 0:
                first_done = done[0]
            if b is not None:
                g.free[b] = done
            with torch.cuda.stream(self.comm_stream):
                self.comm_stream.wait_event(dw_done)
                if zdp:
                    o = self._zoff[s]
                    if accumulate:
                        tmp = torch.empty_like(self.dw_stage[j][:shard])
                        self.comm.reduce_scatter_slice(tmp, 0, shard, self.dw_stage[j])
                        self.grad_shard[o:o + shard].add_(tmp)
                    else:
                        self.comm.reduce_scatter_slice(self.grad_shard, o, shard, self.dw_stage[j])
                elif direct:
                    self.comm.all_reduce(self.dp_grad[s], tag=s)
                else:
                    self.comm.all_reduce(self.dw_stage[j][:elems], tag=s)
                    self.dp_grad[s].add_(self.dw_stage[j][:elems])
                if not direct:
                    dw_free[j] = self._mark(self.comm_stream)
        cur.wait_stream(side)
        cur.wait_stream(self.comm_stream)                   # gradients are complete for whoever runs next on `cur`
        return dx

    def backward_step(self, *args, **kwargs):
        """One gradient step with the ordering the epilogue-fused scatter needs.  Every rank zeroes its gradient
        shards; the ranks meet at a barrier (no rank may add into a shard that its owner has not zeroed yet);
        `backward(*args, **kwargs)` runs; the ranks meet again (every rank's terms have arrived) and only then
        are the shards valid to read.  The host waits for the device before each barrier, so the barrier orders
        the ranks' device work, not just their hosts.  Without fused_scatter the collectives order everything
        themselves and this is `backward` (gradients overwritten, or added with accumulate=True)."""
        import torch
        if not self.fused_scatter:
            return self.backward(*args, **kwargs)
        cur = torch.cuda.current_stream(self.device)
        self.zero_grad()
        cur.synchronize()
        self.comm.barrier()
        out = self.backward(*args, **kwargs)
        cur.synchronize()
        self.comm.barrier()
        return out


class ZdpSplitMLP:
    """Linear -> activation -> Linear split along ffn (first layer OUT, second layer RED), slice by slice.  A ZDP
    slice has both its weights, W1[F_s,:] and W2[:,F_s], sharded over the ranks and gathered for use: only those
    of the slice in use (and of the next one, being gathered) exist in full; its dW1 and dW2 are reduce-scattered
    as soon as they exist, by a collective from slice-sized staging or, with fused_scatter, by the GEMMs'
    epilogues.  A DP slice (`slice_modes`, one mode per slice, default all ZDP) keeps both weights whole on every
    rank and has its gradients all-reduced.

    param_shard[0/1], grad_shard[0/1]: this rank's parts of W1 [ffn, hidden] / W2 [hidden, ffn] and of the summed
    gradients, ZDP slice after ZDP slice (ShardLayout of each); dp_weight[0/1][s], dp_grad[0/1][s]: the compact
    matrices of DP slice s.
    """

    def __init__(self, hidden, ffn, k_split, act=B.ACT_GELU_TANH, dw_dtype=B.DTYPE_FP32, comm=None, device="cuda",
                 flags=0, fused_scatter=False, slice_modes=None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("ZdpSplitMLP needs a CUDA device: there is no CPU path")
        self.comm = comm if comm is not None else DistComm()
        self.hidden, self.ffn, self.act, self.dw_dtype, self.flags = int(hidden), int(ffn), int(act), int(dw_dtype), int(flags)
        world = self.comm.world
        self.layouts = [ShardLayout(ffn, hidden, k_split, B.SPLIT_OUT, world),
                        ShardLayout(hidden, ffn, k_split, B.SPLIT_RED, world)]
        self.k = self.layouts[0].k
        self.modes = [ZDP] * self.k if slice_modes is None else [int(m) for m in slice_modes]
        if len(self.modes) != self.k or any(m not in (DP, ZDP) for m in self.modes):
            raise ValueError("slice_modes needs one mode (0 = DP, 1 = ZDP) per slice")
        self.zdp_slices = [s for s in range(self.k) if self.modes[s] == ZDP]
        self._zord = {s: i for i, s in enumerate(self.zdp_slices)}
        self._zoff, totals = [{}, {}], [0, 0]          # where slice s's part starts in this rank's shard buffers
        for i, l in enumerate(self.layouts):
            for s in self.zdp_slices:
                self._zoff[i][s] = totals[i]
                totals[i] += l.slices[s][3]
        self.device = torch.device(device)
        gdt = torch.float32 if dw_dtype == B.DTYPE_FP32 else torch.bfloat16
        self.param_shard = [torch.zeros(max(t, 8), dtype=torch.bfloat16, device=self.device) for t in totals]
        self.fused_scatter = bool(fused_scatter)
        if self.fused_scatter:
            self.peer_grad_shards = [self.comm.peer_buffers(max(t, 8), gdt, self.device) for t in totals]
            self.grad_shard = [p[self.comm.rank] for p in self.peer_grad_shards]
            for t in self.grad_shard:
                t.zero_()
        else:
            self.grad_shard = [torch.zeros(max(t, 8), dtype=gdt, device=self.device) for t in totals]
        dp = [s for s in range(self.k) if self.modes[s] == DP]
        self.dp_weight = [{s: torch.zeros(l.slices[s][2], dtype=torch.bfloat16, device=self.device) for s in dp}
                          for l in self.layouts]
        self.dp_grad = [{s: torch.zeros(l.slices[s][2], dtype=gdt, device=self.device) for s in dp}
                        for l in self.layouts]
        nb = min(2, len(self.zdp_slices))
        self.w_stage = [[torch.zeros(l.stage_elems, dtype=torch.bfloat16, device=self.device) for _ in range(nb)]
                        for l in self.layouts]
        need = any(self.modes[s] == ZDP and not self._scatter_ok(s) for s in range(self.k))
        self.dw_stage = [[torch.zeros(l.stage_elems, dtype=gdt, device=self.device) for _ in range(nb if need else 0)]
                         for l in self.layouts]
        self.comm_stream = torch.cuda.Stream(device=self.device)
        self._ws = None

    def _scatter_ok(self, s):
        ls = self.layouts[0].slices[s][1] - self.layouts[0].slices[s][0]
        m = 32 * self.comm.world
        return self.fused_scatter and self.modes[s] == ZDP and ls % m == 0 and self.hidden % m == 0

    def load_full_weights(self, w1_full, w2_full):
        for i, w in enumerate((w1_full, w2_full)):
            l = self.layouts[i]
            w = w.to(self.device)
            shard = l.shard_of(w, self.comm.rank)
            for s in self.zdp_slices:
                n, off = l.slices[s][3], l.slices[s][4]
                self.param_shard[i][self._zoff[i][s]:self._zoff[i][s] + n].copy_(shard[off:off + n])
            for s, t in self.dp_weight[i].items():
                t.copy_(l.slice_matrix(w, s).contiguous().reshape(-1))

    def full_from_parts(self, i, shard_bufs, dp_parts):
        """The full matrix i (0: [ffn, hidden], 1: [hidden, ffn]) from all ranks' shard buffers (laid out like
        param_shard[i] / grad_shard[i]) and the DP slices' compact tensors (checkpoint save; copies only)."""
        import torch
        l = self.layouts[i]
        ref = shard_bufs[0] if shard_bufs else next(iter(dp_parts.values()))
        full = torch.empty(l.N, l.K, dtype=ref.dtype, device=ref.device)
        for s, (b, e, elems, n, _, ld) in enumerate(l.slices):
            if self.modes[s] == ZDP:
                o = self._zoff[i][s]
                flat = torch.cat([sh[o:o + n] for sh in shard_bufs])[:elems]
            else:
                flat = dp_parts[s][:elems]
            l.slice_matrix(full, s).copy_(flat.reshape(-1, ld))
        return full

    def zero_grad(self):
        for t in self.grad_shard:
            t.zero_()
        for d in self.dp_grad:
            for t in d.values():
                t.zero_()

    def staging_bytes(self, M):
        nbytes = lambda ts: sum(t.numel() * t.element_size() for t in ts)
        _, f = B.osdp_split_linear_workspace_bytes(M, self.ffn, self.hidden, self.k, B.SPLIT_OUT, self.act, B.OP_MLP_FWD,
                                                   self.flags & B.FLAG_CARRY_BF16)
        _, b = B.osdp_split_linear_workspace_bytes(M, self.ffn, self.hidden, self.k, B.SPLIT_OUT, self.act, B.OP_MLP_BWD,
                                                   self.flags & (B.FLAG_CARRY_BF16 | B.FLAG_RECOMPUTE))
        return {"weight_staging": nbytes(self.w_stage[0] + self.w_stage[1]),
                "grad_staging": nbytes(self.dw_stage[0] + self.dw_stage[1]), "workspace": max(f, b)}

    def state_bytes(self):
        """Bytes of weights and gradients resident on this rank (shards of ZDP slices, whole DP slices)."""
        nbytes = lambda ts: sum(t.numel() * t.element_size() for t in ts)
        return {"weights": nbytes(self.param_shard + [t for d in self.dp_weight for t in d.values()]),
                "grads": nbytes(self.grad_shard + [t for d in self.dp_grad for t in d.values()])}

    def _workspace(self, M):
        n = self.staging_bytes(M)["workspace"]
        if self._ws is None or self._ws.numel() != max(n, 256):
            self._ws = B.new_workspace(n, device=self.device)
        return self._ws

    def _gather(self, i, free_events):
        """Both weights of the i-th ZDP slice into staging buffer i & 1, on the communication stream."""
        import torch
        s = self.zdp_slices[i]
        with torch.cuda.stream(self.comm_stream):
            for ev in free_events:
                self.comm_stream.wait_event(ev)
            for m, l in enumerate(self.layouts):
                self.comm.all_gather_slice(self.w_stage[m][i & 1], self.param_shard[m], self._zoff[m][s], l.slices[s][3])
            ev = torch.cuda.Event()
            ev.record(self.comm_stream)
        return ev

    def _weights(self, s, ready, free, cur):
        """The two compact weight matrices of slice s, valid on `cur`: resident (DP), or gathered one ZDP slice
        ahead of use.  Returns (w1, w2, staging buffer index or None)."""
        if self.modes[s] == DP:
            return self.dp_weight[0][s], self.dp_weight[1][s], None
        i = self._zord[s]
        if i + 1 < len(self.zdp_slices):
            ready[i + 1] = self._gather(i + 1, free[(i + 1) & 1])   # buffer (i + 1) & 1 was last read by ordinal i - 1
        cur.wait_event(ready[i])
        return self.w_stage[0][i & 1], self.w_stage[1][i & 1], i & 1

    def forward(self, x, b1=None, b2=None, out=None, z1_save=None):
        import torch
        M = x.shape[0]
        cur = torch.cuda.current_stream(self.device)
        if out is None:
            out = torch.empty(M, self.hidden, dtype=torch.bfloat16, device=self.device)
        ws = self._workspace(M)
        self.comm_stream.wait_stream(cur)
        free, ready = [[], []], {}
        if self.zdp_slices:
            ready[0] = self._gather(0, [])
        for s in range(self.k):
            w1, w2, j = self._weights(s, ready, free, cur)
            B.osdp_zdp_mlp_fwd_slice(x, w1, w2, self.layouts[1].slices[s][5], b1, b2, M, self.hidden, self.ffn, self.k,
                                     self.act, s, out, z1_save, ws, stream=cur, check=True,
                                     flags=self.flags & B.FLAG_CARRY_BF16)
            if j is not None:
                ev = torch.cuda.Event()
                ev.record(cur)
                free[j] = [ev]
        cur.wait_stream(self.comm_stream)                   # join (also what a stream capture needs)
        return out

    def backward(self, dy, x, z1_saved=None, b1=None, dx=None, db1=None, db2=None):
        """z1_saved None: the pre-activation is recomputed per slice (needs b1).  Gradients of the weights are
        summed over ranks into grad_shard (with fused_scatter they add to what is there: zero_grad first) and,
        for DP slices, into dp_grad."""
        import torch
        M = x.shape[0]
        cur = torch.cuda.current_stream(self.device)
        if dx is None:
            dx = torch.empty(M, self.hidden, dtype=torch.bfloat16, device=self.device)
        flags = (self.flags & B.FLAG_CARRY_BF16) | (B.FLAG_RECOMPUTE if z1_saved is None else 0)
        if flags & B.FLAG_RECOMPUTE:
            self.flags |= B.FLAG_RECOMPUTE          # the workspace plan has one more slice-sized buffer
        ws = self._workspace(M)
        self.comm_stream.wait_stream(cur)
        w_free, dw_free, ready = [[], []], [None, None], {}
        if self.zdp_slices:
            ready[0] = self._gather(0, [])
        for s in range(self.k):
            w1, w2, j = self._weights(s, ready, w_free, cur)
            ld2 = self.layouts[1].slices[s][5]
            args = (dy, x, w1, w2, ld2, b1, z1_saved, M, self.hidden, self.ffn, self.k, self.act, s, dx)
            if j is None:
                # DP slice: the kernels write the slice's gradients where they live, then they are summed over ranks
                B.osdp_zdp_mlp_bwd_slice(*args, self.dp_grad[0][s], self.dp_grad[1][s], ld2, None, None, self.dw_dtype,
                                         flags, db1, db2, ws, stream=cur, check=True)
                done = torch.cuda.Event()
                done.record(cur)
                with torch.cuda.stream(self.comm_stream):
                    self.comm_stream.wait_event(done)
                    for m in range(2):
                        self.comm.all_reduce(self.dp_grad[m][s], tag=(m, s))
                continue
            if self._scatter_ok(s):
                peers = [[int(t.data_ptr()) + self._zoff[m][s] * t.element_size() for t in self.peer_grad_shards[m]]
                         for m in range(2)]
                B.osdp_zdp_mlp_bwd_slice(*args, None, None, 0, peers[0], peers[1], self.dw_dtype, flags, db1, db2, ws,
                                         stream=cur, check=True)
                done = torch.cuda.Event()
                done.record(cur)
            else:
                if dw_free[j] is not None:
                    cur.wait_event(dw_free[j])              # the collectives that read these buffers are done
                B.osdp_zdp_mlp_bwd_slice(*args, self.dw_stage[0][j], self.dw_stage[1][j], ld2, None, None,
                                         self.dw_dtype, flags, db1, db2, ws, stream=cur, check=True)
                done = torch.cuda.Event()
                done.record(cur)
                with torch.cuda.stream(self.comm_stream):
                    self.comm_stream.wait_event(done)
                    for m, l in enumerate(self.layouts):
                        self.comm.reduce_scatter_slice(self.grad_shard[m], self._zoff[m][s], l.slices[s][3],
                                                       self.dw_stage[m][j])
                    dw_free[j] = torch.cuda.Event()
                    dw_free[j].record(self.comm_stream)
            w_free[j] = [done]
        cur.wait_stream(self.comm_stream)
        return dx

    def backward_step(self, *args, **kwargs):
        """One gradient step with the ordering the epilogue-fused scatter needs.  Every rank zeroes its gradient
        shards; the ranks meet at a barrier (no rank may add into a shard that its owner has not zeroed yet);
        `backward(*args, **kwargs)` runs; the ranks meet again (every rank's terms have arrived) and only then
        are the shards valid to read.  The host waits for the device before each barrier, so the barrier orders
        the ranks' device work, not just their hosts.  Without fused_scatter the collectives order everything
        themselves and this is `backward` (gradients overwritten, or added with accumulate=True)."""
        import torch
        if not self.fused_scatter:
            return self.backward(*args, **kwargs)
        cur = torch.cuda.current_stream(self.device)
        self.zero_grad()
        cur.synchronize()
        self.comm.barrier()
        out = self.backward(*args, **kwargs)
        cur.synchronize()
        self.comm.barrier()
        return out
