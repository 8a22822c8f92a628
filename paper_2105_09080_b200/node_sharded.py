"""Node-sharded Gossip-PGA: the n nodes split over several devices, as in the paper's own deployment
(Section 3: gossip between neighbouring nodes, All-Reduce for the global average; appendix,
implementation details: one parameter copy sent and one received per one-peer step).

The arithmetic of a shard's iteration is the library's (`gpga_shard_export`, `gpga_shard_step`), the
schedule of who sends what to whom is the library's too (`gpga_shard_plan`).  This module only
moves the messages: between shards that live in one process (`exchange_local`: one copy per
message) or between ranks of a `torch.distributed` group (`exchange_dist`: isend / irecv for the
gossip messages, an all-gather of the column sums for the global average; NCCL on GPUs, gloo on CPU).

With the send fused into the export kernel (`gpga_shard_export_to`) nothing is moved here at all:
the kernel stores every outgoing row, or the shard's column sums, straight into the receivers'
buffers, and this module only works out the destination addresses (`direct_destinations`) and
orders export and step (`run_local_direct` on one device, `run_dist_direct` over peer-mapped
symmetric memory between the ranks of a group).
"""
from __future__ import annotations

import ctypes as C

from . import binding as B


class ShardPlan(C.Structure):
    """Mirror of gpga_shard_plan_t."""
    _fields_ = [("kind", C.c_int32), ("messages", C.c_int32), ("send_to", C.c_int32 * 2), ("recv_from", C.c_int32 * 2),
                ("send_offset", C.c_int64 * 2), ("dst_offset", C.c_int64 * 2), ("recv_offset", C.c_int64 * 2),
                ("bytes", C.c_int64 * 2), ("gather_bytes", C.c_int64), ("hop", C.c_int64)]


GPGA_SHARD_RING, GPGA_SHARD_EXP, GPGA_SHARD_GLOBAL = 0, 1, 2


def shard_plan(topology, H, n_total, shards, shard, d, k) -> ShardPlan:
    plan = ShardPlan()
    st = B.lib().gpga_shard_plan(topology, H, n_total, shards, shard, d, k, C.byref(plan))
    if st != B.GPGA_OK:
        raise B.GpgaError(st, B.lib().gpga_last_error(None).decode())
    return plan


class NodeShard:
    """One shard on the current CUDA device: a handle over n_total / shards nodes and its exchange
    buffers (uint8 tensors `send` and `recv`)."""

    def __init__(self, n_total, d, topology, H, gamma, seed, shards, shard, sigma=0.0, ld=None, col0=0,
                 device="cuda", logistic=None):
        """logistic: None for the quadratic objective, else dict(l2=..., m=..., batch=...)."""
        import torch
        assert n_total % shards == 0
        self.n_total, self.d, self.topology, self.H = n_total, d, topology, H
        self.shards, self.shard, self.n = shards, shard, n_total // shards
        self.g = B.Gpga(self.n, d, topology, H, gamma, seed)
        if logistic:
            self.g.set_objective(B.GPGA_OBJ_LOGISTIC, l2=logistic["l2"], m=logistic["m"], batch=logistic["batch"])
        else:
            self.g.set_objective(B.GPGA_OBJ_QUADRATIC, sigma=sigma)
        if ld:
            self.g.set_row_stride(ld)
        if col0:
            self.g.set_column_offset(col0)
        self.g._check(B.lib().gpga_set_node_shard(self.g._h, shards, shard))
        nbytes = int(B.lib().gpga_shard_exchange_bytes(self.g._h))
        self.send = torch.zeros(nbytes, dtype=torch.uint8, device=device)
        self.recv = torch.zeros(nbytes, dtype=torch.uint8, device=device)

    def bind(self, x_a, x_b, data, labels=None):
        """data: the local nodes' b (quadratic) or A (logistic, with their labels)."""
        self.g.bind(x_a, x_b, data, labels)

    def init_from_seed(self, x0_kind, x0_std=1.0, b_shift=0.0):
        """Fill this shard's rows of b and X^(0) on the device, keyed by the global node index."""
        self.g.init_from_seed(x0_kind, x0_std, b_shift)

    def plan(self, k) -> ShardPlan:
        return shard_plan(self.topology, self.H, self.n_total, self.shards, self.shard, self.d, k)

    def export(self, k, stream=None):
        self.g._check(B.lib().gpga_shard_export(self.g._h, k, self.send.data_ptr(), self.g._sp(stream)))

    def step(self, k, stream=None):
        self.g._check(B.lib().gpga_shard_step(self.g._h, k, self.recv.data_ptr(), self.g._sp(stream)))

    def export_to(self, k, dests, stream=None, keep=True):
        """First half of iteration k with the send fused in: `dests` are the device addresses
        (`direct_destinations`) the kernel stores the outgoing messages to."""
        arr = (C.c_void_p * len(dests))(*[int(a) for a in dests])
        keep_ptr = self.send.data_ptr() if keep else None
        self.g._check(B.lib().gpga_shard_export_to(self.g._h, k, keep_ptr, arr, len(dests), self.g._sp(stream)))

    def step_from(self, k, recv_ptr, stream=None):
        """Second half of iteration k from the receive area at device address `recv_ptr`."""
        self.g._check(B.lib().gpga_shard_step(self.g._h, k, int(recv_ptr), self.g._sp(stream)))

    def step_interior(self, k, stream=None):
        """The rows of X^(k+1) that need nothing received (can run while the messages travel)."""
        self.g._check(B.lib().gpga_shard_step_interior(self.g._h, k, self.g._sp(stream)))

    def step_boundary(self, k, stream=None):
        """The remaining rows, from the receive buffer; completes iteration k."""
        self.g._check(B.lib().gpga_shard_step_boundary(self.g._h, k, self.recv.data_ptr(), self.g._sp(stream)))

    def set_period(self, H):
        """Averaging period of the schedule from now on (Gossip-AGA drives it iteration by iteration)."""
        self.H = H
        self.g.set_period(H)

    def mean_loss(self):
        """Mean over this shard's nodes of the local loss at their own iterates."""
        return self.g.mean_loss()

    def state_sums(self, out=None, stream=None):
        """The fp64 column sums of this shard's current rows into `out` (a uint8 tensor; default: the
        start of the send buffer, which is free between two iterations only)."""
        out = self.send if out is None else out
        self.g._check(B.lib().gpga_shard_state_sums(self.g._h, out.data_ptr(), self.g._sp(stream)))

    def diagnostics(self, gathered=None, stream=None):
        """This shard's parts (consensus distance, global loss) of the whole problem's diagnostics, from
        all shards' column sums in `gathered` (default: the receive buffer, free between two iterations only)."""
        gathered = self.recv if gathered is None else gathered
        xi, loss = C.c_double(), C.c_double()
        self.g._check(B.lib().gpga_shard_diagnostics(self.g._h, gathered.data_ptr(), self.g._sp(stream),
                                                     C.byref(xi), C.byref(loss)))
        return xi.value, loss.value

    def get_x(self):
        return self.g.get_x()

    def close(self):
        self.g.close()


def exchange_local(shards, k):
    """Deliver iteration k's messages between shards of one process: one copy per message (the
    column sums of a global average: one copy per pair of shards).  `shards[s]` is shard s; each has
    `.send`, `.recv` (uint8 tensors) and `.plan(k)`."""
    for src in shards:
        plan = src.plan(k)
        if plan.kind == GPGA_SHARD_GLOBAL:
            nb = plan.gather_bytes
            for dst in shards:
                dst.recv[src.shard * nb:(src.shard + 1) * nb].copy_(src.send[:nb], non_blocking=True)
            continue
        for m in range(plan.messages):
            dst = shards[plan.send_to[m]]
            lo, nb = plan.send_offset[m], plan.bytes[m]
            dst.recv[plan.dst_offset[m]:plan.dst_offset[m] + nb].copy_(src.send[lo:lo + nb], non_blocking=True)


def exchange_dist(shard, k, group=None, tags=True):
    """Deliver iteration k's messages of this rank's shard through torch.distributed: rank r holds
    shard r.  Gossip messages go point to point (all sends and receives of the iteration posted
    together), the column sums of a global average by an all-gather in rank order.  tags=False posts
    every message with tag 0, i.e. relies on posting order alone, as a backend without tags does."""
    import torch.distributed as dist
    plan = shard.plan(k)
    if plan.kind == GPGA_SHARD_GLOBAL:
        nb = plan.gather_bytes
        world = dist.get_world_size(group)
        dist.all_gather([shard.recv[r * nb:(r + 1) * nb] for r in range(world)], shard.send[:nb], group=group)
        return
    me, ops, local = dist.get_rank(group), [], []
    for m in range(plan.messages):
        lo, nb = plan.send_offset[m], plan.bytes[m]
        if plan.send_to[m] == me:       # a neighbour in the same shard (one shard, or a two-shard ring's both sides)
            local.append((plan.dst_offset[m], lo, nb))
        else:
            ops.append(dist.P2POp(dist.isend, shard.send[lo:lo + nb], plan.send_to[m], group=group, tag=m if tags else 0))
    # Receives are posted in the order of the SENDER's message index: ring slot 0 (the row above) is the
    # upper shard's message 1, slot 1 its lower shard's message 0.  A backend without tags (NCCL) pairs
    # the messages of two ranks in posting order, which matters when both neighbours are one rank
    # (a ring of two shards); a backend with tags (gloo) gets the index as the tag.
    slots = range(plan.messages - 1, -1, -1) if plan.kind == GPGA_SHARD_RING else range(plan.messages)
    for m in slots:
        if plan.recv_from[m] != me:
            lo = plan.recv_offset[m]
            tag = ((1 - m) if plan.kind == GPGA_SHARD_RING else m) if tags else 0
            ops.append(dist.P2POp(dist.irecv, shard.recv[lo:lo + plan.bytes[m]], plan.recv_from[m], group=group, tag=tag))
    for dst, lo, nb in local:
        shard.recv[dst:dst + nb].copy_(shard.send[lo:lo + nb])
    if ops:
        for req in dist.batch_isend_irecv(ops):
            req.wait()


def run_dist(shard, K, k0=0, group=None, tags=True):
    """K iterations of this rank's shard: export, exchange, step."""
    for k in range(k0, k0 + K):
        shard.export(k)
        exchange_dist(shard, k, group, tags)
        shard.step(k)


def run_dist_overlapped(shard, K, k0=0, group=None):
    """The same with the exchange on a stream of its own, overlapped with the rows that need nothing
    received: export -> [exchange on the side stream | interior rows on the main stream] -> boundary
    rows.  CUDA shards on the double buffer only."""
    import torch
    main = torch.cuda.current_stream()
    side = torch.cuda.Stream()
    exported, delivered = torch.cuda.Event(), torch.cuda.Event()
    for k in range(k0, k0 + K):
        shard.export(k)
        exported.record(main)
        with torch.cuda.stream(side):
            side.wait_event(exported)
            exchange_dist(shard, k, group)
            delivered.record(side)
        shard.step_interior(k)
        main.wait_event(delivered)
        shard.step_boundary(k)


def direct_destinations(plan, shard, shards, base_of):
    """Where the export kernel of `shard` stores iteration k's messages (`plan` = its plan for k):
    `base_of(s)` is the device address of shard s's receive area for this iteration.  Gossip:
    message m lands in the area of shard send_to[m] at dst_offset[m]; global average: this shard's
    column sums land in EVERY shard's area, in this shard's slot of the all-gather."""
    if plan.kind == GPGA_SHARD_GLOBAL:
        return [base_of(s) + shard * plan.gather_bytes for s in range(shards)]
    return [base_of(plan.send_to[m]) + plan.dst_offset[m] for m in range(plan.messages)]


def run_local_direct(shards, K, k0=0, keep=True):
    """K iterations of all shards of one process on one device and stream, no copies between them:
    every shard's export kernel writes into the other shards' receive areas.  Two receive areas per
    shard, used alternately by the parity of k (iteration k + 1's exports may run while another
    shard's step of iteration k still reads its area).  Stream order puts every export of iteration
    k before every step of iteration k.  keep=False: no copy of the exported rows is kept for the
    shard's own step (it then forms its half-step again when every row was exported)."""
    import torch
    if not hasattr(shards[0], "recv_pair"):
        for sh in shards:
            sh.recv_pair = (sh.recv, torch.zeros_like(sh.recv))
    for k in range(k0, k0 + K):
        par = k & 1
        for sh in shards:
            dests = direct_destinations(sh.plan(k), sh.shard, sh.shards, lambda s: shards[s].recv_pair[par].data_ptr())
            sh.export_to(k, dests, keep=keep)
        for sh in shards:
            sh.step_from(k, sh.recv_pair[par].data_ptr())


def run_dist_direct(shard, K, k0=0, group=None):
    """The same between the ranks of a torch.distributed group on several GPUs of one node: the two
    receive areas of every rank live in symmetric memory (mapped into every peer), the export kernel
    stores through the peers' addresses, and a barrier of the symmetric-memory group, in stream order
    between export and step, tells every rank that its senders' kernels have completed.  No library
    call moves data; nothing loads from a peer's memory."""
    import torch.distributed as dist
    import torch.distributed._symmetric_memory as symm
    import torch
    group = group or dist.group.WORLD
    nbytes = shard.recv.numel()
    area = (nbytes + 255) // 256 * 256
    buf = symm.empty(2 * area, dtype=torch.uint8, device=shard.recv.device)
    hdl = symm.rendezvous(buf, group.group_name)
    bases = [int(a) for a in hdl.buffer_ptrs]
    me = dist.get_rank(group)
    for k in range(k0, k0 + K):
        off = (k & 1) * area
        dests = direct_destinations(shard.plan(k), me, shard.shards, lambda s: bases[s] + off)
        shard.export_to(k, dests)
        hdl.barrier()
        shard.step_from(k, bases[me] + off)
    hdl.barrier()   # nobody frees its area while a peer's last export may still be storing to it
    torch.cuda.synchronize()


def aga_update(k, warmup_iters, H_init, F, F_init, H):
    """Algorithm 2's period rule (the library's host arithmetic): returns (F_init, H) after a
    global-average iteration k whose mean loss was F."""
    fi, h = C.c_double(F_init), C.c_int64(H)
    st = B.lib().gpga_aga_update(int(k), int(warmup_iters), int(H_init), float(F), C.byref(fi), C.byref(h))
    if st != B.GPGA_OK:
        raise B.GpgaError(st, B.lib().gpga_last_error(None).decode())
    return fi.value, h.value


def run_adaptive(shards, K, H_init, warmup_iters, exchange, mean_of_losses, k0=0):
    """Gossip-AGA (Algorithm 2) on node shards: a counter C counts iterations since the last global
    average; when it reaches the period H the iteration is a global average, the mean loss F over
    ALL nodes is taken at that iteration's state (`mean_of_losses(local mean losses)`: the
    all-reduce of Algorithm 2), and the period is updated by `aga_update`.  `shards`: the shards this
    process drives; `exchange(k)` delivers iteration k's messages.  Returns the period lengths."""
    H, count, F_init, periods = H_init, 0, 0.0, []
    for k in range(k0, k0 + K):
        count += 1
        glob = count == H
        F = mean_of_losses([sh.mean_loss() for sh in shards]) if glob else 0.0
        for sh in shards:
            sh.set_period(1 if glob else 0)     # this iteration: a global average, or a gossip step
        for sh in shards:
            sh.export(k)
        exchange(k)
        for sh in shards:
            sh.step(k)
        if glob:
            periods.append(H)
            count = 0
            F_init, H = aga_update(k, warmup_iters, H_init, F, F_init, H)
    return periods


def run_local_adaptive(shards, K, H_init, warmup_iters, k0=0):
    """Gossip-AGA over all shards of one process (equal shard sizes: the mean of the shard means)."""
    return run_adaptive(shards, K, H_init, warmup_iters, lambda k: exchange_local(shards, k),
                        lambda losses: sum(losses) / len(losses), k0)


def run_dist_adaptive(shard, K, H_init, warmup_iters, k0=0, group=None):
    """Gossip-AGA with one shard per rank: the mean loss is all-reduced over the group (the one scalar
    all-reduce of Algorithm 2), so every rank takes the same period sequence."""
    import torch
    import torch.distributed as dist

    def mean_of_losses(losses):
        t = torch.tensor([losses[0]], dtype=torch.float64, device=shard.recv.device)
        dist.all_reduce(t, group=group)
        return float(t.item()) / dist.get_world_size(group)

    return run_adaptive([shard], K, H_init, warmup_iters, lambda k: exchange_dist(shard, k, group), mean_of_losses, k0)


def _gather_bytes(shard):
    return (shard.d + 3) // 4 * 4 * 8


def _diag_buffers(shard, own):
    """Where the column sums go: the exchange buffers (free between two iterations), or buffers of
    their own (for a call in the middle of an iteration, while the messages are in the exchange buffers)."""
    if not own:
        return shard.send, shard.recv
    if not hasattr(shard, "_diag"):
        import torch
        nb = _gather_bytes(shard)
        shard._diag = (torch.zeros(nb, dtype=torch.uint8, device=shard.recv.device),
                       torch.zeros(nb * shard.shards, dtype=torch.uint8, device=shard.recv.device))
    return shard._diag


def diagnostics_local(shards, own_buffers=False):
    """Consensus distance and global loss f(xbar) of the whole problem from shards of one process:
    every shard's column sums are copied into every shard's gather area in shard order, the parts
    are added.  Uses the exchange buffers, so call it between two iterations -- or with
    own_buffers=True at any point."""
    nb = _gather_bytes(shards[0])
    bufs = [_diag_buffers(sh, own_buffers) for sh in shards]
    for sh, (out, _) in zip(shards, bufs):
        sh.state_sums(out)
    for src, (out, _) in zip(shards, bufs):
        for _, gathered in bufs:
            gathered[src.shard * nb:(src.shard + 1) * nb].copy_(out[:nb], non_blocking=True)
    parts = [sh.diagnostics(gathered) for sh, (_, gathered) in zip(shards, bufs)]
    return sum(p[0] for p in parts), sum(p[1] for p in parts)


def diagnostics_dist(shard, group=None, own_buffers=False):
    """The same with one shard per rank: an all-gather of the column sums, an all-reduce of the two parts."""
    import torch
    import torch.distributed as dist
    nb, world = _gather_bytes(shard), dist.get_world_size(group)
    out, gathered = _diag_buffers(shard, own_buffers)
    shard.state_sums(out)
    dist.all_gather([gathered[r * nb:(r + 1) * nb] for r in range(world)], out[:nb], group=group)
    t = torch.tensor(shard.diagnostics(gathered), dtype=torch.float64, device=shard.recv.device)
    dist.all_reduce(t, group=group)
    return float(t[0].item()), float(t[1].item())
