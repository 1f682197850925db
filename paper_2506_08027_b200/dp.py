"""Data-parallel linear-layer step: tokens split over ranks, every rank owning a row range of the weight.

Sec. 3.2 of the paper fixes what one device computes: weights, activations and output gradients are converted to
MXFP8 with blocks along each product's reduction axis, then FPROP, DGRAD and WGRAD run on the copies.  Sharded,
that arithmetic needs two exchanges and nothing else:

* the weight operand of every rank is the ranks' shard conversions one under another: each rank converts its own
  rows straight into its slot of the gathered buffers and ONE all-gather per buffer moves MXFP8 bytes
  (1 + 1/32 bytes per element and orientation instead of 2 bytes of BF16).  Blocks never cross a shard, so the
  gathered bytes are exactly the conversion of the whole weight; only the column-blocked scales need a
  permutation afterwards (mxfp8_sf_concat_k), because their blocks run down the sharded axis;
* dW is the sum over ranks of partial products over their own tokens; rank r keeps rows r*F/world .. .  The
  WGRAD kernel adds its tiles into the owners' FP32 buffers while it runs (mxfp8_gemm_reduce_scatter, over
  buffers mapped from the other ranks' processes), so the reduction and the scatter ride under the product.

The collectives go through torch.distributed (NCCL on one GPU per rank); every arithmetic step is a call into the
C library.  `ShardPlan` is the host-side arithmetic (which bytes go where) and needs no GPU.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import binding as B


def _swizzled_scale_bytes(mn: int, nkb: int) -> int:
    return ((mn + 127) // 128) * ((nkb + 3) // 4) * 512


class ShardPlan:
    """Which rows of the weight a rank owns and where its conversions sit in the gathered buffers.

    The gathered buffers are laid out so that rank r's contribution to each of them is ONE contiguous slot r of
    equal size, which is what an all-gather moves:
      q_row, q_col  [F, H] bytes           slot r = rows r*F_r .. (r+1)*F_r
      s_row         swizzled [F, H/32]     slot r = atom rows r*F_r/128 .. (whole 512-byte atoms, same order)
      s_col_parts   world x swizzled [H, F_r/32]   slot r = rank r's array; joined along the block axis afterwards
    """

    def __init__(self, world: int, rank: int, T: int, H: int, F: int):
        if world < 1 or not 0 <= rank < world:
            raise ValueError("rank %d of %d" % (rank, world))
        if world > 8:
            raise ValueError("at most 8 owners per WGRAD launch")
        if T <= 0 or H <= 0 or F <= 0 or T % 128 or H % 128:
            raise ValueError("tokens per rank and hidden size must be positive multiples of 128")
        if F % (128 * world):
            raise ValueError("every rank must own whole 128-row tiles of the weight: F %% (128 * world) != 0")
        self.world, self.rank, self.T, self.H, self.F = world, rank, T, H, F
        self.F_r = F // world
        self.q_slot_bytes = self.F_r * H
        self.s_row_slot_bytes = _swizzled_scale_bytes(self.F_r, H // 32)
        self.s_col_part_bytes = _swizzled_scale_bytes(H, self.F_r // 32)
        self.s_row_bytes = _swizzled_scale_bytes(F, H // 32)
        self.s_col_bytes = _swizzled_scale_bytes(H, F // 32)
        assert self.s_row_slot_bytes * world == self.s_row_bytes and self.s_col_part_bytes * world == self.s_col_bytes

    def rows(self, r: int | None = None):
        r = self.rank if r is None else r
        return r * self.F_r, (r + 1) * self.F_r

    def slot(self, nbytes_per_slot: int, r: int | None = None):
        r = self.rank if r is None else r
        return r * nbytes_per_slot, (r + 1) * nbytes_per_slot

    def first_owner(self) -> int:
        """The owner whose rows this rank's WGRAD launch produces first: its own, so that at any time the ranks
        send to different GPUs."""
        return self.rank


def share_owner_buffers(t: torch.Tensor, group=None):
    """Every rank passes its own FP32 buffer; returns (addresses, keepalive): the device address of every rank's
    buffer as mapped into THIS process (CUDA IPC through torch's storage sharing; the own buffer directly).  The
    mappings live as long as `keepalive` does; peer access to the other ranks' devices is switched on here."""
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    if world == 1:
        return [t.data_ptr()], []
    rank = dist.get_rank(group)
    assert t.is_cuda and t.is_contiguous()
    handle = t.untyped_storage()._share_cuda_()
    mine = (handle, t.storage_offset() * t.element_size(), t.device.index)
    everyone = [None] * world
    dist.all_gather_object(everyone, mine, group=group)
    addresses, keep = [], []
    for r, (h, offset, dev) in enumerate(everyone):
        if r == rank:
            addresses.append(t.data_ptr())
            continue
        storage = torch.UntypedStorage._new_shared_cuda(*h)
        keep.append(storage)
        addresses.append(storage.data_ptr() + offset)
        if dev != t.device.index:
            with torch.cuda.device(t.device):
                B.mxfp8_enable_peer_access(dev)
    return addresses, keep


class DataParallelLinear:
    """One linear layer's FPROP + DGRAD + WGRAD on MXFP8 copies, data parallel (see the module text).

    step(x [T, H] BF16, w_shard [F/world, H] BF16, dy [T, F] BF16) -> (y [T, F] BF16, dx [T, H] BF16,
    dw_shard [F/world, H] FP32): all device tensors of this rank; the returned tensors are owned by this object
    and valid, in stream order, until the next step.  Every rank calls step() the same number of times.
    """

    def __init__(self, T: int, H: int, F: int, scale_rule: int = B.RULE_PAPER, group=None, device=None, exchange_when_alone: bool = False):
        self.group = group
        self.world = dist.get_world_size(group) if dist.is_initialized() else 1
        self.rank = dist.get_rank(group) if dist.is_initialized() else 0
        self.plan = p = ShardPlan(self.world, self.rank, T, H, F)
        self.rule = scale_rule
        self.device = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
        B.lib()   # fails loudly when the CUDA library is missing
        # NCCL moves device memory in stream order; any other backend (two ranks sharing one GPU in a test) goes through the host
        self.on_stream = not dist.is_initialized() or dist.get_backend(group) == "nccl"
        # a single rank has nothing to exchange; `exchange_when_alone` issues the collectives all the same (a one-rank group must exist)
        self.exchange = self.world > 1 or exchange_when_alone
        u8 = dict(dtype=torch.uint8, device=self.device)
        self.wq_row, self.wq_col = torch.empty(F, H, **u8), torch.empty(F, H, **u8)
        self.ws_row, self.ws_col = torch.empty(p.s_row_bytes, **u8), torch.empty(p.s_col_bytes, **u8)
        self.ws_col_parts = torch.empty(p.s_col_bytes, **u8)
        self.xq = [torch.empty(T, H, **u8) for _ in range(2)]
        self.xs = [torch.empty(B.mxfp8_scale_bytes(T, H, o, B.SF_SWIZZLED), **u8) for o in (B.ROW, B.COL)]
        self.dyq = [torch.empty(T, F, **u8) for _ in range(2)]
        self.dys = [torch.empty(B.mxfp8_scale_bytes(T, F, o, B.SF_SWIZZLED), **u8) for o in (B.ROW, B.COL)]
        self.y = torch.empty(T, F, dtype=torch.bfloat16, device=self.device)
        self.dx = torch.empty(T, H, dtype=torch.bfloat16, device=self.device)
        self.dw_shard = torch.zeros(p.F_r, H, dtype=torch.float32, device=self.device)
        self._token = torch.zeros(1, dtype=torch.float32, device=self.device)
        self.owner_addresses, self._keep = share_owner_buffers(self.dw_shard, group)
        self.owners = B.make_owner_pointers(self.owner_addresses)
        lo, hi = p.rows()
        a, b = p.slot(p.s_row_slot_bytes)
        c, d = p.slot(p.s_col_part_bytes)
        self._w_slots = (self.wq_row[lo:hi], self.ws_row[a:b], self.wq_col[lo:hi], self.ws_col_parts[c:d])
        self._gathers = ((self.wq_row.view(-1), self.wq_row[lo:hi].view(-1)), (self.wq_col.view(-1), self.wq_col[lo:hi].view(-1)),
                         (self.ws_row, self.ws_row[a:b]), (self.ws_col_parts, self.ws_col_parts[c:d]))
        E, K_, MN = B.E4M3, B.K_MAJOR, B.MN_MAJOR
        self._products = B.make_gemm_problems([
            (self.xq[0], self.xs[0], self.wq_row, self.ws_row, T, F, H, K_, K_, E, E, self.y),          # FPROP  Y  = X  W^T
            (self.dyq[0], self.dys[0], self.wq_col, self.ws_col, T, H, F, K_, MN, E, E, self.dx),       # DGRAD  dX = dY W
        ])
        self._sources = None
        self._items = None

    # ------------------------------------------------------------------ exchanges
    def _all_gather_slots(self):
        if not self.exchange:
            return []
        if self.on_stream:
            return [dist.all_gather_into_tensor(full, mine, group=self.group, async_op=True) for full, mine in self._gathers]
        torch.cuda.synchronize(self.device)
        for full, mine in self._gathers:
            parts = [torch.empty(mine.numel(), dtype=torch.uint8) for _ in range(self.world)]
            dist.all_gather(parts, mine.cpu(), group=self.group)
            full.copy_(torch.cat(parts))
        return []

    def _everyone_arrived(self):
        """Returns, in stream order, only after every rank's work queued so far has finished."""
        if not self.exchange:
            return
        if self.on_stream:
            dist.all_reduce(self._token, group=self.group)
        else:
            torch.cuda.synchronize(self.device)
            dist.barrier(group=self.group)

    # ------------------------------------------------------------------ the step
    def step(self, x: torch.Tensor, w_shard: torch.Tensor, dy: torch.Tensor):
        p = self.plan
        assert x.shape == (p.T, p.H) and w_shard.shape == (p.F_r, p.H) and dy.shape == (p.T, p.F)
        assert x.dtype == w_shard.dtype == dy.dtype == torch.bfloat16
        key = (x.data_ptr(), dy.data_ptr())
        if self._sources != key:
            self._items = B.make_quantize_items([(x, self.xq[0], self.xs[0], self.xq[1], self.xs[1]),
                                                 (dy, self.dyq[0], self.dys[0], self.dyq[1], self.dys[1])])
            self._sources = key
        # the own rows of dW start from zero; the gather below cannot complete anywhere before every rank got here
        self.dw_shard.zero_()
        B.mxfp8_quantize(w_shard, B.BOTH, self.rule, B.E4M3, *self._w_slots, B.SF_SWIZZLED)
        pending = self._all_gather_slots()
        # activations and gradients are converted while the weight bytes travel
        B.mxfp8_quantize_multi(self._items, B.BF16, B.BOTH, self.rule, B.E4M3, B.SF_SWIZZLED)
        for work in pending:
            work.wait()
        B.mxfp8_sf_concat_k(self.ws_col_parts, self.world, p.H, p.F_r, self.ws_col)
        B.mxfp8_gemm_multi(self._products, B.BF16)
        # WGRAD  dW = dY^T X over this rank's tokens, added into every owner's rows as the tiles finish
        B.mxfp8_gemm_reduce_scatter(self.dyq[1], self.dys[1], self.xq[1], self.xs[1], p.F, p.H, p.T, B.MN_MAJOR, B.MN_MAJOR,
                                    B.E4M3, B.E4M3, self.owners, p.first_owner())
        self._everyone_arrived()
        return self.y, self.dx, self.dw_shard
