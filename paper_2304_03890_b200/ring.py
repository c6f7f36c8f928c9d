"""C-Allreduce across real ranks (one process per GPU, `torch.distributed` point-to-point transfers): the
ring of Sec. III-A-2 / Fig. 4 followed by the compress-once allgather of Sec. III-A-1 / III-E-1, with the same
chunking and the same order of operations as `ccoll_allreduce_sim`, so that rank r's result equals row r of the
replay bit for bit.

What crosses the wire is only compressed streams (and, before each, its 8-byte length: the streams have
variable size, Sec. III-E-2).  A received stream lands in this rank's own memory before any kernel reads it;
no kernel ever loads from a peer.  All arithmetic is done by the codec that is passed in:

  * `GpuCodec` — the C-ABI kernels (`ccoll_compress`, `ccoll_reduce_step_op`, `ccoll_decompress`) on CUDA
    tensors; with the NCCL backend the streams travel GPU to GPU over NVLink.
  * the tests pass a CPU codec built on the oracle to check the ring itself with `gloo` ranks.

Schedule on rank r of P (chunk c = values [c*C, (c+1)*C), C = ccoll_chunk_len):
  round 0        compress own chunk r
  round k=1..P-1 send the current stream to r+1, receive the stream of chunk r-k from r-1, reduce it with the
                 local chunk r-k and recompress (the last round also keeps the uncompressed result: this rank
                 owns chunk r+1)
  allgather      P-1 hops: forward the received stream unchanged, decompress a copy; the owner never
                 decompresses its own chunk.

Overlap (Sec. III-E: the paper hides compression behind communication by polling between pieces of work).
Here a chunk is cut into `segments` pieces on block boundaries, each a stream of its own, and the codec's
operations are queued without waiting for them: while the device reduces and recompresses piece s of a round,
the host is already exchanging piece s+1, and a piece's length is waited for only when it is about to be
sent, one round later.  On a GPU the transfers are issued on a side stream, so that reading a length or
staging a stream waits for that transfer alone and not for the kernels queued behind it.  The codec works
block by block (Sec. III-D), so cutting on block boundaries leaves every decoded value unchanged: the result
equals the unsegmented ring's (and the replay's) bit for bit; only the framing bytes on the wire grow.
"""
import torch
import torch.distributed as dist

from . import binding as B


class Ready:
    """A stream that is already complete (codecs that compute synchronously return these)."""

    def __init__(self, stream):
        self._stream = stream

    def stream(self):
        return self._stream


class _Pending:
    """A stream whose kernel is queued: its length reaches the host through a pinned word and an event."""

    def __init__(self, buf, host_len, event, keep):
        self.buf, self.host_len, self.event, self.keep = buf, host_len, event, keep

    def stream(self):
        self.event.synchronize()
        return self.buf[: int(self.host_len[0])]


class GpuCodec:
    """The three device operations of the ring, through the C ABI, queued on the current CUDA stream."""

    _SLOTS = 512  # lengths in flight at most (two per segment are)

    def __init__(self, eb, op=B.SUM, block_len=B.BLOCK_LEN):
        self.eb, self.op, self.block_len = float(eb), op, block_len
        self._host = torch.zeros(self._SLOTS, dtype=torch.int64).pin_memory()
        self._slot = 0

    def prepare(self, longest, in_flight):
        """Called once before anything is queued: the workspace must not change while kernels are in flight,
        and every stream whose length has not been read yet needs a pinned word of its own."""
        if in_flight > self._SLOTS:
            raise ValueError(f"at most {self._SLOTS // 2} segments")
        B.ensure_workspace(longest)

    def empty_stream(self, nbytes, like):
        return torch.empty(nbytes, dtype=torch.uint8, device=like.device)

    def _queued(self, n, device, launch):
        out = torch.empty(B.ccoll_compress_bound(n, self.block_len), dtype=torch.uint8, device=device)
        nbytes = torch.zeros(1, dtype=torch.int64, device=device)
        launch(out, nbytes)
        host_len = self._host[self._slot: self._slot + 1]
        self._slot = (self._slot + 1) % self._SLOTS
        host_len.copy_(nbytes, non_blocking=True)
        event = torch.cuda.Event()
        event.record()
        return _Pending(out, host_len, event, (nbytes,))

    def compress(self, x):
        return self._queued(x.numel(), x.device, lambda out, nb: B.ccoll_compress(x, self.eb, out, nb, self.block_len))

    def reduce_step(self, stream, local, result_out):
        return self._queued(local.numel(), local.device, lambda out, nb: B.ccoll_reduce_step_op(
            stream, stream.numel(), local, self.eb, self.op, out, nb, result_out, self.block_len))

    def decompress(self, stream, n, out):
        B.ccoll_decompress(stream, stream.numel(), n, out, self.block_len)

    def finish(self):
        """Waits for everything queued and raises if a kernel reported an error."""
        status = B.ccoll_get_status()
        if status != B.OK:
            raise B.CcollError(status, "ring (device)")


def _exchange_here(send_buf, like, codec, dst, src, group):
    """Send `send_buf` (a uint8 stream) to dst and receive the neighbour's stream from src: lengths first."""
    # gloo carries host memory only: a device stream is then staged through the host (NCCL takes it as it is)
    staged = send_buf.is_cuda and dist.get_backend(group) == "gloo"
    dev = torch.device("cpu") if staged else send_buf.device
    wire_out = send_buf.cpu() if staged else send_buf
    n_out = torch.tensor([send_buf.numel()], dtype=torch.int64, device=dev)
    n_in = torch.zeros(1, dtype=torch.int64, device=dev)
    for w in dist.batch_isend_irecv([dist.P2POp(dist.isend, n_out, dst, group), dist.P2POp(dist.irecv, n_in, src, group)]):
        w.wait()
    nbytes = int(n_in.item())
    wire_in = torch.empty(nbytes, dtype=torch.uint8) if staged else codec.empty_stream(nbytes, like)
    for w in dist.batch_isend_irecv([dist.P2POp(dist.isend, wire_out, dst, group), dist.P2POp(dist.irecv, wire_in, src, group)]):
        w.wait()
    return wire_in.to(send_buf.device) if staged else wire_in


def _exchange(send_buf, like, codec, dst, src, group, side):
    """The exchange, on the side stream when there is one; the compute stream then waits for the received bytes."""
    if side is None:
        return _exchange_here(send_buf, like, codec, dst, src, group)
    main = torch.cuda.current_stream()
    with torch.cuda.stream(side):
        send_buf.record_stream(side)   # allocated on the compute stream, read here
        incoming = _exchange_here(send_buf, like, codec, dst, src, group)
        incoming.record_stream(main)   # allocated here, read by kernels on the compute stream
    main.wait_stream(side)
    return incoming


def segment_bounds(C, segments, block_len=B.BLOCK_LEN):
    """Cuts [0, C) into at most `segments` pieces on block boundaries (on group boundaries, 32 blocks, where
    the pieces are long enough): list of (lo, hi)."""
    segments = max(1, int(segments))
    unit = 32 * block_len if C >= segments * 32 * block_len else block_len
    per = -(-C // segments)
    per = max(unit, -(-per // unit) * unit)
    return [(lo, min(lo + per, C)) for lo in range(0, max(C, 1), per)]


def c_allreduce(x, codec, group=None, segments=1):
    """All-reduce of the 1-D fp32 tensor x over the ranks of `group`; returns (result, bytes this rank sent)."""
    P = dist.get_world_size(group)
    r = dist.get_rank(group)
    n = x.numel()
    out = torch.empty_like(x)
    if P == 1:
        out.copy_(x)
        return out, 0
    C = B.ccoll_chunk_len(n, P, codec.block_len)
    right, left = (r + 1) % P, (r - 1) % P
    if group is not None:
        right, left = dist.get_global_rank(group, right), dist.get_global_rank(group, left)
    segs = segment_bounds(C, segments, codec.block_len)
    side = torch.cuda.Stream(device=x.device) if x.is_cuda else None

    def piece(t, c, sg):
        return t[min(c * C + sg[0], n): min(c * C + sg[1], n)]

    if hasattr(codec, "prepare"):
        codec.prepare(segs[0][1] - segs[0][0], 2 * len(segs))
    sent = 0
    owned = (r + 1) % P
    cur = [codec.compress(piece(x, r, sg)) for sg in segs]        # round 0, all pieces queued
    for k in range(1, P):
        c = (r - k) % P
        for i, sg in enumerate(segs):
            mine = cur[i].stream()                                 # waits for this piece's kernel only
            sent += mine.numel()
            incoming = _exchange(mine, x, codec, right, left, group, side)
            # the owner's round leaves the uncompressed result where it belongs
            keep = piece(out, c, sg) if k == P - 1 else None
            cur[i] = codec.reduce_step(incoming, piece(x, c, sg), keep if keep is not None and keep.numel() else None)
    cur = [p.stream() for p in cur]
    for h in range(1, P):
        c = (owned - h) % P
        for i, sg in enumerate(segs):
            sent += cur[i].numel()
            cur[i] = _exchange(cur[i], x, codec, right, left, group, side)  # forwarded unchanged on the next hop
            dst = piece(out, c, sg)
            if dst.numel():
                codec.decompress(cur[i], dst.numel(), dst)
    if hasattr(codec, "finish"):
        codec.finish()
    return out, sent
