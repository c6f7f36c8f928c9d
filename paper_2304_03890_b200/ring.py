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
The decompression of hop h is queued on the device while the transfer of hop h+1 is already posted, which is
the device-side counterpart of the overlap the paper obtains by polling (Sec. III-E).
"""
import torch
import torch.distributed as dist

from . import binding as B


class GpuCodec:
    """The three device operations of the ring, through the C ABI."""

    def __init__(self, eb, op=B.SUM, block_len=B.BLOCK_LEN):
        self.eb, self.op, self.block_len = float(eb), op, block_len

    def empty_stream(self, nbytes, like):
        return torch.empty(nbytes, dtype=torch.uint8, device=like.device)

    def compress(self, x):
        return B.compress(x, self.eb, self.block_len)

    def reduce_step(self, stream, local, want_result):
        if want_result:
            return B.reduce_step(stream, local, self.eb, want_sum=True, block_len=self.block_len, op=self.op)
        return B.reduce_step(stream, local, self.eb, block_len=self.block_len, op=self.op), None

    def decompress(self, stream, n, out):
        B.ensure_workspace(n)
        B.ccoll_decompress(stream, stream.numel(), n, out, self.block_len)


def _exchange(send_buf, like, codec, dst, src, group):
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


def c_allreduce(x, codec, group=None):
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

    def chunk(t, c):
        return t[min(c * C, n): min((c + 1) * C, n)]

    sent = 0
    cur = codec.compress(chunk(x, r))                      # round 0
    for k in range(1, P):
        sent += cur.numel()
        incoming = _exchange(cur, x, codec, right, left, group)
        c = (r - k) % P
        cur, result = codec.reduce_step(incoming, chunk(x, c), want_result=(k == P - 1))
    owned = (r + 1) % P
    chunk(out, owned).copy_(result)                        # the owner keeps the uncompressed result
    for h in range(1, P):
        sent += cur.numel()
        cur = _exchange(cur, x, codec, right, left, group)  # forwarded unchanged on the next hop
        c = (owned - h) % P
        dst = chunk(out, c)
        if dst.numel():
            codec.decompress(cur, dst.numel(), dst)
    return out, sent
