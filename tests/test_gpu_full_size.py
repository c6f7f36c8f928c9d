"""The five benchmark configurations at FULL size, in the launch configuration bench.py uses.  The oracle is
too slow to redo them whole, so: (1) sampled groups / windows are recomputed by the oracle and must match
bit for bit (a group's payload depends on its own 4096 values only; a ring window depends on the same window
of every rank); (2) properties that hold at any size are checked over everything on the GPU."""
import struct

import numpy as np
import pytest
import torch

from oracle import ccz
from paper_2304_03890_b200 import binding as B
from paper_2304_03890_b200 import fields

pytestmark = pytest.mark.gpu
GROUP = 4096


def stream_views(stream, n):
    """(dir [G+1], bitmap [G], payload_base) of a CCZ1 stream held on the GPU."""
    G = (n + GROUP - 1) // GROUP
    head = stream[: 32 + 8 * G + 4].cpu().numpy()
    assert head[:4].tobytes() == b"CCZ1"
    assert struct.unpack("<Q", head[8:16].tobytes())[0] == n
    d = np.frombuffer(head[32: 32 + 4 * (G + 1)].tobytes(), dtype="<u4").astype(np.int64)
    bm = np.frombuffer(head[32 + 4 * (G + 1): 32 + 8 * G + 4].tobytes(), dtype="<u4")
    base = (36 + 8 * G + 15) // 16 * 16
    assert struct.unpack("<Q", head[24:32].tobytes())[0] == base + 4 * d[G] == stream.numel()
    assert np.all(np.diff(d) >= 0)
    return d, bm, base


def check_sampled_groups(x, stream, eb, groups):
    """Group g of the big stream must equal the oracle's encoding of that group's values alone."""
    n = x.numel()
    d, bm, base = stream_views(stream, n)
    for g in groups:
        xs = x[g * GROUP: min(n, (g + 1) * GROUP)].cpu().numpy()
        ref = ccz.compress(xs, eb)                       # a one-group stream
        got = stream[base + 4 * d[g]: base + 4 * d[g + 1]].cpu().numpy()
        assert np.array_equal(got, ref[48:]), f"group {g}"
        assert bm[g] == struct.unpack("<I", ref[40:44].tobytes())[0], f"bitmap of group {g}"


def sample_groups(G, k=24, seed=0):
    rng = np.random.default_rng(seed)
    return sorted(set([0, 1, G - 1, G // 2] + list(rng.integers(0, G, k))))


def test_config2_compress_decompress_full():
    cfg = fields.config2(device="cuda")
    x, eb = cfg["x"], float(cfg["eb"])
    n = x.numel()
    assert n == 67108864
    stream = B.compress(x, eb)
    check_sampled_groups(x, stream, eb, sample_groups(n // GROUP, 32))
    dec = B.decompress(stream, n)
    assert float((dec.double() - x.double()).abs().max()) <= eb
    # the forced-constant blocks come back exactly
    xb, db = x.view(-1, 128), dec.view(-1, 128)
    forced = (xb == xb[:, :1]).all(dim=1)
    assert 0.15 < float(forced.float().mean()) < 0.25
    assert torch.equal(db[forced], xb[forced])
    # sampled groups of the decoded field against the oracle's decoder
    for g in sample_groups(n // GROUP, 8, seed=1):
        xs = x[g * GROUP: (g + 1) * GROUP].cpu().numpy()
        ref = ccz.decompress(ccz.compress(xs, eb), GROUP)
        assert dec[g * GROUP: (g + 1) * GROUP].cpu().numpy().tobytes() == ref.tobytes()
    ratio = 4 * n / stream.numel()
    assert 1.5 < ratio < 124.1          # inside the envelope of the paper's Table II (plausibility only)


def ring_window_oracle(xs, eb):
    """Oracle replay of the ring for one chunk-aligned window: xs[k] = the window of the k-th rank the chunk
    visits.  Returns (uncompressed final sum, decoded final stream)."""
    s = ccz.compress(xs[0], eb)
    total = xs[0]
    for k in range(1, len(xs)):
        s, total = ccz.reduce_step(s, xs[k], eb, want_sum=True)
    return total, ccz.decompress(s, xs[0].size)


def check_allreduce(x, eb, windows=6):
    P, n = x.shape
    out, moved = B.allreduce_sim(x, eb)
    # within P*eb of the fp64 sum, everywhere
    exact = x[0].double()
    for r in range(1, P):
        exact += x[r].double()
    slack = P * 2.0 ** -23 * float(exact.abs().max())
    for r in range(P):
        assert float((out[r].double() - exact).abs().max()) <= P * eb + slack
    del exact
    C = B.ccoll_chunk_len(n, P)
    rng = np.random.default_rng(5)
    for c in sorted(set([0, P - 1] + list(rng.integers(0, P, windows)))):
        lo, hi = min(n, c * C), min(n, (c + 1) * C)
        G = (hi - lo + GROUP - 1) // GROUP
        for g in sorted(set([0, G - 1, int(rng.integers(0, G))])):
            a, b_ = lo + g * GROUP, min(hi, lo + (g + 1) * GROUP)
            xs = [x[(c + k) % P, a:b_].cpu().numpy() for k in range(P)]
            total, dec = ring_window_oracle(xs, eb)
            owner = (c + P - 1) % P
            assert out[owner, a:b_].cpu().numpy().tobytes() == total.tobytes(), (c, g)
            for r in (owner + 1) % P, (owner + P // 2) % P:
                if r != owner:
                    assert out[r, a:b_].cpu().numpy().tobytes() == dec.tobytes(), (c, g, r)
    return moved


def test_config3_allreduce_full():
    cfg = fields.config3(device="cuda")
    x, eb = cfg["x"], float(np.float32(cfg["eb"]))
    assert tuple(x.shape) == (8, 16777216)
    moved = check_allreduce(x, eb)
    # traffic: 2(P-1)/P * D / CR per rank (Sec. III-E), so far below the uncompressed 2(P-1)/P * D
    assert moved < 2 * 7 * 4 * 16777216


def test_config5_gradient_allreduce_full():
    cfg = fields.config5(device="cuda")
    x, eb = cfg["x"], float(np.float32(cfg["eb"]))
    assert tuple(x.shape) == (16, 25557032)
    check_allreduce(x, eb, windows=4)


def test_config4_scatter_and_bcast_full():
    P = 32
    cfg = fields.config4(device="cuda")
    root, eb = cfg["x"], float(cfg["eb"])
    n = root.numel()
    assert n == 268435456
    C = B.ccoll_chunk_len(n, P)
    sc, cb = B.bcast_sim(root, P, eb, mode=B.SCATTER)
    assert torch.equal(sc[0], root[:C])                  # the root keeps its chunk
    for r in range(1, P):
        assert float((sc[r].double() - root[r * C: (r + 1) * C].double()).abs().max()) <= eb
    rng = np.random.default_rng(2)
    for r in sorted(set([1, P - 1] + list(rng.integers(1, P, 4)))):
        for g in (0, C // GROUP - 1, int(rng.integers(0, C // GROUP))):
            xs = root[r * C + g * GROUP: r * C + (g + 1) * GROUP].cpu().numpy()
            ref = ccz.decompress(ccz.compress(xs, eb), GROUP)
            assert sc[r, g * GROUP: (g + 1) * GROUP].cpu().numpy().tobytes() == ref.tobytes()
    sizes = cb.cpu().numpy()
    assert np.all(sizes > 48) and int(sizes.sum()) < 4 * n
    # bcast: every rank gets all chunks (32 GiB of output); rank r's chunk c equals scatter's rank c output
    bc, cb2 = B.bcast_sim(root, P, eb, mode=B.BCAST)
    assert torch.equal(cb2, cb)
    assert torch.equal(bc[0], root)
    for r in (1, 7, P - 1):
        assert torch.equal(bc[r, :C], bc[1, :C])
        for c in range(1, P):
            assert torch.equal(bc[r, c * C: (c + 1) * C], sc[c])
        assert float((bc[r, :C].double() - root[:C].double()).abs().max()) <= eb


def test_maximum_stream_size():
    """n = CCOLL_MAX_VALUES (2^29 values, 2 GiB of fp32): one stream of 131072 groups; one more value is refused."""
    n = 1 << 29
    g = torch.Generator(device="cuda")
    g.manual_seed(fields.seed_for(9))
    # a cheap smooth-ish signal at full length: random walk per 4096-value group on top of a slow ramp
    x = torch.randn(n, generator=g, device="cuda").mul_(1e-2)
    x = x.view(-1, GROUP).cumsum(dim=1).view(-1).contiguous()
    eb = 1e-2
    stream = B.compress(x, eb)
    G = n // GROUP
    check_sampled_groups(x, stream, eb, sample_groups(G, 12, seed=3))
    dec = B.decompress(stream, n)
    step = 1 << 26
    for a in range(0, n, step):            # in pieces: the fp64 temporaries would not fit otherwise
        assert float((dec[a:a + step].double() - x[a:a + step].double()).abs().max()) <= eb
    del dec, stream
    out = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.CcollError) as e:
        B.lib()  # noqa: keep the library loaded
        B._check(B.lib().ccoll_compress(x.data_ptr(), n + 1, eb, 128, out.data_ptr(), None, None), "ccoll_compress")
    assert e.value.code == B.ERR_UNSUPPORTED
