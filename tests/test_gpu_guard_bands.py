"""Out-of-bounds stores that the caching allocator would hide: every output of the library (y,
winners, each gradient) and its workspace is carved out of a larger buffer filled with a byte
pattern, with a guard band in front and behind.  After the forward pass, the backward pass (stored
and recomputed winners), the statistics pass and the allocation-free forward the bands must be
untouched.  Seeded random descriptors over all modes, dtypes, windows, strides and widths."""
import numpy as np
import pytest
import torch

from paper_2504_06881_b200 import inputs, tconv

pytestmark = pytest.mark.gpu

GUARD = 4096          # bytes in front of and behind every carved buffer
PATTERN = 0xA5


class Arena:
    """Carves 256-byte aligned byte ranges, each with guard bands, out of one pattern-filled buffer."""

    def __init__(self, nbytes):
        self.buf = torch.full((nbytes,), PATTERN, dtype=torch.uint8, device="cuda")
        self.pos = 0
        self.used = []

    def take(self, nbytes, dtype=torch.uint8, shape=None):
        start = (self.pos + GUARD + 255) // 256 * 256
        end = start + nbytes
        self.pos = end
        assert self.pos + GUARD <= self.buf.numel(), "arena too small"
        self.used.append((start, end))
        t = self.buf[start:end].view(dtype)
        return t.view(shape) if shape is not None else t

    def check(self, what):
        mask = torch.ones(self.pos + GUARD, dtype=torch.bool, device="cuda")
        for a, b in self.used:
            mask[a:b] = False
        bad = (self.buf[:self.pos + GUARD] != PATTERN) & mask
        assert not bad.any(), f"{what}: {int(bad.sum())} guard bytes overwritten, first at {int(bad.nonzero()[0])}"


ALL = [("max_plus", "max"), ("max_plus", "sum"), ("min_plus", "min"), ("min_plus", "sum"), ("min_plus", "max"),
       ("compound", "sum"), ("parallel", "sum")]


@pytest.mark.parametrize("seed", [31, 32, 33])
def test_outputs_and_workspace_stay_inside_their_buffers(seed):
    rs = np.random.RandomState(seed)
    done = 0
    while done < 40:
        mode, chan = ALL[rs.randint(len(ALL))]
        dtype = ["f32", "bf16"][rs.randint(2)]
        R, S = [(3, 3), (3, 3), (3, 3), (1, 3), (5, 5), (2, 2), (1, 1)][rs.randint(7)]
        st, dl = [1, 1, 2, 3][rs.randint(4)], [1, 1, 2, 4][rs.randint(4)]
        pad = rs.randint(0, 3) if rs.rand() < 0.4 else (S - 1) * dl // 2
        N, C, K = rs.randint(1, 9), rs.randint(1, 40), rs.randint(1, 70)
        H = rs.randint(1, 40)
        W = [rs.randint(1, 70), 4 * rs.randint(1, 16), 8 * rs.randint(1, 8), 28, 14, 7][rs.randint(6)]
        d = inputs.layer(N, C, H, W, K, R, S, stride=st, pad=pad, dil=dl, mode=mode, chan=chan, dtype=dtype)
        if min(inputs.output_hw(d)) <= 0:
            continue
        OH, OW = inputs.output_hw(d)
        if N * K * C * R * S * OH * OW > 1.0e8:
            continue
        done += 1
        dt = tconv.TORCH_DTYPE[dtype]
        es = 4 if dtype == "f32" else 2
        two, par = mode in ("compound", "parallel"), mode == "parallel"
        g = torch.Generator(device="cuda").manual_seed(int(rs.randint(1 << 30)))
        x = torch.randn(N, C, H, W, device="cuda", generator=g).to(dt)
        w = (0.3 * torch.randn(K, C, R, S, device="cuda", generator=g)).to(dt)
        w2 = (0.3 * torch.randn(K, C, R, S, device="cuda", generator=g)).to(dt) if par else None
        al = torch.rand(K, C, device="cuda", generator=g) if two else None
        be = torch.rand(K, C, device="cuda", generator=g) if two else None
        bias = torch.rand(K, device="cuda", generator=g)
        gy = torch.randn(N, K, OH, OW, device="cuda", generator=g).to(dt)
        nwin = tconv.tconv_winner_bytes(d)
        nws_f, nws_b, nws_s = (tconv.tconv_workspace_bytes(d, False), tconv.tconv_workspace_bytes(d, True),
                               tconv.tconv_stats_workspace_bytes(d))
        sizes = [N * K * OH * OW * es, nwin, nws_f, nws_b, nws_s, N * C * H * W * es, 2 * K * C * R * S * 4,
                 2 * K * C * 4, 3 * K * 4, N * K * OH * OW * es]
        A = Arena(sum(sizes) + (len(sizes) + 8) * (2 * GUARD + 256))
        f32 = torch.float32
        y = A.take(sizes[0], dt, (N, K, OH, OW))
        win = A.take(nwin)
        ws_f, ws_b, ws_s = A.take(nws_f), A.take(nws_b), A.take(nws_s)
        gx = A.take(sizes[5], dt, (N, C, H, W))
        gw = A.take(K * C * R * S * 4, f32, (K, C, R, S))
        gw2 = A.take(K * C * R * S * 4, f32, (K, C, R, S)) if par else None
        ga = A.take(K * C * 4, f32, (K, C)) if two else None
        gb = A.take(K * C * 4, f32, (K, C)) if two else None
        gbias = A.take(K * 4, f32, (K,))
        s1, s2 = A.take(K * 4, f32, (K,)), A.take(K * 4, f32, (K,))
        y2 = A.take(sizes[9], dt, (N, K, OH, OW))
        assert tconv.tconv_forward(d, x, w, w2, al, be, bias, y, win, ws_f) == 0
        torch.cuda.synchronize()
        A.check(f"forward {d} [{tconv.tconv_last_kernel()}]")
        for winners in (win, None):
            rc = tconv.tconv_backward(d, x, w, w2, al, be, gy, winners, gx, gw, gw2, ga, gb, gbias, ws_b)
            assert rc == 0, tconv.tconv_status_string(rc)
            torch.cuda.synchronize()
            A.check(f"backward winners={'stored' if winners is not None else 'recomputed'} {d} [{tconv.tconv_last_kernel()}]")
        assert tconv.tconv_forward_stats(d, x, w, w2, al, be, bias, y2, None, s1, s2, ws_s) == 0
        torch.cuda.synchronize()
        A.check(f"forward_stats {d}")
        if nws_f <= tconv.tconv_forward_noalloc_max_scratch():
            assert tconv.tconv_forward_noalloc(d, x, w, w2, al, be, bias, y2, win) == 0
            torch.cuda.synchronize()
            A.check(f"forward_noalloc {d}")
            assert torch.equal(y, y2)
        assert tconv.tconv_device_status() == 0


@pytest.mark.parametrize("seed", [41, 42])
def test_three_dimensional_entry_points_stay_inside_their_buffers(seed):
    """The same guard bands around the outputs and the workspace of tconv3d_forward / tconv3d_backward,
    on seeded random one-dimensional layers (long windows, the kernels with their own scratch layout)
    and small volumes, stored and recomputed winners."""
    from paper_2504_06881_b200 import tconv3d
    rs = np.random.RandomState(seed)
    done = 0
    while done < 30:
        mode, chan = ALL[rs.randint(len(ALL))]
        dtype = ["f32", "bf16"][rs.randint(2)]
        if rs.rand() < 0.7:          # one-dimensional
            S = int(rs.choice([4, 5, 9, 16, 33, 80, 81, 200, 256]))
            st = int(rs.choice([1, 2, 4, 3]))
            L = int(rs.randint(S, 6 * S + 200))
            d = inputs.layer3d(int(rs.randint(1, 5)), int(rs.randint(1, 6)), 1, 1, L, int(rs.randint(1, 40)),
                               T=1, R=1, S=S, stride=(1, 1, st), pad=(0, 0, int(rs.randint(0, S // 2 + 1))),
                               mode=mode, chan=chan, dtype=dtype)
        else:
            d = inputs.layer3d(int(rs.randint(1, 3)), int(rs.randint(1, 5)), int(rs.randint(3, 9)),
                               int(rs.randint(3, 9)), int(rs.randint(3, 12)), int(rs.randint(1, 9)),
                               T=int(rs.randint(1, 4)), R=int(rs.randint(1, 4)), S=int(rs.randint(1, 4)),
                               stride=int(rs.randint(1, 3)), pad=int(rs.randint(0, 2)), mode=mode, chan=chan, dtype=dtype)
        od = inputs.output_dhw(d)
        if min(od) <= 0:
            continue
        done += 1
        dt = tconv.TORCH_DTYPE[dtype]
        two, par = mode in ("compound", "parallel"), mode == "parallel"
        N, C, K = d["N"], d["C"], d["K"]
        g = torch.Generator(device="cuda").manual_seed(int(rs.randint(1 << 30)))
        xs, ws_ = (N, C, d["D"], d["H"], d["W"]), (K, C, d["T"], d["R"], d["S"])
        x = torch.randn(xs, device="cuda", generator=g).to(dt)
        w = (0.3 * torch.randn(ws_, device="cuda", generator=g)).to(dt)
        w2 = (0.3 * torch.randn(ws_, device="cuda", generator=g)).to(dt) if par else None
        al = torch.rand(K, C, device="cuda", generator=g) if two else None
        be = torch.rand(K, C, device="cuda", generator=g) if two else None
        bias = torch.rand(K, device="cuda", generator=g)
        ys = (N, K) + tuple(od)
        gy = torch.randn(ys, device="cuda", generator=g).to(dt)
        es = 4 if dtype == "f32" else 2
        ny, nx = int(np.prod(ys)) * es, int(np.prod(xs)) * es
        nwin, nws = tconv3d.tconv3d_winner_bytes(d), tconv3d.tconv3d_workspace_bytes(d, True)
        nw4 = int(np.prod(ws_)) * 4
        arena = Arena(ny + nx + nwin + nws + 2 * nw4 + 3 * K * C * 4 + 16 * (GUARD + 256))
        y = arena.take(ny, dt, ys)
        win = arena.take(nwin)
        wsb = arena.take(nws)
        gx = arena.take(nx, dt, xs)
        gw = arena.take(nw4, torch.float32, ws_)
        gw2 = arena.take(nw4, torch.float32, ws_) if par else None
        ga = arena.take(K * C * 4, torch.float32, (K, C)) if two else None
        gb = arena.take(K * C * 4, torch.float32, (K, C)) if two else None
        gbias = arena.take(K * 4, torch.float32, (K,))
        assert tconv3d.tconv3d_forward(d, x, w, w2, al, be, bias, y, win) == 0
        torch.cuda.synchronize()
        arena.check(f"tconv3d_forward {d}")
        for winners in (win, None):
            assert tconv3d.tconv3d_backward(d, x, w, w2, al, be, gy, winners, gx, gw, gw2, ga, gb, gbias, wsb) == 0
            torch.cuda.synchronize()
            arena.check(f"tconv3d_backward (winners {'stored' if winners is not None else 'recomputed'}) {d}")
