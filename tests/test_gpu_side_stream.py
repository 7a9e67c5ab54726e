"""The convenience wrappers allocate their workspace (and outputs) on the current stream but run the
kernels on the stream they are given.  When that is a side stream the caching allocator must not
hand the workspace to the next allocation while the kernels still use it: forward and backward run
on a side stream behind a few milliseconds of other work, the default stream meanwhile allocates
buffers of the sizes the wrappers dropped and keeps overwriting them, and the results must equal those of the same calls on the default
stream, bit for bit."""
import pytest
import torch

from paper_2504_06881_b200 import inputs, tconv

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mode", ["compound", "max_plus"])
def test_wrappers_on_a_side_stream(mode):
    d, dist = inputs.cfg2(mode)
    d = dict(d, N=8)
    t = inputs.draw(d, 1500, **dist)
    two, par = mode in ("compound", "parallel"), mode == "parallel"
    dev = {k: torch.from_numpy(v).cuda() for k, v in t.items()}
    args = dict(w2=dev["w2"] if par else None, alpha=dev["alpha"] if two else None, beta=dev["beta"] if two else None)
    y0, win0 = tconv.forward(d, dev["x"], dev["w"], bias=dev["bias"], want_winners=True, **args)
    g0 = tconv.backward(d, dev["x"], dev["w"], dev["g"], winners=win0, **args)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    sizes = {tconv.tconv_workspace_bytes(d, False), tconv.tconv_workspace_bytes(d, True),
             y0.numel() * y0.element_size(), win0.numel()} | {v.numel() * v.element_size() for v in g0.values()}
    sizes.discard(0)
    spin = torch.empty(1 << 24, device="cuda")
    for rep in range(3):
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for _ in range(40):
                spin.add_(1.0)                  # a few ms: the library's kernels queue behind it
        y1, win1 = tconv.forward(d, dev["x"], dev["w"], bias=dev["bias"], want_winners=True, stream=side, **args)
        g1 = tconv.backward(d, dev["x"], dev["w"], dev["g"], winners=win1, stream=side, **args)
        # the default stream asks for blocks of the sizes the wrappers just dropped and keeps
        # overwriting them while the side stream works through the calls
        junk = [torch.empty(n, dtype=torch.uint8, device="cuda") for n in sizes for _ in range(2)]
        for it in range(150):
            for j in junk:
                j.fill_(0xEE if it % 2 else 0x11)
        torch.cuda.synchronize()
        assert torch.equal(y1, y0) and torch.equal(win1, win0), rep
        for k in g0:
            assert torch.equal(g1[k], g0[k]), (rep, k)
        del junk
