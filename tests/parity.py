"""Helpers of the GPU parity tests: run one layer through the C ABI (via the thin
binding) and through the CPU oracle on the same seeded inputs, and compare."""
import numpy as np
import torch

from oracle import tconv_oracle as ora
from paper_2504_06881_b200 import inputs, tconv

# tolerances of the contract: forward outputs and winners bit-exact (+0 == -0);
# gradients within rtol * sum|contribution| elementwise (the summation error bound)
RTOL_GRAD = {"f32": 1e-5, "bf16": 2e-2}


def same_bits(a, b):
    a = np.asarray(a, np.float32); b = np.asarray(b, np.float32)
    return (a.view(np.uint32) == b.view(np.uint32)) | ((a == 0) & (b == 0))


def to_dev(t, d, dev="cuda"):
    """numpy layer tensors -> CUDA tensors in the layer's dtypes."""
    dt = tconv.TORCH_DTYPE[d["dtype"]]
    out = {}
    for k, v in t.items():
        tt = torch.from_numpy(v).to(dev)
        out[k] = tt.to(dt).contiguous() if k in ("x", "w", "w2", "g") else tt.contiguous()
    return out


def layer_args(d, t):
    two = d["mode"] in ("compound", "parallel")
    return dict(w2=t["w2"] if d["mode"] == "parallel" else None,
                alpha=t["alpha"] if two else None, beta=t["beta"] if two else None)


def winners_as_numpy(d, winners):
    N, C, K = d["N"], d["C"], d["K"]
    OH, OW = inputs.output_hw(d)
    chan = ora.resolved_chan(d)
    raw = winners.cpu().numpy()
    if chan != "sum":
        return raw.view(np.int32).reshape(N, K, OH, OW)
    # Sum-form codes: rows padded to a multiple of 4 codes; the padding is not part of the result
    OWP = (OW + 3) // 4 * 4
    if d["R"] * d["S"] <= 16:
        return raw.reshape(N, K, C, OH, OWP)[..., :OW]
    return raw.view(np.uint16).reshape(N, K, C, OH, OWP)[..., :OW]


def oracle_wide_codes(d, t, la):
    """Sum-form winners for windows of more than 16 taps (the oracle emits nibble codes only
    up to 16 taps): rebuilt per channel from single-channel Max/Min runs of the oracle."""
    N, C, K = d["N"], d["C"], d["K"]
    OH, OW = inputs.output_hw(d)
    codes = np.zeros((N, K, C, OH, OW), np.uint16)
    for c in range(C):
        d1 = dict(d, C=1)
        x1 = np.ascontiguousarray(t["x"][:, c:c + 1])
        if d["mode"] in ("min_plus", "compound", "parallel"):
            o = ora.forward(dict(d1, mode="min_plus", chan="min"), x1,
                            np.ascontiguousarray(t["w"][:, c:c + 1]))
            codes[:, :, c] |= o["idx"].astype(np.uint16)
        if d["mode"] in ("max_plus", "compound", "parallel"):
            wm = t["w2"] if d["mode"] == "parallel" else t["w"]
            o = ora.forward(dict(d1, mode="max_plus", chan="max"), x1,
                            np.ascontiguousarray(wm[:, c:c + 1]))
            codes[:, :, c] |= (o["idx"].astype(np.uint16) << 8)
    return codes


def check_forward(d, t, use_bias=True, check_winners=True):
    """GPU forward vs oracle: y and winners bit-exact.  Returns (gpu tensors, y, winners)."""
    la = layer_args(d, t)
    bias = t["bias"] if use_bias else None
    ref = ora.forward(d, t["x"], t["w"], la["w2"], la["alpha"], la["beta"], bias)
    g = to_dev(t, d)
    ga = layer_args(d, g)
    y, winners = tconv.forward(d, g["x"], g["w"], ga["w2"], ga["alpha"], ga["beta"],
                               g["bias"] if use_bias else None, want_winners=check_winners)
    torch.cuda.synchronize()
    yg = y.float().cpu().numpy()
    ok = same_bits(yg, ref["y"])
    assert ok.all(), (f"{d}: {int((~ok).sum())} of {ok.size} outputs differ; first at "
                      f"{np.argwhere(~ok)[0]}: gpu {yg[~ok][0]!r} ref {ref['y'][~ok][0]!r} "
                      f"[{tconv.tconv_last_kernel()}]")
    if check_winners:
        wg = winners_as_numpy(d, winners)
        want = ref["idx"] if ref["idx"] is not None else ref["codes"]
        if want is None:
            want = oracle_wide_codes(d, t, la)
        assert np.array_equal(wg, want), (f"{d}: {int((wg != want).sum())} winners differ "
                                          f"[{tconv.tconv_last_kernel()}]")
    return g, y, winners


def compare_grads(d, got: dict, ref: dict, rtol=None):
    rtol = RTOL_GRAD[d["dtype"]] if rtol is None else rtol
    report = {}
    for name, (rv, ra) in ref.items():
        if name not in got:
            continue
        gv = got[name].float().cpu().numpy().astype(np.float64)
        err = np.abs(gv - rv)
        bound = rtol * ra + 1e-30
        bad = err > bound
        scale = max(np.abs(rv).max(), 1e-30)
        report[name] = float(err.max() / scale)
        assert not bad.any(), (f"{d} {name}: {int(bad.sum())} of {bad.size} elements off; worst "
                               f"err {err[bad].max():.3e} vs bound {bound[bad][err[bad].argmax()]:.3e} "
                               f"[{tconv.tconv_last_kernel()}]")
    return report


def check_layer(d, dists=None, seed=0, use_bias=True, stored_winners=True, recompute=True):
    """Forward + backward parity of one layer.  Returns the normwise gradient errors."""
    t = inputs.draw(d, seed, **(dists or {}))
    g, y, winners = check_forward(d, t, use_bias=use_bias)
    la = layer_args(d, t)
    ref = ora.backward(d, t["x"], t["w"], t["g"], la["w2"], la["alpha"], la["beta"])
    ga = layer_args(d, g)
    rep = {}
    if stored_winners:
        got = tconv.backward(d, g["x"], g["w"], g["g"], ga["w2"], ga["alpha"], ga["beta"], winners)
        torch.cuda.synchronize()
        rep = compare_grads(d, got, ref)
    if recompute:
        got = tconv.backward(d, g["x"], g["w"], g["g"], ga["w2"], ga["alpha"], ga["beta"], None)
        torch.cuda.synchronize()
        rep = compare_grads(d, got, ref)
    return rep


def _backward_by_k_slices(ds, xs, w, g, w2, al, be, step=2):
    """The oracle's backward on a one-image problem, output channels cut into slices that run
    as concurrent oracle calls (the C loops run outside the interpreter lock): grad_x and its
    bound add up over the slices, the parameter gradients concatenate along k."""
    from concurrent.futures import ThreadPoolExecutor
    K = ds["K"]
    cuts = [(a, min(K, a + step)) for a in range(0, K, step)]

    def one(cut):
        a, b = cut
        sl = lambda v: None if v is None else np.ascontiguousarray(v[a:b])
        return ora.backward(dict(ds, K=b - a), xs, sl(w), np.ascontiguousarray(g[:, a:b]), sl(w2), sl(al), sl(be))

    with ThreadPoolExecutor(max_workers=max(1, min(len(cuts), ora.threads()))) as ex:
        parts = list(ex.map(one, cuts))
    out = {}
    for name in parts[0]:
        if name == "grad_x":
            out[name] = tuple(sum(p[name][i] for p in parts) for i in (0, 1))
        else:
            out[name] = tuple(np.concatenate([p[name][i] for p in parts], 0) for i in (0, 1))
    return out


def _one_output_reference(d, t, n, k, oh, ow):
    """The oracle on the receptive field of one output: the window's taps gathered into an
    R x S patch per channel (zeros where the window leaves the image), run as a layer with a
    single output.  Returns (y, winner index or per-channel codes)."""
    C, R, S = d["C"], d["R"], d["S"]
    patch = np.zeros((1, C, R, S), np.float32)
    for r in range(R):
        ih = oh * d["stride_h"] - d["pad_h"] + r * d["dil_h"]
        if not 0 <= ih < d["H"]:
            continue
        for s in range(S):
            iw = ow * d["stride_w"] - d["pad_w"] + s * d["dil_w"]
            if 0 <= iw < d["W"]:
                patch[0, :, r, s] = t["x"][n, :, ih, iw]
    d1 = dict(d, N=1, K=1, H=R, W=S, stride_h=1, stride_w=1, pad_h=0, pad_w=0, dil_h=1, dil_w=1)
    two = d["mode"] in ("compound", "parallel")
    ref = ora.forward(d1, patch, np.ascontiguousarray(t["w"][k:k + 1]),
                      np.ascontiguousarray(t["w2"][k:k + 1]) if d["mode"] == "parallel" else None,
                      np.ascontiguousarray(t["alpha"][k:k + 1]) if two else None,
                      np.ascontiguousarray(t["beta"][k:k + 1]) if two else None,
                      np.ascontiguousarray(t["bias"][k:k + 1]))
    win = ref["idx"][0, 0, 0, 0] if ref["idx"] is not None else ref["codes"][0, 0, :, 0, 0]
    return ref["y"][0, 0, 0, 0], win


def sampled_check(d, t, sample_n, sample_k, fwd_blocks=(), random_outputs=0, random_seed=0):
    """Full-size GPU run against the oracle on a sample.  Forward, winners and backward:
    images sample_n x output channels [sample_k[0], sample_k[1]) (the upstream gradient is zero
    outside that block).  Forward and winners only: every (n, k0, k1) of fwd_blocks, and
    random_outputs seeded random outputs (n, k, oh, ow), each against the oracle run on that
    output's receptive field.  t holds numpy tensors x, w, w2, alpha, beta, bias, g."""
    dt = tconv.TORCH_DTYPE[d["dtype"]]
    two = d["mode"] in ("compound", "parallel")
    par = d["mode"] == "parallel"
    k0, k1 = sample_k
    # upstream gradient: zero outside the sample
    gm = np.zeros_like(t["g"])
    for n in sample_n:
        gm[n, k0:k1] = t["g"][n, k0:k1]
    dev = {k: torch.from_numpy(v).cuda() for k, v in t.items()}
    for k in ("x", "w", "w2"):
        dev[k] = dev[k].to(dt)
    gdev = torch.from_numpy(gm).cuda().to(dt)
    y, win = tconv.forward(d, dev["x"], dev["w"], dev["w2"] if par else None,
                           dev["alpha"] if two else None, dev["beta"] if two else None, dev["bias"],
                           want_winners=True)
    kernel_fwd = tconv.tconv_last_kernel()
    grads = tconv.backward(d, dev["x"], dev["w"], gdev, dev["w2"] if par else None,
                           dev["alpha"] if two else None, dev["beta"] if two else None, win)
    torch.cuda.synchronize()
    assert tconv.tconv_device_status() == 0
    assert "tiled" in kernel_fwd, kernel_fwd
    sum_form = ora.resolved_chan(d) == "sum"

    def winners_of(n, ka, kb):
        """winners of image n, output channels [ka, kb), as the oracle lays them out"""
        OH, OW = inputs.output_hw(d)
        if not sum_form:
            return win.view(torch.int32).view(d["N"], d["K"], OH, OW)[n, ka:kb].cpu().numpy()
        assert d["R"] * d["S"] <= 16, "one-byte codes"
        OWP = (OW + 3) // 4 * 4
        raw = win.view(d["N"], d["K"], d["C"], OH, OWP)[n, ka:kb, :, :, :OW]
        return raw.cpu().numpy()

    def forward_block(n, ka, kb):
        dsb = dict(d, N=1, K=kb - ka)
        slb = lambda a: np.ascontiguousarray(a[ka:kb])
        ref = ora.forward(dsb, np.ascontiguousarray(t["x"][n:n + 1]), slb(t["w"]), slb(t["w2"]) if par else None,
                          slb(t["alpha"]) if two else None, slb(t["beta"]) if two else None, slb(t["bias"]))
        yg = y[n, ka:kb].float().cpu().numpy()
        ok = same_bits(yg, ref["y"][0])
        assert ok.all(), (d["mode"], n, ka, kb, f"{int((~ok).sum())} outputs differ, first at {np.argwhere(~ok)[0]}")
        want = ref["idx"] if ref["idx"] is not None else ref["codes"]
        got = winners_of(n, ka, kb)
        assert np.array_equal(got, want[0]), (d["mode"], n, ka, kb, f"{int((got != want[0]).sum())} winners differ")

    ds = dict(d, N=1, K=k1 - k0)
    sl = lambda a: np.ascontiguousarray(a[k0:k1])
    al, be = (sl(t["alpha"]), sl(t["beta"])) if two else (None, None)
    acc = {}
    for n in sample_n:
        forward_block(n, k0, k1)
        xs = np.ascontiguousarray(t["x"][n:n + 1])
        rb = _backward_by_k_slices(ds, xs, sl(t["w"]), np.ascontiguousarray(gm[n:n + 1, k0:k1]),
                                   sl(t["w2"]) if par else None, al, be)
        compare_grads(d, {"grad_x": grads["grad_x"][n:n + 1]}, {"grad_x": rb["grad_x"]})
        for name, (gv, ga) in rb.items():
            if name == "grad_x":
                continue
            if name not in acc:
                acc[name] = [np.zeros_like(gv), np.zeros_like(ga)]
            acc[name][0] += gv
            acc[name][1] += ga
    # parameter gradients of the sampled channels, zeros elsewhere
    for name, (gv, ga) in acc.items():
        got = grads[name]
        compare_grads(d, {name: got[k0:k1]}, {name: (gv, ga)})
        rest = torch.cat([got[:k0], got[k1:]])
        assert torch.count_nonzero(rest) == 0, name
    others = [n for n in range(d["N"]) if n not in sample_n]
    if others:
        assert torch.count_nonzero(grads["grad_x"][others[:4]]) == 0
    for (n, ka, kb) in fwd_blocks:
        forward_block(n, ka, kb)
    if random_outputs:
        rs = np.random.RandomState(random_seed)
        OH, OW = inputs.output_hw(d)
        pts = np.stack([rs.randint(0, d["N"], random_outputs), rs.randint(0, d["K"], random_outputs),
                        rs.randint(0, OH, random_outputs), rs.randint(0, OW, random_outputs)], 1)
        ii = [torch.from_numpy(pts[:, j]).cuda() for j in range(4)]
        yg = y[ii[0], ii[1], ii[2], ii[3]].float().cpu().numpy()
        if sum_form:
            OWP = (OW + 3) // 4 * 4
            wg = win.view(d["N"], d["K"], d["C"], OH, OWP)[ii[0], ii[1], :, ii[2], ii[3]].cpu().numpy()
        else:
            wg = win.view(torch.int32).view(d["N"], d["K"], OH, OW)[ii[0], ii[1], ii[2], ii[3]].cpu().numpy()
        for j, (n, k, oh, ow) in enumerate(pts):
            yr, wr = _one_output_reference(d, t, int(n), int(k), int(oh), int(ow))
            assert same_bits(yg[j], yr).all(), (d["mode"], "random output", tuple(pts[j]), yg[j], yr)
            assert np.array_equal(wg[j], wr), (d["mode"], "random output winners", tuple(pts[j]))
    return kernel_fwd
