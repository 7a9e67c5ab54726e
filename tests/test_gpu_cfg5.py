"""Benchmark configuration 5: one training step of the ResNet-18-shaped hybrid network
(N=64, 224x224, every 3x3 convolution of stages 2-4 a tropical layer computing in bf16).

Three tropical layers are captured during the step (the stride-2 layer of stage 2, a 256-channel
14x14 layer, a 512-channel 7x7 layer) and checked against the CPU oracle on a sample; the logits
of the whole network are compared with the same network evaluated through the paper's unfold
formulation in torch."""
import numpy as np
import pytest
import torch

from paper_2504_06881_b200 import inputs, tconv
from paper_2504_06881_b200.nn import HybridResNet18, TropicalConv2d
import parity
import unfold_torch

pytestmark = pytest.mark.gpu


def _layer_desc(m, x):
    N, C, H, W = x.shape
    return inputs.layer(N, C, H, W, m.out_channels, 3, 3, stride=m.stride, pad=m.padding, dil=m.dilation,
                        mode=m.mode, chan=m.chan, dtype=m.dtype)


@pytest.mark.parametrize("mode", ["compound", "parallel"])
def test_resnet18_hybrid_training_step(mode):
    torch.manual_seed(1050)
    rs = np.random.RandomState(1050)
    N = 64
    net = HybridResNet18(mode=mode, dtype="bf16").cuda()
    x = torch.from_numpy(rs.standard_normal((N, 3, 224, 224)).astype(np.float32)).cuda()
    labels = torch.from_numpy(rs.randint(0, 1000, N)).cuda()
    opt = torch.optim.SGD(net.parameters(), lr=0.01, momentum=0.9)
    watch = {"layer2.0.conv1": net.layer2[0].conv1, "layer3.1.conv1": net.layer3[1].conv1,
             "layer4.1.conv2": net.layer4[1].conv2}
    cap = {}
    hooks = []
    for name, m in watch.items():
        hooks.append(m.register_forward_hook(lambda mod, inp, out, name=name: cap.setdefault(name, {}).update(
            x=inp[0].detach().clone())))
        hooks.append(m.register_full_backward_hook(lambda mod, gin, gout, name=name: cap[name].update(
            g=gout[0].detach().clone())))
    before = [p.detach().clone() for p in net.parameters()]
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    logits = net(x)
    loss = torch.nn.functional.cross_entropy(logits, labels)
    opt.zero_grad()
    loss.backward()
    opt.step()
    t1.record()
    torch.cuda.synchronize()
    for h in hooks:
        h.remove()
    assert torch.isfinite(loss).item()
    assert tconv.tconv_device_status() == 0
    # every parameter received a finite gradient and moved
    for p, b in zip(net.parameters(), before):
        assert p.grad is not None and torch.isfinite(p.grad).all()
    assert any(not torch.equal(p.detach(), b) for p, b in zip(net.parameters(), before))
    print(f"\ncfg5 {mode}: first step {t0.elapsed_time(t1):.1f} ms, loss {loss.item():.4f}")

    # captured layers against the oracle (weights as they were during the step)
    for (name, m), k_slice in zip(watch.items(), ((0, 4), (250, 254), (508, 512))):
        c = cap[name]
        d = _layer_desc(m, c["x"])
        named = dict(zip([n_ for n_, _ in net.named_parameters()], before))
        t = {"x": inputs.to_bf16_values(c["x"].float().cpu().numpy()),
             "w": inputs.to_bf16_values(named[name + ".weight"].cpu().numpy()),
             "w2": inputs.to_bf16_values(named[name + ".weight2"].cpu().numpy()) if mode == "parallel"
             else np.zeros(tuple(named[name + ".weight"].shape), np.float32),
             "alpha": named[name + ".alpha"].cpu().numpy().astype(np.float32),
             "beta": named[name + ".beta"].cpu().numpy().astype(np.float32),
             "bias": np.zeros(d["K"], np.float32),
             "g": inputs.to_bf16_values(c["g"].float().cpu().numpy())}
        parity.sampled_check(d, t, sample_n=(3, N - 1), sample_k=k_slice)

    # whole network through the unfold formulation: same logits within bf16 tolerance
    net.eval()
    with torch.no_grad():
        xs = x[:8]
        ours = net(xs).float()
        saved = TropicalConv2d.forward

        def unfold_forward(self, inp):
            xb = inp.to(torch.bfloat16)
            w = self.weight.to(torch.bfloat16)
            w2 = self.weight2.to(torch.bfloat16) if self.weight2 is not None else None
            y = unfold_torch.tropical_unfold(xb, w, w2, self.alpha.float(), self.beta.float(), self.stride[0],
                                             self.padding[0], self.dilation[0])
            return y.to(torch.bfloat16).to(inp.dtype)

        TropicalConv2d.forward = unfold_forward
        try:
            ref = net(xs).float()
        finally:
            TropicalConv2d.forward = saved
    scale = ref.abs().max().item()
    assert (ours - ref).abs().max().item() <= 2e-2 * scale + 1e-3, ((ours - ref).abs().max().item(), scale)
