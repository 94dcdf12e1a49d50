"""An independent statement of the networks, used only to pin the oracle.

Written with torch.nn.functional (NCHW) and differentiated by autograd; it
shares no code with oracle/.  The whole network's parameters are one flat
vector: the concatenation of the module vectors, i.e. stem, blocks 1..3n, head,
each in its documented order, convolution weights stored [C_out, R, S, C_in].
"""
import torch
import torch.nn.functional as F


class _Reader:
    def __init__(self, theta):
        self.theta, self.off = theta, 0

    def take(self, *shape):
        n = 1
        for s in shape:
            n *= s
        out = self.theta[self.off:self.off + n].reshape(*shape)
        self.off += n
        return out

    def conv(self, co, r, ci):
        return self.take(co, r, r, ci).permute(0, 3, 1, 2)      # -> [co, ci, r, r]


class _Norms:
    """Batch norms in network order.  buffers None: training mode without running statistics.  Otherwise a
    list that is filled with [running_mean, running_var] tensors on first use (zeros / ones, as
    torch.nn.BatchNorm2d starts them) and updated by torch itself in training mode (momentum 0.1), or read
    in inference mode."""

    def __init__(self, buffers, training):
        self.buffers, self.training, self.i = buffers, training, 0

    def __call__(self, x, g, b, eps):
        if self.buffers is None:
            return F.batch_norm(x, None, None, g, b, training=True, momentum=0.0, eps=eps)
        if self.i == len(self.buffers):
            self.buffers.append([torch.zeros(x.shape[1], dtype=x.dtype), torch.ones(x.shape[1], dtype=x.dtype)])
        rm, rv = self.buffers[self.i]
        self.i += 1
        return F.batch_norm(x, rm, rv, g, b, training=self.training, momentum=0.1, eps=eps)


def network_loss(arch, theta, images_nhwc, labels, buffers=None):
    """Mean softmax cross-entropy of the network `arch` with parameters `theta`
    (1-D torch tensor) on one batch.  images_nhwc: [B,H,W,C] tensor."""
    return F.cross_entropy(network_logits(arch, theta, images_nhwc, buffers, True), labels.long())


def network_logits(arch, theta, images_nhwc, buffers=None, training=True):
    _bn = _Norms(buffers, training)
    rd = _Reader(theta)
    eps = arch.bn_eps
    x = images_nhwc.permute(0, 3, 1, 2)
    wrn = arch.family == "wrn"
    x = F.conv2d(x, rd.conv(arch.stem_width, 3, arch.in_c), padding=1)
    if not wrn:
        x = F.relu(_bn(x, rd.take(arch.stem_width), rd.take(arch.stem_width), eps))
    ci = arch.stem_width
    for stage, n_blocks in enumerate(arch.stage_blocks()):
        co = arch.widths[stage]
        for j in range(n_blocks):
            stride = 2 if (stage > 0 and j == 0) else 1
            proj = ci != co or stride != 1
            if not wrn:
                w1 = rd.conv(co, 3, ci); g1 = rd.take(co); b1 = rd.take(co)
                w2 = rd.conv(co, 3, co); g2 = rd.take(co); b2 = rd.take(co)
                h = F.relu(_bn(F.conv2d(x, w1, stride=stride, padding=1), g1, b1, eps))
                h = _bn(F.conv2d(h, w2, padding=1), g2, b2, eps)
                if proj and arch.shortcut == "zero_pad":
                    lo = (co - ci) // 2
                    sc = F.pad(x[:, :, ::stride, ::stride], (0, 0, 0, 0, lo, co - ci - lo))
                elif proj:
                    ws = rd.conv(co, 1, ci); gs = rd.take(co); bs = rd.take(co)
                    sc = _bn(F.conv2d(x, ws, stride=stride), gs, bs, eps)
                else:
                    sc = x
                x = F.relu(h + sc)
            else:
                g1 = rd.take(ci); b1 = rd.take(ci); w1 = rd.conv(co, 3, ci)
                g2 = rd.take(co); b2 = rd.take(co); w2 = rd.conv(co, 3, co)
                o = F.relu(_bn(x, g1, b1, eps))
                h = F.conv2d(o, w1, stride=stride, padding=1)
                h = F.conv2d(F.relu(_bn(h, g2, b2, eps)), w2, padding=1)
                if proj:
                    sc = F.conv2d(o, rd.conv(co, 1, ci), stride=stride)
                else:
                    sc = x
                x = h + sc
            ci = co
    if wrn:
        x = F.relu(_bn(x, rd.take(ci), rd.take(ci), eps))
    x = x.mean(dim=(2, 3))
    logits = F.linear(x, rd.take(arch.num_classes, ci), rd.take(arch.num_classes))
    assert rd.off == theta.numel(), (rd.off, theta.numel())
    return logits


def loss_and_grad(arch, theta_np, images_np, labels_np):
    theta = torch.tensor(theta_np, dtype=torch.float64, requires_grad=True)
    loss = network_loss(arch, theta, torch.tensor(images_np, dtype=torch.float64),
                        torch.tensor(labels_np))
    (g,) = torch.autograd.grad(loss, theta)
    return float(loss.detach()), g.numpy()
