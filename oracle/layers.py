"""CPU oracle, part 1: the layer mathematics.

TEST INFRASTRUCTURE ONLY.  Nothing in the product path (the CUDA library and its
Python binding) imports, links or calls this file; only the tests, the smoke
check and the cpu-baseline leg of the benchmark do.

The FDG paper treats a layer as an abstract map z_l = A_l(z_{l-1}; theta_l)
(Background section, the paragraph before Eq. 1) and back-propagates through it
with the chain rule (Eq. 8, Eq. 9).  It defines no layer of its own: its
experiments use the standard residual CNNs it cites.  The functions below are
therefore the textbook definitions of those layers written out directly, each
with its derivative, in plain numpy.  Layout is NHWC for activations and
[C_out, R, S, C_in] for convolution weights.  The only library primitive used
as a step is a matrix product (one per filter tap); there is no blocking,
fusion or reordering.

Pins (tests/test_oracle_layers.py): central finite differences in fp64 for every
function here, and agreement with the corresponding torch.nn.functional routine
differentiated by autograd.
"""
import numpy as np


# ----------------------------------------------------------------------------
# storage precision
# ----------------------------------------------------------------------------
def round_bf16(a):
    """Rounds every element to the nearest bfloat16 (8 exponent bits, 7 stored mantissa
    bits; ties to even) and returns it in the dtype it came in.

    The paper fixes no precision.  Where a tensor is held in bfloat16 between two
    steps of the path, the decisions taken on it (the sign test of a ReLU gate)
    depend on that rounding, so the oracle can reproduce it: bfloat16 is the upper
    half of an IEEE float32 word, and rounding adds half a unit of the dropped
    half (plus the tie-break bit) before truncating.  Pin: agreement with
    torch.Tensor.to(torch.bfloat16) on random and boundary values.
    """
    a = np.asarray(a)
    bits = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    keep = (bits >> np.uint32(16)) & np.uint32(1)
    bits = (bits + np.uint32(0x7FFF) + keep) & np.uint32(0xFFFF0000)
    return bits.view(np.float32).astype(a.dtype).reshape(a.shape)


def identity(a):
    return a


# ----------------------------------------------------------------------------
# convolution (cross-correlation, zero padding, no bias)
# ----------------------------------------------------------------------------
def conv_out_size(n, r, stride, pad):
    return (n + 2 * pad - r) // stride + 1


def conv2d_forward(x, w, stride, pad):
    """y[n,p,q,o] = sum_{r,s,i} xpad[n, p*stride+r, q*stride+s, i] * w[o,r,s,i]."""
    n, h, wd, ci = x.shape
    co, r_, s_, ci2 = w.shape
    assert ci == ci2
    oh = conv_out_size(h, r_, stride, pad)
    ow = conv_out_size(wd, s_, stride, pad)
    xp = np.zeros((n, h + 2 * pad, wd + 2 * pad, ci), dtype=x.dtype)
    xp[:, pad:pad + h, pad:pad + wd, :] = x
    y = np.zeros((n, oh, ow, co), dtype=x.dtype)
    for r in range(r_):
        for s in range(s_):
            patch = xp[:, r:r + stride * oh:stride, s:s + stride * ow:stride, :]
            y += patch @ w[:, r, s, :].T
    return y


def conv2d_backward(dy, x, w, stride, pad):
    """Derivatives of conv2d_forward: returns (dx, dw).

    dw[o,r,s,i] = sum_{n,p,q} dy[n,p,q,o] * xpad[n, p*stride+r, q*stride+s, i]
    dxpad[n, p*stride+r, q*stride+s, i] += sum_o dy[n,p,q,o] * w[o,r,s,i]
    """
    n, h, wd, ci = x.shape
    co, r_, s_, _ = w.shape
    _, oh, ow, _ = dy.shape
    xp = np.zeros((n, h + 2 * pad, wd + 2 * pad, ci), dtype=x.dtype)
    xp[:, pad:pad + h, pad:pad + wd, :] = x
    dxp = np.zeros_like(xp)
    dw = np.zeros_like(w)
    dy2 = dy.reshape(-1, co)
    for r in range(r_):
        for s in range(s_):
            patch = xp[:, r:r + stride * oh:stride, s:s + stride * ow:stride, :]
            dw[:, r, s, :] = dy2.T @ patch.reshape(-1, ci)
            dxp[:, r:r + stride * oh:stride, s:s + stride * ow:stride, :] += dy @ w[:, r, s, :]
    dx = dxp[:, pad:pad + h, pad:pad + wd, :].copy()
    return dx, dw


# ----------------------------------------------------------------------------
# batch normalisation, training mode (statistics of the current batch)
# ----------------------------------------------------------------------------
def batchnorm_forward(x, gamma, beta, eps):
    """Per-channel: xhat = (x - mean) / sqrt(var + eps), y = gamma*xhat + beta.

    mean and var (biased, divisor = number of elements per channel) are taken
    over batch and spatial positions.  Returns y and (xhat, invstd) for the
    backward pass.
    """
    mean = x.mean(axis=(0, 1, 2))
    var = ((x - mean) ** 2).mean(axis=(0, 1, 2))
    invstd = 1.0 / np.sqrt(var + x.dtype.type(eps))
    xhat = (x - mean) * invstd
    y = gamma * xhat + beta
    return y, (xhat, invstd)


def batchnorm_backward(dy, saved, gamma):
    """Derivative of batchnorm_forward, statistics included in the chain rule.

    dbeta = sum dy ; dgamma = sum dy*xhat ;
    dx = gamma*invstd * (dy - dbeta/M - xhat*dgamma/M),  M = elements per channel.
    """
    xhat, invstd = saved
    m = dy.shape[0] * dy.shape[1] * dy.shape[2]
    dbeta = dy.sum(axis=(0, 1, 2))
    dgamma = (dy * xhat).sum(axis=(0, 1, 2))
    dx = (gamma * invstd) * (dy - dbeta / m - xhat * (dgamma / m))
    return dx, dgamma, dbeta


def batchnorm_running_update(running, x, momentum=0.1):
    """Running statistics kept beside a training-mode batch norm for later inference.

    The paper reports test errors (Tables 3-6), so its networks normalise test batches with
    statistics gathered during training; it does not say how.  Reading taken: the exponential
    running average of the framework its experiments ran on, momentum 0.1, started at mean 0 /
    variance 1, fed with the batch mean and the UNBIASED batch variance (divisor M - 1):
        running <- (1 - momentum) * running + momentum * batch statistic.
    `running` = [mean, var], updated in place.
    """
    m = x.shape[0] * x.shape[1] * x.shape[2]
    mean = x.mean(axis=(0, 1, 2))
    var = ((x - mean) ** 2).sum(axis=(0, 1, 2)) / (m - 1)
    running[0][:] = (1.0 - momentum) * running[0] + momentum * mean
    running[1][:] = (1.0 - momentum) * running[1] + momentum * var


def batchnorm_eval(x, gamma, beta, running, eps):
    """Inference-mode batch norm: y = gamma * (x - running mean) / sqrt(running var + eps) + beta."""
    return gamma * ((x - running[0]) / np.sqrt(running[1] + x.dtype.type(eps))) + beta


# ----------------------------------------------------------------------------
# ReLU
# ----------------------------------------------------------------------------
def relu_forward(x):
    return np.maximum(x, 0)


def relu_backward(dy, y):
    """y is the ReLU output; the derivative at exactly 0 is taken as 0."""
    return dy * (y > 0)


# ----------------------------------------------------------------------------
# head: global average pool, fully connected layer, softmax cross-entropy
# ----------------------------------------------------------------------------
def gap_forward(x):
    return x.mean(axis=(1, 2))


def gap_backward(dy, shape):
    n, h, w, c = shape
    return np.broadcast_to(dy[:, None, None, :] / (h * w), shape).astype(dy.dtype)


def fc_forward(x, w, b):
    """x [N, F], w [classes, F], b [classes]."""
    return x @ w.T + b


def fc_backward(dy, x, w):
    dx = dy @ w
    dw = dy.T @ x
    db = dy.sum(axis=0)
    return dx, dw, db


def softmax_xent_forward(logits, labels):
    """Mean over the batch of -log softmax(logits)[label]; returns (loss, probs)."""
    z = logits - logits.max(axis=1, keepdims=True)
    e = np.exp(z)
    p = e / e.sum(axis=1, keepdims=True)
    n = logits.shape[0]
    loss = -np.log(p[np.arange(n), labels]).mean()
    return loss, p


def softmax_xent_backward(probs, labels):
    n = probs.shape[0]
    d = probs.copy()
    d[np.arange(n), labels] -= 1
    return d / n
