"""Layer-by-layer check of one backward pass of every module of a network (post-activation 6n+2 / ResNet-18 blocks,
or the pre-activation blocks of the wide residual networks) against the oracle's layer functions
(oracle/layers.py), used by the full-size test, the architecture tests and the smoke check.

A capture (fdg_capture_begin) keeps every gradient tensor of each module's backward pass at iteration 2K - 1,
the first one in which all K modules back-propagate (module k then handles batch k).  Every layer of every
block is recomputed by the oracle from the library's own inputs to that layer -- the incoming gradient it
captured and the activations it saved for that batch, so every ReLU gate is the same on both sides -- and
compared element by element."""
import numpy as np

import fdg_synth as S
from oracle import layers as L

EPS = 1e-5


def _relmax(a, b):
    return float(np.abs(a - b).max() / max(np.abs(b).max(), 1e-30))


def units_of(layout):
    """[(unit name, [(offset, shape)] in unit order)] in module order."""
    units = []
    for name, kind, shape in layout:
        unit, off = name.split("@")
        if not units or units[-1][0] != unit:
            units.append((unit, []))
        units[-1][1].append((int(off), tuple(shape)))
    return units


def take(flat, entry):
    off, shape = entry
    return flat[off:off + int(np.prod(shape))].reshape(shape).astype(np.float64)


def check_backward_layerwise(g, params, arch, K, seed=0, tol=1e-2):
    """`g`: a context with lr = 0 and weight decay 0 (weights stay as set), bf16 storage, not yet stepped, created
    without graphs; `params`: {module: flat parameters}.  Returns (blocks checked, worst error per kind of tensor)."""
    import torch
    b, hw0, classes = arch["batch"], arch["in_h"], arch["num_classes"]
    _units, _take = units_of, take
    T = 2 * K - 1

    def step(t):
        x = torch.from_numpy(S.images(seed, t, b, hw0, hw0, 3)).cuda()
        y = torch.from_numpy(S.labels(seed, t, b, classes)).cuda()
        g.step(x, y)
    for t in range(1, T):
        step(t)
    g.sync()
    # Modules k < K back-propagate batch k at iteration T and then forward a new batch into the slot they free,
    # so what they saved for batch k is read now; the top module forwards and back-propagates batch K at T itself.
    saved = {}

    def fetch(k):
        units = _units(g.param_layout(k))
        for u, (name, ent) in enumerate(units):
            if name == "head":
                continue
            preact = len(ent[0][1]) == 1                             # a pre-activation block starts with a batch norm
            if name == "stem":
                want = (0, 3) if len(ent) > 1 else (3,)              # the wide networks' stem is a bare convolution
            else:
                want = (0, 1, 2, 3) + ((4,) if (len(ent) > 6 and not preact) else ())
            for which in want:
                bb, a = g.saved_tensor_of(k, u, which, k)
                assert bb == k, (k, u, which, bb)
                saved[(k, u, which)] = a

    for k in range(1, K):
        fetch(k)
    for k in range(1, K + 1):
        g.capture_begin(k)
    step(T)
    g.sync()
    fetch(K)
    worst = {}
    checked = 0

    def cmp(key, got, want, where, tol=tol):
        err = _relmax(np.asarray(got, dtype=np.float64).reshape(-1), np.asarray(want, dtype=np.float64).reshape(-1))
        worst[key] = max(worst.get(key, 0.0), err)
        assert err <= tol, (where, key, err)

    q = L.round_bf16
    for k in range(1, K + 1):
        units = _units(g.param_layout(k))
        flat, grads = params[k], g.get_grads(k)

        def cap(u, which, shape):
            bb, a = g.captured(k, u, which)
            assert bb == k, (k, u, which, bb)
            return a.reshape(shape).astype(np.float64)

        for u, (name, ent) in enumerate(units):
            where = (k, name)
            if name == "head":
                with_bn = len(ent) == 4                              # wide networks: batch norm + ReLU before the pooling
                efc = ent[2:] if with_bn else ent
                feat = int(efc[0][1][1])
                hwl = int(round((saved[(k, u - 1, 3)].size / (b * feat)) ** 0.5))
                ylast = saved[(k, u - 1, 3)].reshape(b, hwl, hwl, feat).astype(np.float64)
                wfc, bfc = _take(flat, efc[0]), _take(flat, efc[1])
                labels = S.labels(seed, k, b, classes).astype(np.int64)
                if with_bn:
                    gh, bh = _take(flat, ent[0]), _take(flat, ent[1])
                    bno, svh = L.batchnorm_forward(ylast, gh, bh, EPS)
                    feat_in = q(L.relu_forward(bno))
                else:
                    feat_in = ylast
                pooled = L.gap_forward(feat_in)
                loss, probs = L.softmax_xent_forward(L.fc_forward(pooled, wfc, bfc), labels)
                dpool, dwo, dbo = L.fc_backward(L.softmax_xent_backward(probs, labels), pooled, wfc)
                dfeat = q(L.gap_backward(dpool, ylast.shape))
                if with_bn:
                    dyl, dgh, dbh = L.batchnorm_backward(L.relu_backward(dfeat, feat_in), svh, gh)
                    cmp("head.dx", cap(u - 1, 0, ylast.shape), q(dyl), where)
                    cmp("head.bn.dgamma", _take(grads, ent[0]), dgh, where, 1e-3)
                    cmp("head.bn.dbeta", _take(grads, ent[1]), dbh, where, 1e-3)
                else:
                    cmp("head.dx", cap(u - 1, 0, ylast.shape), dfeat, where)
                cmp("fc.dw", _take(grads, efc[0]), dwo, where, 1e-3 if with_bn else 1e-4)
                cmp("fc.db", _take(grads, efc[1]), dbo, where, 1e-3 if with_bn else 1e-4)
                continue
            if name == "stem" and len(ent) == 1:                     # a bare convolution: only its weight gradient
                w1 = q(_take(flat, ent[0]))
                x_in = q(S.images(seed, k, b, hw0, hw0, 3).astype(np.float64))
                dy = cap(u, 0, (b, hw0, hw0, w1.shape[0]))
                cmp("stem.dw", _take(grads, ent[0]), L.conv2d_backward(dy, x_in, w1, 1, 1)[1], where)
                continue
            if len(ent[0][1]) == 1:
                _check_preact(k, u, ent, flat, grads, saved, cap, cmp, q, g, b, where, _units, _take)
                checked += 1
                continue
            if name == "stem":
                w1 = q(_take(flat, ent[0])); g1, b1 = _take(flat, ent[1]), _take(flat, ent[2])
                co = w1.shape[0]
                x_in = q(S.images(seed, k, b, hw0, hw0, 3).astype(np.float64))
                c = saved[(k, u, 0)].reshape(b, hw0, hw0, co).astype(np.float64)
                y = saved[(k, u, 3)].reshape(c.shape).astype(np.float64)
                dy = cap(u, 0, c.shape)
                dc_o, dg_o, db_o = L.batchnorm_backward(L.relu_backward(dy, y), L.batchnorm_forward(c, g1, b1, EPS)[1], g1)
                dc = cap(u, 3, c.shape)
                cmp("stem.dc", dc, q(dc_o), where)
                cmp("stem.dgamma", _take(grads, ent[1]), dg_o, where)
                cmp("stem.dbeta", _take(grads, ent[2]), db_o, where)
                cmp("stem.dw", _take(grads, ent[0]), L.conv2d_backward(dc, x_in, w1, 1, 1)[1], where)
                continue
            w1 = q(_take(flat, ent[0])); g1, b1 = _take(flat, ent[1]), _take(flat, ent[2])
            w2 = q(_take(flat, ent[3])); g2, b2 = _take(flat, ent[4]), _take(flat, ent[5])
            co, ci = w1.shape[0], w1.shape[3]
            proj = len(ent) > 6
            stride = 2 if proj else 1
            x_flat = saved[(k, u - 1, 3)] if u > 0 else g.saved_tensor_of(k - 1, len(_units(g.param_layout(k - 1))) - 1, 3, k)[1]
            hw_in = int(round((x_flat.size / (b * ci)) ** 0.5))
            x_in = x_flat.reshape(b, hw_in, hw_in, ci).astype(np.float64)
            hw = hw_in // stride
            shp = (b, hw, hw, co)
            c1, a1, c2, y = (saved[(k, u, i)].reshape(shp).astype(np.float64) for i in range(4))
            dy = cap(u, 0, shp)
            dsum = L.relu_backward(dy, y)
            dc2_o, dg2_o, db2_o = L.batchnorm_backward(dsum, L.batchnorm_forward(c2, g2, b2, EPS)[1], g2)
            dc2 = cap(u, 1, shp)
            cmp("dc2", dc2, q(dc2_o), where)
            cmp("bn2.dgamma", _take(grads, ent[4]), dg2_o, where)
            cmp("bn2.dbeta", _take(grads, ent[5]), db2_o, where)
            da1_o, dw2_o = L.conv2d_backward(dc2, a1, w2, 1, 1)
            da1 = cap(u, 2, shp)
            cmp("da1", da1, q(da1_o), where)
            cmp("conv2.dw", _take(grads, ent[3]), dw2_o, where)
            dc1_o, dg1_o, db1_o = L.batchnorm_backward(L.relu_backward(da1, a1), L.batchnorm_forward(c1, g1, b1, EPS)[1], g1)
            dc1 = cap(u, 3, shp)
            cmp("dc1", dc1, q(dc1_o), where)
            cmp("bn1.dgamma", _take(grads, ent[1]), dg1_o, where)
            cmp("bn1.dbeta", _take(grads, ent[2]), db1_o, where)
            dx_o, dw1_o = L.conv2d_backward(dc1, x_in, w1, stride, 1)
            cmp("conv1.dw", _take(grads, ent[0]), dw1_o, where)
            if proj:
                ws = q(_take(flat, ent[6])); gs, bs = _take(flat, ent[7]), _take(flat, ent[8])
                cs = saved[(k, u, 4)].reshape(shp).astype(np.float64)
                dcs_o, dgs_o, dbs_o = L.batchnorm_backward(dsum, L.batchnorm_forward(cs, gs, bs, EPS)[1], gs)
                dcs = cap(u, 5, shp)
                cmp("dcs", dcs, q(dcs_o), where)
                cmp("scbn.dgamma", _take(grads, ent[7]), dgs_o, where)
                cmp("scbn.dbeta", _take(grads, ent[8]), dbs_o, where)
                dxs_o, dws_o = L.conv2d_backward(dcs, x_in, ws, stride, 0)
                cmp("sc.dw", _take(grads, ent[6]), dws_o, where)
                dx_o = dx_o + q(dxs_o)
            else:
                dx_o = dx_o + dsum
            cmp("dx", cap(u, 4, x_in.shape), q(dx_o), where)
            checked += 1
    for k in range(1, K + 1):
        g.capture_end(k)
    return checked, worst


def _check_preact(k, u, ent, flat, grads, saved, cap, cmp, q, g, b, where, _units, _take):
    """One pre-activation block: o = relu(bn1(x)), c1 = conv1(o), a2 = relu(bn2(c1)), y = conv2(a2) + shortcut, the
    shortcut being x or a 1x1 convolution of o.  Saved: o, c1, a2, y.  Captured: dy, da2, dc1, do (+ the shortcut's
    share), dx, and the shortcut's share alone."""
    g1, b1 = _take(flat, ent[0]), _take(flat, ent[1])
    w1 = q(_take(flat, ent[2]))
    g2, b2 = _take(flat, ent[3]), _take(flat, ent[4])
    w2 = q(_take(flat, ent[5]))
    proj = len(ent) > 6
    co, ci = w1.shape[0], w1.shape[3]
    x_flat = saved[(k, u - 1, 3)] if u > 0 else g.saved_tensor_of(k - 1, len(_units(g.param_layout(k - 1))) - 1, 3, k)[1]
    hw_in = int(round((x_flat.size / (b * ci)) ** 0.5))
    x_in = x_flat.reshape(b, hw_in, hw_in, ci).astype(np.float64)
    hw = int(round((saved[(k, u, 3)].size / (b * co)) ** 0.5))
    stride = hw_in // hw
    shp = (b, hw, hw, co)
    o = saved[(k, u, 0)].reshape(x_in.shape).astype(np.float64)
    c1, a2 = (saved[(k, u, i)].reshape(shp).astype(np.float64) for i in (1, 2))
    dy = cap(u, 0, shp)
    da2_o, dw2_o = L.conv2d_backward(dy, a2, w2, 1, 1)
    da2 = cap(u, 1, shp)
    cmp("da2", da2, q(da2_o), where)
    cmp("conv2.dw", _take(grads, ent[5]), dw2_o, where)
    dc1_o, dg2_o, db2_o = L.batchnorm_backward(L.relu_backward(da2, a2), L.batchnorm_forward(c1, g2, b2, EPS)[1], g2)
    dc1 = cap(u, 2, shp)
    cmp("dc1", dc1, q(dc1_o), where)
    cmp("bn2.dgamma", _take(grads, ent[3]), dg2_o, where)
    cmp("bn2.dbeta", _take(grads, ent[4]), db2_o, where)
    do_o, dw1_o = L.conv2d_backward(dc1, o, w1, stride, 1)
    cmp("conv1.dw", _take(grads, ent[2]), dw1_o, where)
    if proj:
        ws = q(_take(flat, ent[6]))
        dos_o, dws_o = L.conv2d_backward(dy, o, ws, stride, 0)
        dos = cap(u, 5, x_in.shape)
        cmp("dos", dos, q(dos_o), where)
        cmp("sc.dw", _take(grads, ent[6]), dws_o, where)
        do_o = do_o + dos
    do = cap(u, 3, x_in.shape)
    cmp("do", do, q(do_o), where)
    dx_o, dg1_o, db1_o = L.batchnorm_backward(L.relu_backward(do, o), L.batchnorm_forward(x_in, g1, b1, EPS)[1], g1)
    if not proj:
        dx_o = dx_o + dy
    cmp("dx", cap(u, 4, x_in.shape), q(dx_o), where)
    cmp("bn1.dgamma", _take(grads, ent[0]), dg1_o, where)
    cmp("bn1.dbeta", _take(grads, ent[1]), db1_o, where)


def check_forward_layerwise_preact(g, params, arch, K, seed=0, tol=1e-2):
    """Forward twin for the pre-activation family: after K iterations every module has forwarded one batch (module k
    batch 1 at iteration k).  Every layer of every block -- batch norm + ReLU, the 3x3 convolutions, the shortcut and
    the residual sum -- is recomputed by the oracle from what the library saved as that layer's input and compared
    with what it saved as the layer's output.  Returns (blocks checked, worst error per kind of tensor)."""
    import torch
    b, hw0, classes = arch["batch"], arch["in_h"], arch["num_classes"]
    for t in range(1, K + 1):
        g.step(torch.from_numpy(S.images(seed, t, b, hw0, hw0, 3)).cuda(), torch.from_numpy(S.labels(seed, t, b, classes)).cuda())
    g.sync()
    q = L.round_bf16
    worst, checked = {}, 0

    def cmp(key, got, want, where):
        err = _relmax(np.asarray(got, dtype=np.float64).reshape(-1), np.asarray(want, dtype=np.float64).reshape(-1))
        worst[key] = max(worst.get(key, 0.0), err)
        assert err <= tol, (where, key, err)

    x_prev = None                                                    # output of the unit before, as the library saved it
    for k in range(1, K + 1):
        units = units_of(g.param_layout(k))
        flat = params[k]
        for u, (name, ent) in enumerate(units):
            if name == "head":
                continue
            if name == "stem":
                w1 = q(take(flat, ent[0]))
                x_in = q(S.images(seed, 1, b, hw0, hw0, 3).astype(np.float64))
                y = g.saved_tensor_of(k, u, 3, 1)[1].reshape(b, hw0, hw0, w1.shape[0]).astype(np.float64)
                cmp("stem.y", y, q(L.conv2d_forward(x_in, w1, 1, 1)), (k, name))
                x_prev = y
                continue
            g1, b1 = take(flat, ent[0]), take(flat, ent[1])
            w1 = q(take(flat, ent[2]))
            g2, b2 = take(flat, ent[3]), take(flat, ent[4])
            w2 = q(take(flat, ent[5]))
            proj = len(ent) > 6
            co, ci = w1.shape[0], w1.shape[3]
            hw_in = int(round((x_prev.size / (b * ci)) ** 0.5))
            x_in = x_prev.reshape(b, hw_in, hw_in, ci)
            o = g.saved_tensor_of(k, u, 0, 1)[1].reshape(x_in.shape).astype(np.float64)
            ysz = g.saved_tensor_of(k, u, 3, 1)[1]
            hw = int(round((ysz.size / (b * co)) ** 0.5))
            stride = hw_in // hw
            shp = (b, hw, hw, co)
            c1, a2 = (g.saved_tensor_of(k, u, i, 1)[1].reshape(shp).astype(np.float64) for i in (1, 2))
            y = ysz.reshape(shp).astype(np.float64)
            where = (k, name)
            cmp("o", o, q(L.relu_forward(L.batchnorm_forward(x_in, g1, b1, EPS)[0])), where)
            cmp("c1", c1, q(L.conv2d_forward(o, w1, stride, 1)), where)
            cmp("a2", a2, q(L.relu_forward(L.batchnorm_forward(c1, g2, b2, EPS)[0])), where)
            sc = q(L.conv2d_forward(o, q(take(flat, ent[6])), stride, 0)) if proj else x_in
            cmp("y", y, q(L.conv2d_forward(a2, w2, 1, 1) + sc), where)
            x_prev = y
            checked += 1
    return checked, worst
