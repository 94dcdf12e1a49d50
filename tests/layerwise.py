"""Layer-by-layer check of one backward pass of every module of a 6n+2 network against the oracle's layer
functions (oracle/layers.py), used by the full-size test and by the smoke check.

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
            for which in ((0, 3) if name == "stem" else (0, 1, 2, 3) + ((4,) if len(ent) > 6 else ())):
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
                feat = int(ent[0][1][1])
                hwl = int(round((saved[(k, u - 1, 3)].size / (b * feat)) ** 0.5))
                ylast = saved[(k, u - 1, 3)].reshape(b, hwl, hwl, feat).astype(np.float64)
                wfc, bfc = _take(flat, ent[0]), _take(flat, ent[1])
                pooled = L.gap_forward(ylast)
                loss, probs = L.softmax_xent_forward(L.fc_forward(pooled, wfc, bfc), S.labels(seed, k, b, classes).astype(np.int64))
                dpool, dwo, dbo = L.fc_backward(L.softmax_xent_backward(probs, S.labels(seed, k, b, classes).astype(np.int64)), pooled, wfc)
                cmp("head.dx", cap(u - 1, 0, ylast.shape), q(L.gap_backward(dpool, ylast.shape)), where)
                cmp("fc.dw", _take(grads, ent[0]), dwo, where, 1e-4)
                cmp("fc.db", _take(grads, ent[1]), dbo, where, 1e-4)
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
