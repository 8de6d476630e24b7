"""Independent restatements used to pin the oracle (test code only).

Nothing here calls the oracle or the CUDA path.  Geometry is obtained by physically
rolling coordinate arrays with numpy and cutting tiles, attention is computed as
*global* attention over all H*W tokens under a membership mask, and the bias is
evaluated from coordinate differences through a callable, not through the oracle's
table-index formula.
"""
import numpy as np


def rolled_geometry(H, W, w, sh, sw, periodic_h, periodic_w):
    """Per grid token: window id and mask label, from an explicit roll of coordinate arrays.

    Returns win[H, W], lab[H, W], a[H, W], b[H, W] (offsets inside the window, shifted frame)."""
    sh, sw = sh % H, sw % W
    uu, vv = np.meshgrid(np.arange(H), np.arange(W), indexing="ij")
    # content moves toward lower index: rolled[u'] = x[(u' + s) mod H]
    ru = np.roll(uu, shift=(-sh, -sw), axis=(0, 1))
    rv = np.roll(vv, shift=(-sh, -sw), axis=(0, 1))
    # region id in the rolled frame: the last s rows / columns came from across the edge
    reg = np.zeros((H, W), dtype=np.int64)
    if not periodic_h and sh > 0:
        reg[H - sh:, :] += 2
    if not periodic_w and sw > 0:
        reg[:, W - sw:] += 1
    Mw = -(-W // w)
    win = np.empty((H, W), dtype=np.int64)
    lab = np.empty((H, W), dtype=np.int64)
    a = np.empty((H, W), dtype=np.int64)
    b = np.empty((H, W), dtype=np.int64)
    for r0 in range(0, H, w):
        for c0 in range(0, W, w):
            tu = ru[r0:r0 + w, c0:c0 + w]
            tv = rv[r0:r0 + w, c0:c0 + w]
            g = (r0 // w) * Mw + (c0 // w)
            for i in range(tu.shape[0]):
                for j in range(tu.shape[1]):
                    win[tu[i, j], tv[i, j]] = g
                    lab[tu[i, j], tv[i, j]] = reg[r0 + i, c0 + j]
                    a[tu[i, j], tv[i, j]] = i
                    b[tu[i, j], tv[i, j]] = j
    return win, lab, a, b


def global_attention(q, k, v, win, lab, a, b, bias_fn, scale):
    """Full H*W x H*W attention with the window-membership mask.

    q, k, v: float64 [H, W, heads, d] (one sample).  bias_fn(da, db, head) -> float64 array, with
    da = a_query - a_key and db = b_query - b_key.  Returns o [H, W, heads, d], lse [H, W, heads],
    p [heads, HW, HW]."""
    H, W, nh, d = q.shape
    N = H * W
    qf, kf, vf = (x.reshape(N, nh, d) for x in (q, k, v))
    winf, labf, af, bf = (x.reshape(N) for x in (win, lab, a, b))
    allowed = (winf[:, None] == winf[None, :]) & (labf[:, None] == labf[None, :])
    da = af[:, None] - af[None, :]
    db = bf[:, None] - bf[None, :]
    o = np.empty((N, nh, d))
    lse = np.empty((N, nh))
    ps = np.empty((nh, N, N))
    for h in range(nh):
        s = scale * (qf[:, h, :] @ kf[:, h, :].T) + bias_fn(da, db, h)
        s = np.where(allowed, s, -np.inf)
        m = s.max(axis=1, keepdims=True)
        e = np.exp(s - m)
        z = e.sum(axis=1, keepdims=True)
        p = e / z
        ps[h] = p
        o[:, h, :] = p @ vf[:, h, :]
        lse[:, h] = (m + np.log(z))[:, 0]
    return o.reshape(H, W, nh, d), lse.reshape(H, W, nh), ps


def table_from_fn(w, heads, bias_fn):
    """Bias table [(2w-1)^2, heads] laid out row = (da + w - 1) * (2w - 1) + (db + w - 1)."""
    t = np.empty(((2 * w - 1) ** 2, heads))
    for da in range(-(w - 1), w):
        for db in range(-(w - 1), w):
            for h in range(heads):
                t[(da + w - 1) * (2 * w - 1) + (db + w - 1), h] = bias_fn(np.array(da), np.array(db), h)
    return t


def random_bias_fn(w, heads, seed):
    """A random table exposed as a function of (da, db, head) via a dict lookup."""
    rng = np.random.default_rng(seed)
    vals = {(da, db, h): rng.normal(0.0, 0.5) for da in range(-(w - 1), w) for db in range(-(w - 1), w)
            for h in range(heads)}

    def fn(da, db, h):
        da = np.asarray(da)
        db = np.asarray(db)
        out = np.zeros(da.shape)
        it = np.nditer(da, flags=["multi_index"]) if da.ndim else None
        if it is None:
            return vals.get((int(da), int(db), h), 0.0)
        for x in it:
            key = (int(x), int(db[it.multi_index]), h)
            out[it.multi_index] = vals.get(key, 0.0)   # pairs in different windows are masked anyway
        return out
    return fn
