"""The end-to-end networks evaluated with the CPU checker only (TEST INFRASTRUCTURE: used by the
tests and by the bench's CPU-baseline leg, never by the CUDA library): the same layer graphs as the
CUDA drivers, written independently on top of oracle/oracle.py."""
import numpy as np

from oracle import oracle as orc


def _prep(W, ratio, bits, clip):
    S = orc.num_splits(W.shape[1], ratio)
    Wp, idx, _, _ = orc.split(W, S, 0.0)
    alpha = orc.clip_mse(Wp, bits, True, 2048, 128)["alpha"] if clip == "mse" else orc.maxabs(Wp)
    codes, scale = orc.quantize(Wp, bits, True, alpha)
    return codes, scale, idx


def _qact(x, signed, bits=8):
    return orc.quantize(x, bits, signed, orc.maxabs(x))


def resnet50(cfg):
    """-> (logits, {name: tensor}) for cfg from configs.config4."""
    t = {}
    x = orc.nchw_to_nhwc(cfg["X"])
    first = True
    for spec in cfg["layers"]:
        W, bias = cfg["params"][spec.name]
        codes, ws, idx = _prep(W, cfg["ratio"], cfg["w_bits"], cfg["clip"])
        src = t[spec.input_from] if spec.input_from else x
        xc, xs = _qact(src, signed=first)
        y, _ = orc.qconv(xc, first, xs, codes, ws, idx, spec.stride, spec.pad, bias)
        if spec.residual_from:
            y = orc.add_relu(y, t[spec.residual_from], spec.relu)
            t[spec.name.rsplit(".", 1)[0] + ".out"] = y
        elif spec.relu:
            y = orc.relu(y)
        t[spec.name] = y
        x = y
        if first:
            x = orc.maxpool3x3s2(y)
            t["pool"] = x
            first = False
    feat = orc.global_avgpool(x)
    t["avgpool"] = feat
    W, bias = cfg["params"]["fc"]
    codes, ws, idx = _prep(W.reshape(W.shape[0], W.shape[1]), cfg["ratio"], cfg["w_bits"], cfg["clip"])
    fc_c, fc_s = _qact(feat, signed=False)
    logits, _ = orc.qlinear(fc_c, False, fc_s, codes, ws, idx, bias)
    t["fc"] = logits
    return logits, t


def lstm(cfg):
    """-> (logits [seq*batch, vocab], dict(tops, c)) for cfg from configs.config5."""
    p, hidden = cfg["params"], cfg["hidden"]
    tokens = cfg["tokens"]
    seq, batch = tokens.shape
    q = {}
    for l in range(2):
        for nm in ("W_ih", "W_hh"):
            q[f"{nm}{l}"] = _prep(p[f"{nm}{l}"], cfg["ratio"], cfg["w_bits"], cfg["clip"])
    q["W_dec"] = _prep(p["W_dec"], cfg["ratio"], cfg["w_bits"], cfg["clip"])

    def lin(name, bias, x):
        codes, ws, idx = q[name]
        xc, xs = _qact(x, signed=True)
        return orc.qlinear(xc, True, xs, codes, ws, idx, bias)[0]

    emb = p["emb"][tokens]            # lookup
    h = [np.zeros((batch, hidden), np.float32) for _ in range(2)]
    c = [np.zeros((batch, hidden), np.float32) for _ in range(2)]
    tops = np.empty((seq, batch, hidden), np.float32)
    for t in range(seq):
        x = emb[t]
        for l in range(2):
            g_ih = lin(f"W_ih{l}", p[f"b_ih{l}"], x)
            g_hh = lin(f"W_hh{l}", p[f"b_hh{l}"], h[l])
            c[l], h[l] = orc.lstm_cell(g_ih, g_hh, c[l])
            x = h[l]
        tops[t] = x
    logits = lin("W_dec", p["b_dec"], tops.reshape(seq * batch, hidden))
    return logits, dict(tops=tops, c=c, emb=emb)
