"""Independent pure-Python (lists + math, float64) encoder used to pin the oracle on tiny inputs.
Written element by element with explicit loops; shares nothing with oracle/ or the CUDA path."""
import math


def _lin(x, W, b):
    return [[sum(x[t][i] * W[o][i] for i in range(len(W[o]))) + b[o] for o in range(len(W))] for t in range(len(x))]


def _ln(x, g, b, eps):
    out = []
    for row in x:
        d = len(row)
        mu = sum(row) / d
        var = sum((v - mu) * (v - mu) for v in row) / d
        out.append([(row[i] - mu) / math.sqrt(var + eps) * g[i] + b[i] for i in range(d)])
    return out


def _rms(x, g, eps):
    out = []
    for row in x:
        d = len(row)
        ms = sum(v * v for v in row) / d
        out.append([row[i] / math.sqrt(ms + eps) * g[i] for i in range(d)])
    return out


def _gelu(v):
    return 0.5 * v * (1.0 + math.erf(v / math.sqrt(2.0)))


def _silu(v):
    return v / (1.0 + math.exp(-v))


def _norm(cfg, w, prefix, x):
    if cfg["norm"] == 0:
        return _ln(x, w[prefix + ".g"], w[prefix + ".b"], cfg["norm_eps"])
    return _rms(x, w[prefix + ".g"], cfg["norm_eps"])


def _rot(vec, h, wcol, theta):
    hd = len(vec)
    P = hd // 2
    nf = P // 2
    out = list(vec)
    for j in range(P):
        if j < nf:
            ang = h * theta ** (-(j / nf))
        else:
            ang = wcol * theta ** (-((j - nf) / nf))
        c, s = math.cos(ang), math.sin(ang)
        a, b = vec[j], vec[j + P]
        out[j] = a * c - b * s
        out[j + P] = b * c + a * s
    return out


def _tokens(cfg, item):
    """-> (patch rows or None, list of (h, w)) in the encoder's token order."""
    fam = cfg["family"]
    P = cfg["patch"]
    if fam == 0:      # raster order over an image [C][H][W]
        C, H, Wd = len(item), len(item[0]), len(item[0][0])
        rows, pos = [], []
        for r in range(H // P):
            for c in range(Wd // P):
                rows.append([item[ch][r * P + py][c * P + px] for ch in range(C) for py in range(P) for px in range(P)])
                pos.append((r, c))
        return rows, pos
    if fam == 1:      # merge-group-major over a clip [F][C][H][W]
        pt = cfg["temporal_patch"]
        F_, C, H, Wd = len(item), len(item[0]), len(item[0][0]), len(item[0][0][0])
        rows, pos = [], []
        for t in range(F_ // pt):
            for hb in range(H // P // 2):
                for wb in range(Wd // P // 2):
                    for hi in range(2):
                        for wi in range(2):
                            r, c = 2 * hb + hi, 2 * wb + wi
                            rows.append([item[t * pt + f][ch][r * P + py][c * P + px]
                                         for ch in range(C) for f in range(pt) for py in range(P) for px in range(P)])
                            pos.append((r, c))
        return rows, pos
    raise ValueError


def _conv(x, W, b, stride):
    n, cin, cout = len(x), len(x[0]), len(W)
    n_out = (n - 1) // stride + 1
    y = []
    for t in range(n_out):
        row = []
        for o in range(cout):
            acc = b[o]
            for k in range(3):
                src = stride * t + k - 1
                if 0 <= src < n:
                    for c in range(cin):
                        acc += W[o][k][c] * x[src][c]
            row.append(acc)
        y.append(row)
    return y


def encode_item(cfg, w, item):
    """cfg: architecture dict; w: name -> nested lists; item: nested lists."""
    d, H = cfg["d_model"], cfg["n_heads"]
    hd = d // H
    pos = None
    if cfg["family"] == 2:
        h1 = [[_gelu(v) for v in r] for r in _conv(item, w["conv1.w"], w["conv1.b"], 1)]
        h2 = [[_gelu(v) for v in r] for r in _conv(h1, w["conv2.w"], w["conv2.b"], 2)]
        x = [[h2[t][i] + w["pos"][t][i] for i in range(d)] for t in range(len(h2))]
    else:
        rows, pos = _tokens(cfg, item)
        x = _lin(rows, w["embed.w"], w["embed.b"])
        if cfg["has_cls"]:
            x = [list(w["cls"])] + x
        if cfg["pos"] == 0:
            x = [[x[t][i] + w["pos"][t][i] for i in range(d)] for t in range(len(x))]
        if cfg["embed_norm"]:
            x = _norm(cfg, w, "embed_norm", x)
    S = len(x)
    for L in range(cfg["n_layers"]):
        p = f"blk{L}."
        n = _norm(cfg, w, p + "norm1", x)
        qkv = _lin(n, w[p + "qkv.w"], w[p + "qkv.b"])
        attn = [[0.0] * d for _ in range(S)]
        for h in range(H):
            q = [qkv[t][h * hd:(h + 1) * hd] for t in range(S)]
            k = [qkv[t][d + h * hd: d + (h + 1) * hd] for t in range(S)]
            v = [qkv[t][2 * d + h * hd: 2 * d + (h + 1) * hd] for t in range(S)]
            if cfg["pos"] == 1:
                q = [_rot(q[t], pos[t][0], pos[t][1], cfg["rope_theta"]) for t in range(S)]
                k = [_rot(k[t], pos[t][0], pos[t][1], cfg["rope_theta"]) for t in range(S)]
            for t in range(S):
                sc = [sum(q[t][e] * k[u][e] for e in range(hd)) / math.sqrt(hd) for u in range(S)]
                m = max(sc)
                ex = [math.exp(s_ - m) for s_ in sc]
                z = sum(ex)
                for e in range(hd):
                    attn[t][h * hd + e] = sum(ex[u] / z * v[u][e] for u in range(S))
        pr = _lin(attn, w[p + "proj.w"], w[p + "proj.b"])
        x = [[x[t][i] + pr[t][i] for i in range(d)] for t in range(S)]
        n = _norm(cfg, w, p + "norm2", x)
        if cfg["mlp"] == 1:
            g = _lin(n, w[p + "gate.w"], w[p + "gate.b"])
            u = _lin(n, w[p + "up.w"], w[p + "up.b"])
            a = [[_silu(g[t][i]) * u[t][i] for i in range(len(g[t]))] for t in range(S)]
        else:
            a = [[_gelu(v_) for v_ in r] for r in _lin(n, w[p + "fc1.w"], w[p + "fc1.b"])]
        dn = _lin(a, w[p + "fc2.w"], w[p + "fc2.b"])
        x = [[x[t][i] + dn[t][i] for i in range(d)] for t in range(S)]
    if cfg["final_norm"]:
        x = _norm(cfg, w, "final_norm", x)
    if cfg["head"] == 0:
        return x
    if cfg["head"] == 1:
        if cfg["has_cls"]:
            x = x[1:]
        mid = [[_gelu(v_) for v_ in r] for r in _lin(x, w["head.fc1.w"], w["head.fc1.b"])]
        return _lin(mid, w["head.fc2.w"], w["head.fc2.b"])
    n = _rms(x, w["head.norm.g"], cfg["norm_eps"])
    grouped = [n[4 * g] + n[4 * g + 1] + n[4 * g + 2] + n[4 * g + 3] for g in range(S // 4)]
    mid = [[_gelu(v_) for v_ in r] for r in _lin(grouped, w["head.fc1.w"], w["head.fc1.b"])]
    return _lin(mid, w["head.fc2.w"], w["head.fc2.b"])
