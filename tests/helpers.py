"""Independent reference routines used to pin the oracle (numpy / torch CPU / pure Python).
They are written from the textbook definitions, not from the oracle's code."""
import math

import numpy as np


def read_golden(path):
    out = {}
    with open(path) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            out[key] = [float(v) for v in vals]
    return out


def vanilla_route(z, k):
    """Textbook router: softmax over experts -> top-k -> renormalise (Mixtral convention).
    Uses torch library routines; ties are avoided by the caller."""
    import torch
    p = torch.softmax(torch.from_numpy(z).double(), dim=-1)
    val, idx = torch.topk(p, k, dim=-1)
    val = val / val.sum(-1, keepdim=True)
    return idx.numpy().astype(np.int32), val.numpy()


def swiglu_ffn(h, wg, wu, wd):
    """Dense SwiGLU FFN in fp64 with torch CPU routines: W_down(SiLU(W_gate h) * (W_up h))."""
    import torch
    import torch.nn.functional as Fn
    h, wg, wu, wd = (torch.from_numpy(np.asarray(x, dtype=np.float64)) for x in (h, wg, wu, wd))
    return ((Fn.silu(h @ wg.T) * (h @ wu.T)) @ wd.T).numpy()


def vanilla_moe(h, z, wg, wu, wd, k):
    """y = sum_{e in top-k} alpha_e F_e(h), the standard dispatch-free definition."""
    idx, alpha = vanilla_route(z, k)
    T, H = h.shape
    y = np.zeros((T, H))
    for t in range(T):
        for r in range(k):
            e = idx[t, r]
            y[t] += alpha[t, r] * swiglu_ffn(h[t:t + 1], wg[e], wu[e], wd[e])[0]
    return idx, alpha, y


def bruteforce_layer(h, z, u, M, B, lam, K, wg, wu, wd, norm_topk=1, scale=1.0):
    """Dense evaluation over the whole n x n path grid: every P_ij(h) is computed, every active
    path scored, fully sorted with (score desc, flat id asc), the first K weighted and summed."""
    T, H = h.shape
    n = M.shape[0]
    f32 = np.float32
    y = np.zeros((T, H))
    sel = []
    for t in range(T):
        Uall = [None] * n
        for i in range(n):
            g = wg[i].astype(np.float64) @ h[t].astype(np.float64)
            v = wu[i].astype(np.float64) @ h[t].astype(np.float64)
            Uall[i] = g / (1.0 + np.exp(-g)) * v
        Pgrid = [[wd[j].astype(np.float64) @ Uall[i] for j in range(n)] for i in range(n)]
        cands = []
        for i in range(n):
            for j in range(n):
                if M[i, j]:
                    s = f32(f32(f32(z[t, i]) + f32(B[i, j])) + f32(f32(lam) * f32(u[t, j])))
                    cands.append((-float(s), i * n + j))
        cands.sort()
        s0 = -cands[0][0]
        dom = cands[:K] if norm_topk else cands
        den = sum(math.exp(-c[0] - s0) for c in dom)
        row = []
        for (ns, flat) in cands[:K]:
            beta = math.exp(-ns - s0) / den * scale
            i, j = divmod(flat, n)
            y[t] += beta * Pgrid[i][j]
            row.append((i, j, beta))
        sel.append(row)
    return sel, y


def bruteforce_groups(src, tgt, w, n, dedup=1):
    """Grouping by plain Python sorting of explicit (key, order) tuples."""
    T, K = src.shape
    slots = []           # (source, order key, token, flat ids served)
    if dedup:
        for t in range(T):
            for i in sorted(set(int(x) for x in src[t])):
                slots.append((i, t, t, [t * K + k for k in range(K) if src[t, k] == i]))
    else:
        for q in range(T * K):
            slots.append((int(src.flat[q]), q, q // K, [q]))
    slots.sort(key=lambda s: (s[0], s[1]))
    s1_token = np.array([s[2] for s in slots], dtype=np.int32)
    s1_offsets = np.zeros(n + 1, np.int32)
    for s in slots:
        s1_offsets[s[0] + 1:] += 1
    path_s1row = np.zeros(T * K, np.int32)
    for r, s in enumerate(slots):
        for q in s[3]:
            path_s1row[q] = r
    order = sorted(range(T * K), key=lambda q: (int(tgt.flat[q]), q))
    s2_path = np.array(order, dtype=np.int32).reshape(-1)
    s2_offsets = np.zeros(n + 1, np.int32)
    for q in order:
        s2_offsets[int(tgt.flat[q]) + 1:] += 1
    return dict(R1=len(slots), s1_offsets=s1_offsets, s1_token=s1_token,
                path_s1row=path_s1row.reshape(T, K), s2_offsets=s2_offsets, s2_path=s2_path,
                s2_s1row=path_s1row[s2_path] if T * K else s2_path,
                s2_token=(s2_path // K).astype(np.int32),
                s2_w=w.reshape(-1)[s2_path] if T * K else w.reshape(-1))
