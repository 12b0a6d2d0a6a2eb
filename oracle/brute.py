"""Scalar brute force of one MLA-Online layer: plain Python loops and `math`, no numpy
arithmetic, written independently of oracle/mla_online.py so that a wrong index, sign or
transposed operand in either shows up as a disagreement.  Only for a few tokens.

Test infrastructure; cites the same passages: Eq. rope (key re-rotation), Algorithm 2
(Global heads on every row, Local heads on protected rows), Eq. offonline / factorization
(sliced W_a, shared W_b), RestoreAndReplace (a protected row takes the online Local value in place of
the artifact; the two are never added).
"""
from __future__ import annotations

import math


def _rot(vec, p, base):
    """R(p) on a list of even length, interleaved pairs, theta_j = base^(-2j/d)."""
    d = len(vec)
    out = [0.0] * d
    for j in range(d // 2):
        th = base ** (-2.0 * j / d)
        c, s = math.cos(p * th), math.sin(p * th)
        a, b = vec[2 * j], vec[2 * j + 1]
        out[2 * j] = a * c - b * s
        out[2 * j + 1] = a * s + b * c
    return out


def brute_layer(q_all, kv, seg_off, seg_delta, prot_rows, global_heads, w_uv, w_a, w_b, z_off,
                sm_scale, base, d_latent, group_size=8):
    """q_all [T][H][d_qk], kv [T][d_qk], w_uv [H][d_v][d_c], w_a [G][r_o][8*d_v],
    w_b [d_model][G*r_o], z_off [rows][G*r_o] as nested lists (or anything indexable).
    Returns dict(lse [T][H] (None where the head is not computed), z [T][G*r_o], y [T][d_model],
    y_full [T][d_model])."""
    T = len(kv)
    H = len(q_all[0])
    dqk = len(kv[0])
    G = len(w_a)
    ro = len(w_a[0])
    dv = len(w_uv[0])
    dm = len(w_b)
    S = len(seg_delta)
    seg = [0] * T
    pos = [0] * T
    for i in range(S):
        for r in range(int(seg_off[i]), int(seg_off[i + 1])):
            seg[r] = i
            pos[r] = int(seg_delta[i]) + (r - int(seg_off[i]))
    # keys at their request positions
    kreq = []
    for k in range(T):
        row = [float(x) for x in kv[k]]
        rr = _rot(row[d_latent:], float(seg_delta[seg[k]]), base)
        kreq.append(row[:d_latent] + rr)
    prot = set(int(r) for r in prot_rows)
    gset = set(int(h) for h in global_heads)

    def head_out(t, h):
        """returns (lse, contribution[r_o]) of head h on row t"""
        qv = [float(x) for x in q_all[t][h]]
        vis = [k for k in range(T) if pos[k] <= pos[t]]
        sc = []
        for k in vis:
            acc = 0.0
            for e in range(dqk):
                acc += qv[e] * kreq[k][e]
            sc.append(acc * sm_scale)
        m = max(sc)
        ex = [math.exp(s - m) for s in sc]
        l = sum(ex)
        olat = [0.0] * d_latent
        for w, k in zip(ex, vis):
            for e in range(d_latent):
                olat[e] += (w / l) * float(kv[k][e])
        o = [0.0] * dv
        for a in range(dv):
            acc = 0.0
            for e in range(d_latent):
                acc += float(w_uv[h][a][e]) * olat[e]
            o[a] = acc
        g, j = h // group_size, h % group_size
        c = [0.0] * ro
        for r in range(ro):
            acc = 0.0
            for a in range(dv):
                acc += float(w_a[g][r][dv * j + a]) * o[a]
            c[r] = acc
        return m + math.log(l), c

    lse = [[None] * H for _ in range(T)]
    z = [[0.0] * (G * ro) for _ in range(T)]
    zfull = [[0.0] * (G * ro) for _ in range(T)]
    for t in range(T):
        for h in range(H):
            l_th, c = head_out(t, h)
            g = h // group_size
            for r in range(ro):
                zfull[t][g * ro + r] += c[r]
            if h in gset or t in prot:
                lse[t][h] = l_th
                for r in range(ro):
                    z[t][g * ro + r] += c[r]
        if t not in prot:
            for e in range(G * ro):
                z[t][e] += float(z_off[t][e])

    def wb(zrow):
        return [sum(float(w_b[m][e]) * zrow[e] for e in range(G * ro)) for m in range(dm)]

    y = [wb(z[t]) for t in range(T)]
    y_full = [wb(zfull[t]) for t in range(T)]
    return dict(lse=lse, z=z, y=y, y_full=y_full)


def brute_layer_phase(q_all, kv, seg_off, seg_delta, prot_rows, global_heads, w_uv, w_a, w_b, z_off,
                      sm_scale, base, d_latent, group_size=8):
    """The output-phase variant in the same scalar style (Eq. offonline with R^{-1}; Algorithm 2
    RestorePhase): the whole stored row is the value, turned to its request position like the key;
    the rope dims of a row's output are turned back by its own position before W_uv, which here is
    [H][d_v][d_qk].  Same arguments and result keys as `brute_layer`, plus o_rope [T][H] (the
    restored rope dims, None where the head is not computed)."""
    T = len(kv)
    H = len(q_all[0])
    dqk = len(kv[0])
    G = len(w_a)
    ro = len(w_a[0])
    dv = len(w_uv[0])
    dm = len(w_b)
    S = len(seg_delta)
    pos = [0] * T
    vreq = []
    for i in range(S):
        for r in range(int(seg_off[i]), int(seg_off[i + 1])):
            pos[r] = int(seg_delta[i]) + (r - int(seg_off[i]))
            row = [float(x) for x in kv[r]]
            vreq.append(row[:d_latent] + _rot(row[d_latent:], float(seg_delta[i]), base))
    prot = set(int(r) for r in prot_rows)
    gset = set(int(h) for h in global_heads)

    def head_out(t, h):
        qv = [float(x) for x in q_all[t][h]]
        best = None
        sc = {}
        for k in range(T):
            if pos[k] > pos[t]:
                continue
            sc[k] = sm_scale * sum(qv[e] * vreq[k][e] for e in range(dqk))
            best = sc[k] if best is None else max(best, sc[k])
        den = sum(math.exp(s - best) for s in sc.values())
        out = [0.0] * dqk
        for k, s in sc.items():
            w = math.exp(s - best) / den
            for e in range(dqk):
                out[e] += w * vreq[k][e]
        back = _rot(out[d_latent:], -float(pos[t]), base)     # inverse output RoPE at the row's position
        out = out[:d_latent] + back
        o = [sum(float(w_uv[h][a][e]) * out[e] for e in range(dqk)) for a in range(dv)]
        g, j = h // group_size, h % group_size
        c = [sum(float(w_a[g][r][dv * j + a]) * o[a] for a in range(dv)) for r in range(ro)]
        return best + math.log(den), c, back

    lse = [[None] * H for _ in range(T)]
    o_rope = [[None] * H for _ in range(T)]
    z = [[0.0] * (G * ro) for _ in range(T)]
    zfull = [[0.0] * (G * ro) for _ in range(T)]
    for t in range(T):
        for h in range(H):
            l_th, c, back = head_out(t, h)
            g = h // group_size
            for r in range(ro):
                zfull[t][g * ro + r] += c[r]
            if h in gset or t in prot:
                lse[t][h] = l_th
                o_rope[t][h] = back
                for r in range(ro):
                    z[t][g * ro + r] += c[r]
        if t not in prot:
            for e in range(G * ro):
                z[t][e] += float(z_off[t][e])

    def wb(zrow):
        return [sum(float(w_b[m][e]) * zrow[e] for e in range(G * ro)) for m in range(dm)]

    return dict(lse=lse, o_rope=o_rope, z=z, y=[wb(z[t]) for t in range(T)], y_full=[wb(zfull[t]) for t in range(T)])
