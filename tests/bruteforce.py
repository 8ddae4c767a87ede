"""Independent brute-force restatement of STTM for tiny inputs (test helper).

Written directly from the paper's description and deliberately unlike the oracle in
structure: recursive feature means, a recursive coarse-to-fine search (Fig. 3),
rectangle-overlap enumeration of temporal candidates (Section 3.3), a naive walk along
links to the root, grouping through dictionaries and an explicit sort (Section 3.4).
Pure Python / numpy float64; only usable for a few hundred tokens.
"""
import numpy as np


def level_sizes(H, W, lv1):
    sizes = [(H, W)]
    while max(sizes[-1]) > lv1:
        h, w = sizes[-1]
        sizes.append((-(-h // 2), -(-w // 2)))
    return sizes


def cos(a, b):
    na, nb = np.sqrt(np.dot(a, a)), np.sqrt(np.dot(b, b))
    if na == 0.0 or nb == 0.0:
        return 0.0
    return float(np.dot(a, b) / (na * nb))


def sttm_bruteforce(video, tau_s, tau_t, lv1=4, weight="node", match="topleft"):
    video = np.asarray(video, dtype=np.float64)
    T, H, W, D = video.shape
    sizes = level_sizes(H, W, lv1)
    L = len(sizes)

    def kids_of(l, i, j):
        return [(2 * i + a, 2 * j + b) for a in (0, 1) for b in (0, 1)
                if 2 * i + a < sizes[l - 1][0] and 2 * j + b < sizes[l - 1][1]]

    def feat(t, l, i, j):
        if l == 0:
            return video[t, i, j]
        ks = [feat(t, l - 1, ci, cj) for ci, cj in kids_of(l, i, j)]
        return sum(ks) / len(ks)

    n_cmp = [0, 0]

    def search(t, l, i, j):
        if l == 0:
            return [(0, i, j)]
        parent = feat(t, l, i, j)
        ks = kids_of(l, i, j)
        n_cmp[0] += len(ks)
        if all(cos(feat(t, l - 1, ci, cj), parent) > tau_s for ci, cj in ks):
            return [(l, i, j)]
        out = []
        for ci, cj in ks:
            out += search(t, l - 1, ci, cj)
        return out

    def rect(node):
        l, i, j = node
        s = 1 << l
        return (i * s, min((i + 1) * s, H), j * s, min((j + 1) * s, W))

    kept = []
    for t in range(T):
        nodes = []
        for i in range(sizes[L - 1][0]):
            for j in range(sizes[L - 1][1]):
                nodes += search(t, L - 1, i, j)
        kept.append(nodes)

    link = {}
    for t in range(1, T):
        for v in kept[t]:
            y0, y1, x0, x1 = rect(v)
            cands = []
            for u in kept[t - 1]:
                a0, a1, b0, b1 = rect(u)
                if match == "topleft_only":
                    if a0 <= y0 < a1 and b0 <= x0 < b1:
                        cands.append(u)
                elif a0 < y1 and y0 < a1 and b0 < x1 and x0 < b1:
                    cands.append(u)
            n_cmp[1] += len(cands)
            fv = feat(t, *v)
            scored = [(cos(fv, feat(t - 1, *u)), u) for u in cands]
            passing = [(s, u) for s, u in scored if s > tau_t]
            if passing:
                if match == "best":
                    top = max(s for s, _ in passing)
                    passing = [(s, u) for s, u in passing if s == top]
                dest = min(passing, key=lambda su: (rect(su[1])[0], rect(su[1])[2]))[1]
                link[(t, v)] = (t - 1, dest)

    def root_of(tv):
        while tv in link:
            tv = link[tv]
        return tv

    groups = {}
    for t in range(T):
        for v in kept[t]:
            groups.setdefault(root_of((t, v)), []).append((t, v))

    def anchor(tv):
        t, v = tv
        y0, _, x0, _ = rect(v)
        return t * H * W + y0 * W + x0

    roots = sorted(groups, key=lambda tv: (tv[0], rect(tv[1])[0], rect(tv[1])[2]))
    row_of = {r: k for k, r in enumerate(roots)}
    out_feats = np.zeros((len(roots), D))
    for r, members in groups.items():
        acc, wsum = np.zeros(D), 0.0
        for (t, v) in members:
            y0, y1, x0, x1 = rect(v)
            w = float((y1 - y0) * (x1 - x0)) if weight == "area" else 1.0
            acc += w * feat(t, *v)
            wsum += w
        out_feats[row_of[r]] = acc / wsum

    N = T * H * W
    cover = np.zeros((T, H, W), dtype=np.int8)
    link_arr = np.full(N, -1, dtype=np.int32)
    root_arr = np.zeros(N, dtype=np.int32)
    mmap = np.zeros(N, dtype=np.int32)
    for t in range(T):
        for v in kept[t]:
            y0, y1, x0, x1 = rect(v)
            r = root_of((t, v))
            for y in range(y0, y1):
                for x in range(x0, x1):
                    c = t * H * W + y * W + x
                    cover[t, y, x] = v[0]
                    link_arr[c] = anchor(link[(t, v)]) if (t, v) in link else -1
                    root_arr[c] = anchor(r)
                    mmap[c] = row_of[r]
    return dict(count=len(roots), cover=cover, link=link_arr, root=root_arr, merge_map=mmap,
                out_feats=out_feats, out_pos=np.array([anchor(r) for r in roots], dtype=np.int32),
                members=np.array([len(groups[r]) for r in roots], dtype=np.int32),
                cmp_spatial=n_cmp[0], cmp_temporal=n_cmp[1])
