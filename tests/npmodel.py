"""Test-side, third formulation of the layout contract, used only to pin the oracle.

It is written differently from the oracle on purpose: logical tensors are numpy arrays, a TP shard is what
``np.split`` along the parallel axis returns (the textbook definition of column- and row-parallel
sharding), fused blocks are ``np.concatenate`` of the rank's pieces, and a shard buffer is those blocks laid
end to end on 256-byte boundaries.  ``owner`` is the same contract once more as a per-element function.
"""
from __future__ import annotations

import numpy as np

KINDS = ["ln1", "wq", "wk", "wv", "wo", "ln2", "wgate", "wup", "wdown"]


def np_dtype(es):
    return np.uint16 if es == 2 else np.uint32


def logical_names(L):
    names = ["embed"]
    for l in range(L):
        names += [f"{k}.{l}" for k in KINDS]
    return names + ["ln_f", "head"]


def logical_shapes(sh, value_head=False):
    hd = sh.hidden // sh.heads
    per = {"ln1": (1, sh.hidden), "ln2": (1, sh.hidden),
           "wq": (sh.heads * hd, sh.hidden), "wk": (sh.kv_heads * hd, sh.hidden),
           "wv": (sh.kv_heads * hd, sh.hidden), "wo": (sh.hidden, sh.heads * hd),
           "wgate": (sh.ffn, sh.hidden), "wup": (sh.ffn, sh.hidden), "wdown": (sh.hidden, sh.ffn)}
    out = {"embed": (sh.vocab, sh.hidden)}
    for l in range(sh.layers):
        for k in KINDS:
            out[f"{k}.{l}"] = per[k]
    out["ln_f"] = (1, sh.hidden)
    out["head"] = (1, sh.hidden) if value_head else (sh.vocab, sh.hidden)
    return out


def random_logical(sh, es, seed, value_head=False):
    rng = np.random.default_rng(seed)
    dt = np_dtype(es)
    return {n: rng.integers(0, np.iinfo(dt).max, size=s, dtype=dt, endpoint=True)
            for n, s in logical_shapes(sh, value_head).items()}


def position_coded(sh, es, salt, value_head=False):
    """Element (tensor t, row i, col j) holds a hash of (t, i, j, salt), truncated to the element width."""
    out = {}
    for t, (n, (r, c)) in enumerate(logical_shapes(sh, value_head).items()):
        i = np.arange(r, dtype=np.uint64)[:, None]
        j = np.arange(c, dtype=np.uint64)[None, :]
        with np.errstate(over="ignore"):
          h = (np.uint64(t + 1) * np.uint64(0x9E3779B97F4A7C15) + i * np.uint64(0xC2B2AE3D27D4EB4F)
               + j * np.uint64(0x165667B19E3779F9) + np.uint64(salt) * np.uint64(0x27D4EB2F165667C5))
          h ^= h >> np.uint64(29)
          h *= np.uint64(0xBF58476D1CE4E5B9)
          h ^= h >> np.uint64(32)
        out[n] = h.astype(np_dtype(es))
    return out


QKV_GROUPED, GATE_UP_INTERLEAVED, VOCAB_PADDED = 1, 2, 4


def _stored_blocks(sh, tp, pp, p, r, logical, value_head, layout=0):
    """The tensors shard (p, r) stores, in packing order, as numpy arrays (np.split formulation).  Layout
    variants reorder rows inside a rank's fused block: grouped QKV = per kv head [its q heads; k; v] (a reshape
    to [kv_heads, rows per head group, H]); interleaved gate/up = np.stack of the two row sets."""
    hd = sh.hidden // sh.heads
    local_kv = max(1, sh.kv_heads // tp)                  # kv heads a rank holds
    G = (sh.heads // tp) // local_kv                      # q heads per kv head inside a rank
    def d0(x):
        return np.split(x, tp, axis=0)[r]

    def d1(x):
        return np.split(x, tp, axis=1)[r]

    def dvocab(x):           # vocabulary rows: cut evenly, or padded to a multiple of 128*tp first
        if not layout & VOCAB_PADDED:
            return d0(x)
        v_pad = -(-sh.vocab // (128 * tp)) * 128 * tp
        filler = np.full((v_pad - sh.vocab, x.shape[1]), np.iinfo(x.dtype).max // 0xFF * 0xA5, x.dtype)   # 0xA5 bytes
        return np.split(np.concatenate([x, filler], axis=0), tp, axis=0)[r]

    def dkv(x):              # kv heads: cut like any row block, or, past one head per rank, replicated
        if tp <= sh.kv_heads:
            return d0(x)
        return np.split(x, sh.kv_heads, axis=0)[r // (tp // sh.kv_heads)]

    mine = np.array_split(np.arange(sh.layers), pp)[p]      # an uneven cut gives the first stages one layer more
    blocks = []
    if p == 0:
        blocks.append(dvocab(logical["embed"]))
    for l in mine:
        g = lambda k: logical[f"{k}.{l}"]
        blocks.append(g("ln1"))
        if layout & QKV_GROUPED:
            q = d0(g("wq")).reshape(local_kv, G * hd, sh.hidden)
            k = dkv(g("wk")).reshape(local_kv, hd, sh.hidden)
            v = dkv(g("wv")).reshape(local_kv, hd, sh.hidden)
            blocks.append(np.concatenate([np.concatenate([q[h], k[h], v[h]], axis=0) for h in range(local_kv)],
                                         axis=0))
        else:
            blocks.append(np.concatenate([d0(g("wq")), dkv(g("wk")), dkv(g("wv"))], axis=0))
        blocks.append(d1(g("wo")))
        blocks.append(g("ln2"))
        if layout & GATE_UP_INTERLEAVED:
            blocks.append(np.stack([d0(g("wgate")), d0(g("wup"))], axis=1).reshape(-1, sh.hidden))
        else:
            blocks.append(np.concatenate([d0(g("wgate")), d0(g("wup"))], axis=0))
        blocks.append(d1(g("wdown")))
    if p == pp - 1:
        blocks.append(logical["ln_f"])
        blocks.append(logical["head"] if value_head else dvocab(logical["head"]))
    return blocks


def build_shards(sh, tp, pp, logical, value_head=False, pad=0xA5, layout=0):
    """Shard byte images (uint8 arrays), index = p * tp + r."""
    out = []
    for p in range(pp):
        for r in range(tp):
            chunks, cur = [], 0
            for b in _stored_blocks(sh, tp, pp, p, r, logical, value_head, layout):
                start = -(-cur // 256) * 256
                if start > cur:
                    chunks.append(np.full(start - cur, pad, np.uint8))
                raw = np.ascontiguousarray(b).view(np.uint8).reshape(-1)
                chunks.append(raw)
                cur = start + raw.size
            end = -(-cur // 256) * 256
            if end > cur:
                chunks.append(np.full(end - cur, pad, np.uint8))
            out.append(np.concatenate(chunks))
    return out


def owner(sh, tp, pp, es, name, i, j, value_head=False, layout=0):
    """Per-element statement of the contract: every (shard, byte offset) that holds element (i, j) of the
    logical tensor ``name`` (several for replicated tensors)."""
    hd = sh.hidden // sh.heads
    H, F, V = sh.hidden, sh.ffn, sh.vocab
    nq, nkv = sh.heads, sh.kv_heads
    bounds = [(int(c[0]), int(c[-1]) + 1) for c in np.array_split(np.arange(sh.layers), pp)]
    qr, kr, fr, vr = nq * hd // tp, nkv * hd // tp, F // tp, V // tp
    up = lambda x: -(-x // 256) * 256
    # byte sizes of the stored blocks of one layer, in order
    layer_blocks = [("ln", H), ("qkv", (qr + 2 * kr) * H), ("wo", H * (nq * hd // tp)), ("ln", H),
                    ("gu", 2 * fr * H), ("wdown", H * fr)]

    def layer_base(p, l):
        cur = 0
        if p == 0:
            cur = up(cur) + vr * H * es
        for _ in range(bounds[p][0], l):
            for _, n in layer_blocks:
                cur = up(cur) + n * es
        return cur

    def within_layer(idx):
        # offset of the idx-th stored block of a layer relative to an (aligned) running cursor
        def f(cur):
            for k, (_, n) in enumerate(layer_blocks):
                cur = up(cur)
                if k == idx:
                    return cur
                cur += n * es
        return f

    if name == "embed":
        r = i // vr
        return [(0 * tp + r, up(0) + ((i % vr) * H + j) * es)]
    if name in ("ln_f", "head"):
        p = pp - 1
        cur = layer_base(p, bounds[p][1])
        lnf = up(cur)
        head = up(lnf + H * es)
        if name == "ln_f":
            return [(p * tp + r, lnf + j * es) for r in range(tp)]
        if value_head:
            return [(p * tp + r, head + j * es) for r in range(tp)]
        r = i // vr
        return [(p * tp + r, head + ((i % vr) * H + j) * es)]
    kind, l = name.split(".")
    l = int(l)
    p = next(k for k, (lo, hi) in enumerate(bounds) if lo <= l < hi)
    base = layer_base(p, l)
    blk = {"ln1": 0, "wq": 1, "wk": 1, "wv": 1, "wo": 2, "ln2": 3, "wgate": 4, "wup": 4, "wdown": 5}[kind]
    start = within_layer(blk)(base)
    if kind in ("ln1", "ln2"):
        return [(p * tp + r, start + j * es) for r in range(tp)]
    if kind in ("wq", "wk", "wv") and layout & QKV_GROUPED:
        G = nq // nkv
        head = i // hd
        kv = head // G if kind == "wq" else head              # the kv head whose group the row belongs to
        r = kv // (nkv // tp)
        row = (kv % (nkv // tp)) * (G + 2) * hd                 # earlier groups of this rank
        row += {"wq": (head % G) * hd, "wk": G * hd, "wv": (G + 1) * hd}[kind] + i % hd
        return [(p * tp + r, start + (row * H + j) * es)]
    if kind == "wq":
        r = i // qr
        return [(p * tp + r, start + ((i % qr) * H + j) * es)]
    if kind in ("wk", "wv"):
        r = i // kr
        skip = qr + (kr if kind == "wv" else 0)
        return [(p * tp + r, start + ((skip + i % kr) * H + j) * es)]
    if kind in ("wgate", "wup") and layout & GATE_UP_INTERLEAVED:
        r = i // fr
        return [(p * tp + r, start + ((2 * (i % fr) + (kind == "wup")) * H + j) * es)]
    if kind in ("wgate", "wup"):
        r = i // fr
        skip = fr if kind == "wup" else 0
        return [(p * tp + r, start + ((skip + i % fr) * H + j) * es)]
    if kind == "wo":
        w = nq * hd // tp
        r = j // w
        return [(p * tp + r, start + (i * w + j % w) * es)]
    if kind == "wdown":
        r = j // fr
        return [(p * tp + r, start + (i * fr + j % fr) * es)]
    raise KeyError(name)
