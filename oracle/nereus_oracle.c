/*
 * TEST INFRASTRUCTURE -- NOT PART OF THE PRODUCT.
 *
 * Plain, slow, single-threaded CPU oracle for the EMU reshard: the layout
 * change that carries one model-stage's parameter shards theta = {theta_i},
 * i = 1..tp*pp (EMU definition, Section 5) from a source (TP, PP) layout to a
 * target (TP, PP) layout.  Split and Merge move and re-cut state but leave
 * the logical state as it was (Section 6.2, on preserving training
 * semantics), and Split is a position-wise AllGather followed by a local
 * layout change (Section 6.2, "DAG Execution and Safety" and
 * "Resharding--transport interplay").  So the result has a plain definition
 * and this file is that definition written out, per logical tensor:
 *
 *     1. GATHER  the full logical tensor [rows][cols] from the source shards,
 *     2. CAST    element by element when the target dtype differs (fp32->bf16,
 *                round to nearest even),
 *     3. SLICE   it by the target plan's rule into the target shards.
 *
 * The paper fixes none of the tensor-level layout (fused QKV, fused gate/up,
 * vocabulary rows, row-parallel columns, packing of a shard buffer, the cast):
 * those are this build's layout contract.  They are "parity unpinned" by the
 * paper; what pins them is stated next to each function and in the tests
 * (identity, round trip, np.split/np.concatenate special cases, a brute-force
 * per-element owner function, checksum conservation, published parameter
 * counts, torch's fp32->bf16 conversion over all 2^32 inputs).
 *
 * Only tests, the smoke check and the benchmark's cpu_baseline / reference
 * arm may build, load or call this file.  It shares no code with the CUDA
 * path and includes none of its headers.
 *
 * Layout contract (restated here on purpose, independently of the product):
 *   model      L layers, hidden H, nq query heads, nkv KV heads, hd = H / nq,
 *              FFN F, vocabulary V, element size es (2 = bf16, 4 = fp32),
 *              optional value head [1, H] in place of the LM head [V, H].
 *   plan       (tp, pp): pipeline stage p owns layers [p*L/pp, (p+1)*L/pp) (when pp does not
 *              divide L, the first L mod pp stages own one layer more than the others),
 *              the embedding lives on stage 0, final norm + head on stage
 *              pp-1; shard index = p * tp + r  (TP rank fastest).
 *   TP rank r of t holds
 *     embed, LM head [V, H]   rows    [r*V/t, (r+1)*V/t)
 *     wq [nq*hd, H]           rows of q heads  [r*nq/t, (r+1)*nq/t)
 *     wk, wv [nkv*hd, H]      rows of kv heads [r*nkv/t, (r+1)*nkv/t); when t > nkv (nkv | t) every kv head is
 *                             replicated on t/nkv ranks: rank r holds head r / (t/nkv), the head its q heads use
 *     wo [H, nq*hd]           columns [r*nq*hd/t, (r+1)*nq*hd/t)
 *     wgate, wup [F, H]       rows    [r*F/t, (r+1)*F/t)
 *     wdown [H, F]            columns [r*F/t, (r+1)*F/t)
 *     ln1, ln2, ln_f [H], value head [1, H]   whole tensor (replicated)
 *   shard buffer packing, every stored tensor starting on a 256-byte boundary:
 *     [embed], then per local layer: ln1, {wq;wk;wv} fused, wo, ln2,
 *     {wgate;wup} fused, wdown, then [ln_f, head].
 *     Inside the fused QKV block the rank's Q rows come first, then its K
 *     rows, then its V rows; inside gate/up the rank's gate rows, then its up
 *     rows.  The buffer length is the end of the last tensor rounded up to
 *     256 bytes.  Padding bytes are never read and never written.
 *   layout variants of a plan (order inside a rank's fused block only):
 *     grouped QKV: for each kv head of the rank, its q heads, its k head, its v head;
 *     interleaved gate/up: g0, u0, g1, u1, ... row by row.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <stddef.h>

enum { ORACLE_OK = 0, ORACLE_ERR_ARG = -1, ORACLE_ERR_INDIVISIBLE = -2,
       ORACLE_ERR_UNSUPPORTED = -3, ORACLE_ERR_REPLICA_MISMATCH = -4,
       ORACLE_ERR_NOMEM = -5 };

enum { ORACLE_BF16 = 1, ORACLE_FP32 = 2 };

typedef struct {
    int64_t L, H, nq, nkv, F, V;
    int dtype;        /* ORACLE_BF16 or ORACLE_FP32: dtype of a plan whose dtype field is 0 */
    int value_head;   /* 0: LM head [V, H]; 1: value head [1, H] */
} oracle_model;

/* layout: bit 0 set = fused QKV stored group by group inside a rank's block (for each of the rank's kv heads: its
 * q heads, then its k head, then its v head) instead of [all Q; all K; all V]; bit 1 set = gate and up rows
 * interleaved row by row inside a rank's block (g0, u0, g1, u1, ...) instead of [all gate; all up].  Which
 * heads and rows a rank holds does not depend on these two, only their order inside the fused block.
 * bit 2 set = the vocabulary dimension of embed and LM head is padded up to a multiple of 128*tp before it is
 * cut (the habit of Megatron-style trainers): rank r stores V_pad/tp rows, of which those past row V are
 * padding that no transition reads or writes; V need not divide by tp then. */
enum { ORACLE_QKV_GROUPED = 1, ORACLE_GATE_UP_INTERLEAVED = 2, ORACLE_VOCAB_PADDED = 4 };
typedef struct { int tp, pp, dtype, layout; } oracle_plan;

/* kinds of logical tensor */
enum { K_EMBED, K_LN1, K_WQ, K_WK, K_WV, K_WO, K_LN2, K_WGATE, K_WUP, K_WDOWN, K_LNF, K_HEAD };

static int64_t align256(int64_t x) { return (x + 255) / 256 * 256; }

static int plan_es(const oracle_model* m, oracle_plan p) {
    int d = p.dtype ? p.dtype : m->dtype;
    return d == ORACLE_FP32 ? 4 : 2;
}

int64_t oracle_num_logical(const oracle_model* m) { return 9 * m->L + 3; }

/* logical id -> (kind, layer).  Order: embed, per layer ln1 wq wk wv wo ln2 wgate wup wdown, ln_f, head */
static void decode_id(const oracle_model* m, int64_t id, int* kind, int64_t* layer) {
    static const int per_layer[9] = { K_LN1, K_WQ, K_WK, K_WV, K_WO, K_LN2, K_WGATE, K_WUP, K_WDOWN };
    if (id == 0) { *kind = K_EMBED; *layer = -1; return; }
    if (id == 9 * m->L + 1) { *kind = K_LNF; *layer = -1; return; }
    if (id == 9 * m->L + 2) { *kind = K_HEAD; *layer = -1; return; }
    *layer = (id - 1) / 9;
    *kind = per_layer[(id - 1) % 9];
}

/* Full logical shape [rows][cols] of a tensor kind. */
static void kind_shape(const oracle_model* m, int kind, int64_t* rows, int64_t* cols) {
    int64_t hd = m->H / m->nq;
    switch (kind) {
    case K_EMBED:  *rows = m->V;        *cols = m->H; break;
    case K_HEAD:   *rows = m->value_head ? 1 : m->V; *cols = m->H; break;
    case K_LN1: case K_LN2: case K_LNF: *rows = 1; *cols = m->H; break;
    case K_WQ:     *rows = m->nq * hd;  *cols = m->H; break;
    case K_WK: case K_WV: *rows = m->nkv * hd; *cols = m->H; break;
    case K_WO:     *rows = m->H;        *cols = m->nq * hd; break;
    case K_WGATE: case K_WUP: *rows = m->F; *cols = m->H; break;
    case K_WDOWN:  *rows = m->H;        *cols = m->F; break;
    default:       *rows = 0;           *cols = 0;
    }
}

int oracle_logical_shape(const oracle_model* m, int64_t id, int64_t* rows, int64_t* cols) {
    int kind; int64_t layer;
    if (!m || id < 0 || id >= oracle_num_logical(m)) return ORACLE_ERR_ARG;
    decode_id(m, id, &kind, &layer);
    kind_shape(m, kind, rows, cols);
    return ORACLE_OK;
}

int oracle_check_plan(const oracle_model* m, oracle_plan p) {
    if (!m || p.tp < 1 || p.pp < 1 || (p.layout & ~7)) return ORACLE_ERR_ARG;
    if (m->L < 1 || m->H < 1 || m->nq < 1 || m->nkv < 1 || m->F < 1 || m->V < 1) return ORACLE_ERR_ARG;
    if (m->H % m->nq || m->nq % m->nkv) return ORACLE_ERR_INDIVISIBLE;
    /* tp <= nkv: whole kv heads per rank.  tp > nkv: every kv head is replicated on tp/nkv ranks, which needs
     * nkv | tp; a rank's q heads must then all belong to its one kv head, which tp | nq gives. */
    if (p.tp <= m->nkv ? m->nkv % p.tp : p.tp % m->nkv) return ORACLE_ERR_INDIVISIBLE;
    if (m->nq % p.tp || m->F % p.tp) return ORACLE_ERR_INDIVISIBLE;
    if (p.pp > m->L) return ORACLE_ERR_INDIVISIBLE;         /* every stage needs a layer */
    if (!(p.layout & ORACLE_VOCAB_PADDED) && m->V % p.tp) return ORACLE_ERR_INDIVISIBLE;
    return ORACLE_OK;
}

/* The part of a logical tensor of `kind` that TP rank r of t holds:
 * rows [*r0, *r0 + *nr), columns [*c0, *c0 + *nc) of the full tensor. */
static int64_t padded_vocab(const oracle_model* m, int64_t t) {
    return (m->V + 128 * t - 1) / (128 * t) * (128 * t);
}

static int vocab_cut(const oracle_model* m, int kind) {
    return kind == K_EMBED || (kind == K_HEAD && !m->value_head);
}

static void rank_part(const oracle_model* m, oracle_plan pl, int kind, int64_t r,
                      int64_t* r0, int64_t* nr, int64_t* c0, int64_t* nc) {
    int64_t rows, cols, t = pl.tp;
    kind_shape(m, kind, &rows, &cols);
    *r0 = 0; *nr = rows; *c0 = 0; *nc = cols;
    if (vocab_cut(m, kind) && (pl.layout & ORACLE_VOCAB_PADDED)) {
        int64_t per = padded_vocab(m, t) / t, lo = r * per, hi = (r + 1) * per;   /* rows of the padded table */
        if (lo > rows) lo = rows;
        if (hi > rows) hi = rows;
        *r0 = lo; *nr = hi - lo;                                /* the real rows among them, maybe none */
        return;
    }
    switch (kind) {
    case K_WK: case K_WV:
        if (t > m->nkv) {                                       /* replicated kv heads: rank r holds the one */
            int64_t hd = m->H / m->nq;                          /* head its q heads attend to                */
            *nr = hd; *r0 = (r / (t / m->nkv)) * hd;
            break;
        }
        /* fall through */
    case K_EMBED: case K_WQ: case K_WGATE: case K_WUP:
        *nr = rows / t; *r0 = r * (rows / t); break;            /* dim-0 (column-parallel) */
    case K_HEAD:
        if (!m->value_head) { *nr = rows / t; *r0 = r * (rows / t); }
        break;                                                  /* value head: replicated */
    case K_WO: case K_WDOWN:
        *nc = cols / t; *c0 = r * (cols / t); break;            /* dim-1 (row-parallel) */
    default: break;                                             /* norms: replicated */
    }
}

/* Elements of `kind` stored by one TP rank of t. */
static int64_t rank_elems(const oracle_model* m, oracle_plan pl, int kind) {
    int64_t r0, nr, c0, nc;
    if (vocab_cut(m, kind) && (pl.layout & ORACLE_VOCAB_PADDED))
        return padded_vocab(m, pl.tp) / pl.tp * m->H;           /* padding rows take room in every shard */
    rank_part(m, pl, kind, 0, &r0, &nr, &c0, &nc);
    return nr * nc;
}

/* Row of the fused stored block (counted from the block's first row) that holds local row i of the rank's
 * part of logical tensor `kind`.  Tensors that are stored alone have row i at row i. */
static int64_t part_rowpos(const oracle_model* m, oracle_plan pl, int kind, int64_t i) {
    int64_t hd = m->H / m->nq, t = pl.tp;
    int64_t kv_heads = t > m->nkv ? 1 : m->nkv / t;            /* kv heads a rank holds */
    int64_t G = (m->nq / t) / kv_heads;                        /* q heads per kv head inside a rank */
    int64_t qr = m->nq * hd / t, kr = kv_heads * hd, fr = m->F / t;
    if (kind == K_WQ || kind == K_WK || kind == K_WV) {
        if (pl.layout & ORACLE_QKV_GROUPED) {
            int64_t head = i / hd, within = i % hd, group_rows = (G + 2) * hd;
            if (kind == K_WQ) return (head / G) * group_rows + (head % G) * hd + within;
            if (kind == K_WK) return head * group_rows + G * hd + within;
            return head * group_rows + (G + 1) * hd + within;
        }
        if (kind == K_WQ) return i;
        if (kind == K_WK) return qr + i;
        return qr + kr + i;
    }
    if (kind == K_WGATE || kind == K_WUP) {
        if (pl.layout & ORACLE_GATE_UP_INTERLEAVED) return 2 * i + (kind == K_WUP ? 1 : 0);
        return kind == K_WGATE ? i : fr + i;
    }
    return i;
}

/* Walk the packing order of shard (stage p, any TP rank) and return the byte
 * offset of the first element of logical tensor (kind, layer), or -1 if the
 * stage does not hold it.  *total gets the shard buffer length. */
static int64_t pack_offset(const oracle_model* m, oracle_plan pl, int64_t p,
                           int want_kind, int64_t want_layer, int64_t* total) {
    int64_t es = plan_es(m, pl), cur = 0, found = -1;
    /* layers [first, last) of stage p: an even cut; when pp does not divide L the first L mod pp stages hold
     * one layer more (the split numpy's array_split makes) */
    int64_t base = m->L / pl.pp, extra = m->L % pl.pp;
    int64_t first = p * base + (p < extra ? p : extra), last = first + base + (p < extra ? 1 : 0);
    if (p == 0) {
        cur = align256(cur);
        if (want_kind == K_EMBED) found = cur;
        cur += rank_elems(m, pl, K_EMBED) * es;
    }
    for (int64_t l = first; l < last; ++l) {
        int hit = (l == want_layer);
        cur = align256(cur);                                    /* ln1 */
        if (hit && want_kind == K_LN1) found = cur;
        cur += rank_elems(m, pl, K_LN1) * es;
        cur = align256(cur);                                    /* fused q;k;v: row 0 of each part */
        if (hit && (want_kind == K_WQ || want_kind == K_WK || want_kind == K_WV))
            found = cur + part_rowpos(m, pl, want_kind, 0) * m->H * es;
        cur += (rank_elems(m, pl, K_WQ) + rank_elems(m, pl, K_WK) + rank_elems(m, pl, K_WV)) * es;
        cur = align256(cur);                                    /* wo */
        if (hit && want_kind == K_WO) found = cur;
        cur += rank_elems(m, pl, K_WO) * es;
        cur = align256(cur);                                    /* ln2 */
        if (hit && want_kind == K_LN2) found = cur;
        cur += rank_elems(m, pl, K_LN2) * es;
        cur = align256(cur);                                    /* fused gate;up: row 0 of each part */
        if (hit && (want_kind == K_WGATE || want_kind == K_WUP))
            found = cur + part_rowpos(m, pl, want_kind, 0) * m->H * es;
        cur += (rank_elems(m, pl, K_WGATE) + rank_elems(m, pl, K_WUP)) * es;
        cur = align256(cur);                                    /* wdown */
        if (hit && want_kind == K_WDOWN) found = cur;
        cur += rank_elems(m, pl, K_WDOWN) * es;
    }
    if (p == pl.pp - 1) {
        cur = align256(cur);
        if (want_kind == K_LNF) found = cur;
        cur += rank_elems(m, pl, K_LNF) * es;
        cur = align256(cur);
        if (want_kind == K_HEAD) found = cur;
        cur += rank_elems(m, pl, K_HEAD) * es;
    }
    if (total) *total = align256(cur);
    return found;
}

int oracle_num_shards(const oracle_model* m, oracle_plan pl, int64_t* n) {
    int rc = oracle_check_plan(m, pl);
    if (rc) return rc;
    *n = (int64_t)pl.tp * pl.pp;
    return ORACLE_OK;
}

int oracle_shard_bytes(const oracle_model* m, oracle_plan pl, int64_t shard, int64_t* bytes) {
    int rc = oracle_check_plan(m, pl);
    if (rc) return rc;
    if (shard < 0 || shard >= (int64_t)pl.tp * pl.pp) return ORACLE_ERR_ARG;
    pack_offset(m, pl, shard / pl.tp, -1, -1, bytes);
    return ORACLE_OK;
}

/* Where shard `shard` of plan `pl` keeps its part of logical tensor `id`:
 * byte offset of the part's first element in the shard buffer, and the part's
 * position [r0, r0+nr) x [c0, c0+nc) in the full tensor.  Each row of the part
 * is nc contiguous elements; row i starts oracle_part_row(i) * nc elements
 * after row 0 (i itself unless the plan's layout interleaves the fused block).
 * *held = 0 when the shard's stage does not own the tensor. */
int oracle_locate(const oracle_model* m, oracle_plan pl, int64_t shard, int64_t id,
                  int* held, int64_t* offset, int64_t* r0, int64_t* nr, int64_t* c0, int64_t* nc) {
    int kind; int64_t layer, off;
    int rc = oracle_check_plan(m, pl);
    if (rc) return rc;
    if (shard < 0 || shard >= (int64_t)pl.tp * pl.pp || id < 0 || id >= oracle_num_logical(m))
        return ORACLE_ERR_ARG;
    decode_id(m, id, &kind, &layer);
    off = pack_offset(m, pl, shard / pl.tp, kind, layer, NULL);
    *held = off >= 0;
    *offset = off >= 0 ? off : 0;
    rank_part(m, pl, kind, shard % pl.tp, r0, nr, c0, nc);
    if (!*held) { *nr = 0; *nc = 0; }
    return ORACLE_OK;
}

/* Distance, in rows of nc elements, from row 0 of a rank's part of logical tensor `id` to its row i. */
int64_t oracle_part_row(const oracle_model* m, oracle_plan pl, int64_t id, int64_t i) {
    int kind; int64_t layer;
    decode_id(m, id, &kind, &layer);
    return part_rowpos(m, pl, kind, i) - part_rowpos(m, pl, kind, 0);
}

/* fp32 -> bf16, round to nearest, ties to even, on the bit pattern.
 * NaN (any payload, either sign) -> 0x7FC0; everything else
 * (u + 0x7FFF + lsb) >> 16, so finite values beyond the bf16 range become
 * +-Inf, signed zeros keep their sign and subnormals are rounded, not flushed.
 * The cast belongs to this build's contract (train -> generation weight sync
 * between the actor's two model-stages, Section 5); the paper states no
 * precision. */
uint16_t oracle_rne_bf16(uint32_t u) {
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return 0x7FC0;
    return (uint16_t)((u + 0x7FFFu + ((u >> 16) & 1u)) >> 16);
}

void oracle_rne_bf16_array(const uint32_t* in, uint16_t* out, int64_t n) {
    for (int64_t i = 0; i < n; ++i) out[i] = oracle_rne_bf16(in[i]);
}

/* One logical tensor: gather -> cast -> slice.
 * src_parts[i] / dst_parts[i] point at the FIRST ELEMENT of shard i's part of
 * this tensor (host memory), or are ignored for shards that do not hold it. */
int oracle_reshard_tensor_parts(const oracle_model* m, oracle_plan sp, oracle_plan dp, int64_t id,
                                const void* const* src_parts, void* const* dst_parts) {
    int rc, held, kind; int64_t layer, rows, cols, off, r0, nr, c0, nc;
    if ((rc = oracle_check_plan(m, sp))) return rc;
    if ((rc = oracle_check_plan(m, dp))) return rc;
    if (id < 0 || id >= oracle_num_logical(m) || !src_parts || !dst_parts) return ORACLE_ERR_ARG;
    int64_t ses = plan_es(m, sp), des = plan_es(m, dp);
    if (!(ses == des || (ses == 4 && des == 2))) return ORACLE_ERR_UNSUPPORTED;
    decode_id(m, id, &kind, &layer);
    kind_shape(m, kind, &rows, &cols);

    unsigned char* full = (unsigned char*)malloc((size_t)(rows * cols * ses));
    if (!full) return ORACLE_ERR_NOMEM;

    /* 1. GATHER.  Parts never overlap partly: a part either covers new ground or repeats, exactly, a region an
     * earlier rank brought (replicated norms and value head; kv heads when tp > kv_heads).  The first copy is
     * taken, every later copy must be identical: all ranks hold the same logical state. */
    int64_t seen_r0[64], seen_c0[64]; int n_seen = 0;
    for (int64_t s = 0; s < (int64_t)sp.tp * sp.pp; ++s) {
        oracle_locate(m, sp, s, id, &held, &off, &r0, &nr, &c0, &nc);
        if (!held) continue;
        const unsigned char* part = (const unsigned char*)src_parts[s];
        if (!part) { free(full); return ORACLE_ERR_ARG; }
        int repeat = 0;
        for (int q = 0; q < n_seen; ++q) repeat |= (seen_r0[q] == r0 && seen_c0[q] == c0);
        /* a guard, not arithmetic: more distinct parts than the record holds (tp > 64) is refused rather than
         * checked against an incomplete record */
        if (!repeat && n_seen == 64) { free(full); return ORACLE_ERR_UNSUPPORTED; }
        for (int64_t i = 0; i < nr; ++i) {
            int64_t at = oracle_part_row(m, sp, id, i);                 /* where the plan's layout keeps row i */
            for (int64_t j = 0; j < nc; ++j) {
                unsigned char* to = full + ((r0 + i) * cols + (c0 + j)) * ses;
                const unsigned char* from = part + (at * nc + j) * ses;
                if (!repeat) memcpy(to, from, (size_t)ses);
                else if (memcmp(to, from, (size_t)ses) != 0) { free(full); return ORACLE_ERR_REPLICA_MISMATCH; }
            }
        }
        if (!repeat) { seen_r0[n_seen] = r0; seen_c0[n_seen] = c0; ++n_seen; }
    }

    /* 2. CAST */
    unsigned char* cast = full;
    if (des != ses) {
        cast = (unsigned char*)malloc((size_t)(rows * cols * des));
        if (!cast) { free(full); return ORACLE_ERR_NOMEM; }
        for (int64_t e = 0; e < rows * cols; ++e) {
            uint32_t u; uint16_t b;
            memcpy(&u, full + e * 4, 4);
            b = oracle_rne_bf16(u);
            memcpy(cast + e * 2, &b, 2);
        }
    }

    /* 3. SLICE */
    for (int64_t d = 0; d < (int64_t)dp.tp * dp.pp; ++d) {
        oracle_locate(m, dp, d, id, &held, &off, &r0, &nr, &c0, &nc);
        if (!held) continue;
        unsigned char* part = (unsigned char*)dst_parts[d];
        if (!part) { if (cast != full) free(cast); free(full); return ORACLE_ERR_ARG; }
        for (int64_t i = 0; i < nr; ++i) {
            int64_t at = oracle_part_row(m, dp, id, i);
            for (int64_t j = 0; j < nc; ++j)
                memcpy(part + (at * nc + j) * des, cast + ((r0 + i) * cols + (c0 + j)) * des, (size_t)des);
        }
    }
    if (cast != full) free(cast);
    free(full);
    return ORACLE_OK;
}

/* Same, addressed by whole shard buffers (host memory). */
int oracle_reshard_tensor(const oracle_model* m, oracle_plan sp, oracle_plan dp, int64_t id,
                          const void* const* src_bufs, void* const* dst_bufs) {
    int rc, held; int64_t off, r0, nr, c0, nc;
    if ((rc = oracle_check_plan(m, sp))) return rc;
    if ((rc = oracle_check_plan(m, dp))) return rc;
    if (!src_bufs || !dst_bufs) return ORACLE_ERR_ARG;
    int64_t ns = (int64_t)sp.tp * sp.pp, nd = (int64_t)dp.tp * dp.pp;
    const void** sparts = (const void**)calloc((size_t)ns, sizeof(void*));
    void** dparts = (void**)calloc((size_t)nd, sizeof(void*));
    if (!sparts || !dparts) { free(sparts); free(dparts); return ORACLE_ERR_NOMEM; }
    for (int64_t s = 0; s < ns; ++s) {
        rc = oracle_locate(m, sp, s, id, &held, &off, &r0, &nr, &c0, &nc);
        if (rc) break;
        sparts[s] = held ? (const unsigned char*)src_bufs[s] + off : NULL;
    }
    for (int64_t d = 0; !rc && d < nd; ++d) {
        rc = oracle_locate(m, dp, d, id, &held, &off, &r0, &nr, &c0, &nc);
        if (rc) break;
        dparts[d] = held ? (unsigned char*)dst_bufs[d] + off : NULL;
    }
    if (!rc) rc = oracle_reshard_tensor_parts(m, sp, dp, id, sparts, dparts);
    free(sparts); free(dparts);
    return rc;
}

/* The whole model-stage: every logical tensor in catalogue order. */
int oracle_reshard(const oracle_model* m, oracle_plan sp, oracle_plan dp,
                   const void* const* src_bufs, void* const* dst_bufs) {
    int rc;
    if ((rc = oracle_check_plan(m, sp))) return rc;
    if ((rc = oracle_check_plan(m, dp))) return rc;
    for (int64_t id = 0; id < oracle_num_logical(m); ++id)
        if ((rc = oracle_reshard_tensor(m, sp, dp, id, src_bufs, dst_bufs))) return rc;
    return ORACLE_OK;
}

/* k identical target units: what Extend leaves behind (Section 5.2(c): the new unit is a
 * copy of theta and omega; use sp == dp) and what a Split into k replica units produces (Section 5.2(a)).  By
 * definition every unit is the plain reshard, so the oracle runs it once per unit.
 * dst_bufs is replica-major: unit 0's tp*pp shards, then unit 1's, ... */
int oracle_reshard_replicated(const oracle_model* m, oracle_plan sp, oracle_plan dp, int replicas,
                              const void* const* src_bufs, void* const* dst_bufs) {
    int rc;
    if (replicas < 1) return ORACLE_ERR_ARG;
    if ((rc = oracle_check_plan(m, dp))) return rc;
    for (int r = 0; r < replicas; ++r)
        if ((rc = oracle_reshard(m, sp, dp, src_bufs, dst_bufs + (int64_t)r * dp.tp * dp.pp))) return rc;
    return ORACLE_OK;
}
