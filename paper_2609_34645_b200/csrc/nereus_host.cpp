// Host side of the EMU reshard: model descriptor, shard layout, and the transition compiler that turns a
// plan difference (source plan -> target plan, the change Delta_M of Section 6.1 of the Nereus paper at
// tensor granularity) into rect-copy tasks.  The map is direct: every destination slice is intersected with
// the source slices that overlap it; no full logical tensor and no intermediate layout is ever formed.
#include <algorithm>
#include <cstring>
#include <new>

#include "nereus_internal.hpp"

using namespace nereus;

namespace nereus {

// ---------------------------------------------------------------------------------------------------
// catalogue
// ---------------------------------------------------------------------------------------------------

static StoredTensor whole(int64_t rows, int64_t cols, int layer) {
    return StoredTensor{Cut::Whole, 1, {rows, 0, 0}, {0, 0, 0}, 0, cols, layer};
}
static StoredTensor by_rows(int nseg, int64_t r0, int64_t r1, int64_t r2, int64_t cols, int layer) {
    return StoredTensor{Cut::Rows, nseg, {r0, r1, r2}, {0, 0, 0}, 0, cols, layer};
}
static StoredTensor by_cols(int64_t rows, int64_t cols, int layer) {
    return StoredTensor{Cut::Cols, 1, {rows, 0, 0}, {0, 0, 0}, 0, cols, layer};
}

void build_catalogue(nereus_model_desc_s& d) {
    const int64_t hd = d.H / d.nq;
    d.catalogue.clear();
    d.catalogue.reserve(6 * d.L + 3);
    d.catalogue.push_back(by_rows(1, d.V, 0, 0, d.H, -1));                                   // embed
    d.catalogue.back().pad_to = 128;
    for (int l = 0; l < d.L; ++l) {
        d.catalogue.push_back(whole(1, d.H, l));                                             // ln1
        d.catalogue.push_back(by_rows(3, d.nq * hd, d.nkv * hd, d.nkv * hd, d.H, l));        // q;k;v
        d.catalogue.back().seg_unit[1] = d.catalogue.back().seg_unit[2] = hd;                // kv heads stay whole
        d.catalogue.push_back(by_cols(d.H, d.nq * hd, l));                                   // wo
        d.catalogue.push_back(whole(1, d.H, l));                                             // ln2
        d.catalogue.push_back(by_rows(2, d.F, d.F, 0, d.H, l));                              // gate;up
        d.catalogue.push_back(by_cols(d.H, d.F, l));                                         // wdown
    }
    d.catalogue.push_back(whole(1, d.H, -2));                                                // ln_f
    d.catalogue.push_back(d.value_head ? whole(1, d.H, -2) : by_rows(1, d.V, 0, 0, d.H, -2)); // head
    if (!d.value_head) d.catalogue.back().pad_to = 128;
}

int check_plan(const nereus_model_desc_s& d, nereus_plan_t p) {
    if (p.tp < 1 || p.pp < 1) return NEREUS_ERR_ARG;
    if (p.dtype != 0 && p.dtype != NEREUS_BF16 && p.dtype != NEREUS_FP32) return NEREUS_ERR_ARG;
    if (p.layout & ~(NEREUS_QKV_GROUPED | NEREUS_GATE_UP_INTERLEAVED | NEREUS_VOCAB_PADDED)) return NEREUS_ERR_ARG;
    // tp <= nkv: whole kv heads per rank; tp > nkv: each kv head replicated on tp/nkv ranks (needs nkv | tp)
    if (p.tp <= d.nkv ? d.nkv % p.tp : p.tp % d.nkv) return NEREUS_ERR_INDIVISIBLE;
    if (d.nq % p.tp || d.F % p.tp) return NEREUS_ERR_INDIVISIBLE;
    if (p.pp > d.L) return NEREUS_ERR_INDIVISIBLE;                   // every stage needs a layer
    if (!(p.layout & NEREUS_VOCAB_PADDED) && d.V % p.tp) return NEREUS_ERR_INDIVISIBLE;
    return NEREUS_OK;
}

int owning_stage(const nereus_model_desc_s& d, int id, int pp) {
    const int layer = d.catalogue[id].layer;
    if (layer == -1) return 0;
    if (layer == -2) return pp - 1;
    // even cut; when pp does not divide L the first L mod pp stages own one layer more
    const int base = (int)(d.L / pp), extra = (int)(d.L % pp), big = extra * (base + 1);
    return layer < big ? layer / (base + 1) : extra + (layer - big) / base;
}

// Rows one rank keeps of a padded segment: the padded total cut evenly.
static int64_t padded_share(const StoredTensor& t, int tp) {
    const int64_t q = t.pad_to * tp;
    return (t.seg_rows[0] + q - 1) / q * q / tp;
}

void stored_block(const StoredTensor& t, int tp, int layout, int64_t& rows, int64_t& cols) {
    if (t.cut == Cut::Rows && t.pad_to && (layout & NEREUS_VOCAB_PADDED)) {
        rows = padded_share(t, tp); cols = t.cols;      // padding rows take room in every shard
        return;
    }
    switch (t.cut) {
    case Cut::Whole: rows = t.seg_rows[0]; cols = t.cols; break;
    case Cut::Cols:  rows = t.seg_rows[0]; cols = t.cols / tp; break;
    case Cut::Rows:
        rows = 0;
        for (int s = 0; s < t.nseg; ++s) rows += std::max(t.seg_rows[s] / tp, t.seg_unit[s]);
        cols = t.cols;
        break;
    }
}

void segment_share(const StoredTensor& t, int s, int r, int tp, int layout, int64_t& lo, int64_t& n,
                   bool& primary) {
    if (t.pad_to && (layout & NEREUS_VOCAB_PADDED)) {
        // the real rows among the rank's share of the padded table (none on ranks that hold padding only)
        const int64_t per = padded_share(t, tp);
        lo = std::min<int64_t>((int64_t)r * per, t.seg_rows[s]);
        n = std::min<int64_t>((int64_t)(r + 1) * per, t.seg_rows[s]) - lo;
        primary = true;
        return;
    }
    const int64_t even = t.seg_rows[s] / tp;
    if (even >= t.seg_unit[s]) { lo = r * even; n = even; primary = true; return; }
    // fewer rows than one unit per rank: units are replicated, `copies` consecutive ranks hold the same unit
    const int64_t copies = (int64_t)tp * t.seg_unit[s] / t.seg_rows[s];
    lo = (r / copies) * t.seg_unit[s];
    n = t.seg_unit[s];
    primary = r % copies == 0;
}

void stage_layout(const nereus_model_desc_s& d, nereus_plan_t p, int stage, StageLayout& out) {
    const uint64_t es = elem_size(plan_dtype(d, p));
    const int n = (int)d.catalogue.size();
    out.offset.assign(n, kNotHeld);
    uint64_t cur = 0;
    for (int id = 0; id < n; ++id) {          // the catalogue order is the packing order
        if (owning_stage(d, id, p.pp) != stage) continue;
        int64_t rows, cols;
        stored_block(d.catalogue[id], p.tp, p.layout, rows, cols);
        cur = round_up(cur, 256);
        out.offset[id] = cur;
        cur += (uint64_t)rows * (uint64_t)cols * es;
    }
    out.bytes = round_up(cur, 256);
}

// ---------------------------------------------------------------------------------------------------
// compiler
// ---------------------------------------------------------------------------------------------------

namespace {

// One run of consecutive logical rows of one segment of a Rows-cut tensor as a TP rank stores it:
// logical rows [lo, lo + n) of segment `seg` sit at stored rows at, at + step, at + 2*step, ...
// primary = false on the later copies of rows that several ranks hold (replicated kv heads): as a source
// only the first copy is read.
struct RowPiece {
    int     seg;
    int64_t lo, n;
    int64_t at, step;
    bool    primary;
};

// How rank r of t keeps a Rows-cut tensor under a layout.  Blocked: one piece per segment, stacked.
// Grouped QKV (3 segments): per kv head of the rank, its q heads, then its K rows, then its V rows.
// Interleaved gate/up (2 segments): rows alternate, step 2.
void row_pieces(const nereus_model_desc_s& d, const StoredTensor& x, int layout, int r, int t,
                std::vector<RowPiece>& out) {
    out.clear();
    int64_t lo[3], n[3]; bool primary[3];
    for (int s = 0; s < x.nseg; ++s) segment_share(x, s, r, t, layout, lo[s], n[s], primary[s]);
    if (x.nseg == 3 && (layout & NEREUS_QKV_GROUPED)) {
        const int64_t hd = d.H / d.nq, heads = n[1] / hd;          // kv heads this rank holds
        const int64_t q_rows = n[0] / heads, group_rows = q_rows + 2 * hd;
        for (int64_t j = 0; j < heads; ++j) {
            out.push_back({0, lo[0] + j * q_rows, q_rows, j * group_rows, 1, primary[0]});
            out.push_back({1, lo[1] + j * hd, hd, j * group_rows + q_rows, 1, primary[1]});
            out.push_back({2, lo[2] + j * hd, hd, j * group_rows + q_rows + hd, 1, primary[2]});
        }
        return;
    }
    if (x.nseg == 2 && (layout & NEREUS_GATE_UP_INTERLEAVED)) {
        out.push_back({0, lo[0], n[0], 0, 2, primary[0]});
        out.push_back({1, lo[1], n[1], 1, 2, primary[1]});
        return;
    }
    int64_t base = 0;
    for (int s = 0; s < x.nseg; ++s) {
        out.push_back({s, lo[s], n[s], base, 1, primary[s]});
        base += n[s];
    }
}

struct Emitter {
    std::vector<Rect>& out;
    bool               misaligned = false;

    void emit(Rect r) {
        const uint64_t ws = r.width_dst << r.cast;
        if (r.rows == 0 || r.width_dst == 0) return;
        // a rect whose pieces touch on both sides is one contiguous run
        if (r.rows > 1 && r.src_pitch == ws && r.dst_pitch == r.width_dst) {
            r.width_dst *= r.rows;
            r.rows = 1;
        }
        if (r.rows == 1) { r.src_pitch = r.width_dst << r.cast; r.dst_pitch = r.width_dst; }
        if ((r.src_off | r.dst_off | r.width_dst | (r.rows > 1 ? (r.src_pitch | r.dst_pitch) : 0)) & 15)
            misaligned = true;
        // extend the previous run when this one continues it on both sides
        if (!out.empty()) {
            Rect& p = out.back();
            if (p.rows == 1 && r.rows == 1 && p.src_buf == r.src_buf && p.dst_buf == r.dst_buf &&
                p.cast == r.cast && p.level == r.level && p.replicas == r.replicas &&
                p.src_off + (p.width_dst << p.cast) == r.src_off && p.dst_off + p.width_dst == r.dst_off) {
                p.width_dst += r.width_dst;
                p.src_pitch = p.width_dst << p.cast;
                p.dst_pitch = p.width_dst;
                return;
            }
        }
        out.push_back(r);
    }
};

}  // namespace

static int compile_one(const nereus_model_desc_s& d, nereus_plan_t sp, nereus_plan_t dp, int replicas,
                       nereus_transition_s& t) {
    const int      sdt = plan_dtype(d, sp), ddt = plan_dtype(d, dp);
    const uint64_t ses = elem_size(sdt), des = elem_size(ddt);
    const int      cast = (sdt != ddt) ? 1 : 0;
    const int      n_src = sp.tp * sp.pp, n_unit = dp.tp * dp.pp, n_dst = n_unit * replicas;
    if (n_src + n_dst > kMaxBuffers) return NEREUS_ERR_UNSUPPORTED;

    std::vector<StageLayout> sl(sp.pp), dl(dp.pp);
    for (int p = 0; p < sp.pp; ++p) stage_layout(d, sp, p, sl[p]);
    for (int p = 0; p < dp.pp; ++p) stage_layout(d, dp, p, dl[p]);
    t.src_bytes.resize(n_src);
    t.dst_bytes.resize(n_dst);
    for (int i = 0; i < n_src; ++i) t.src_bytes[i] = sl[i / sp.tp].bytes;
    for (int i = 0; i < n_dst; ++i) t.dst_bytes[i] = dl[(i % n_unit) / dp.tp].bytes;
    t.dst_level.assign(n_dst, 0);
    t.dst_read_level.assign(n_dst, -1);
    t.n_levels = 1;

    Emitter em{t.rects};
    std::vector<RowPiece> spieces, dpieces;
    const int ts = sp.tp, td = dp.tp;
    for (int pd = 0; pd < dp.pp; ++pd) {
        for (int rd = 0; rd < td; ++rd) {
            const int dst_buf = n_src + pd * td + rd;
            for (int id = 0; id < (int)d.catalogue.size(); ++id) {
                const uint64_t doff = dl[pd].offset[id];
                if (doff == kNotHeld) continue;
                const StoredTensor& x = d.catalogue[id];
                const int      ps   = owning_stage(d, id, sp.pp);
                const uint64_t soff = sl[ps].offset[id];
                Rect r{};
                r.dst_buf = dst_buf; r.level = 0; r.cast = cast;
                r.replicas = replicas; r.replica_stride = replicas > 1 ? n_unit : 0;
                if (x.cut == Cut::Whole) {
                    // replicated state: every copy is the same logical state; read TP rank 0's
                    r.src_buf = ps * ts;
                    r.src_off = soff; r.dst_off = doff;
                    r.rows = 1; r.width_dst = (uint64_t)x.seg_rows[0] * x.cols * des;
                    em.emit(r);
                } else if (x.cut == Cut::Rows) {
                    if (ts == td && sp.layout == dp.layout && !(x.pad_to && (dp.layout & NEREUS_VOCAB_PADDED))) {
                        // same cut and same order on both sides: the rank's stored block moves as one run
                        // (a padded block goes the general way, which leaves its padding rows alone)
                        int64_t brows, bcols;
                        stored_block(x, td, dp.layout, brows, bcols);
                        r.src_buf = ps * ts + rd;
                        r.src_off = soff; r.dst_off = doff;
                        r.rows = 1; r.width_dst = (uint64_t)brows * bcols * des;
                        em.emit(r);
                        continue;
                    }
                    // both sides keep runs of logical rows (row pieces): intersect them segment by segment
                    row_pieces(d, x, dp.layout, rd, td, dpieces);
                    for (int rs = 0; rs < ts; ++rs) {
                        row_pieces(d, x, sp.layout, rs, ts, spieces);
                        for (const RowPiece& q : dpieces) {
                            for (const RowPiece& s : spieces) {
                                if (s.seg != q.seg || !s.primary) continue;
                                const int64_t lo = std::max(q.lo, s.lo), hi = std::min(q.lo + q.n, s.lo + s.n);
                                if (lo >= hi) continue;
                                r.src_buf = ps * ts + rs;
                                r.src_off = soff + (uint64_t)(s.at + (lo - s.lo) * s.step) * x.cols * ses;
                                r.dst_off = doff + (uint64_t)(q.at + (lo - q.lo) * q.step) * x.cols * des;
                                r.rows = (uint64_t)(hi - lo);
                                r.width_dst = (uint64_t)x.cols * des;
                                r.src_pitch = (uint64_t)s.step * x.cols * ses;
                                r.dst_pitch = (uint64_t)q.step * x.cols * des;
                                em.emit(r);       // consecutive rows on both sides collapse to one run
                            }
                        }
                    }
                } else {
                    // every row is cut into column pieces on both sides: intersect column intervals
                    const int64_t K = x.cols, ks = K / ts, kd = K / td;
                    const int64_t d0 = rd * kd, d1 = d0 + kd;
                    for (int rs = 0; rs < ts; ++rs) {
                        const int64_t s0 = rs * ks, s1 = s0 + ks;
                        const int64_t lo = std::max(d0, s0), hi = std::min(d1, s1);
                        if (lo >= hi) continue;
                        r.src_buf = ps * ts + rs;
                        r.src_off = soff + (uint64_t)(lo - s0) * ses;
                        r.dst_off = doff + (uint64_t)(lo - d0) * des;
                        r.src_pitch = (uint64_t)ks * ses; r.dst_pitch = (uint64_t)kd * des;
                        r.rows = (uint64_t)x.seg_rows[0]; r.width_dst = (uint64_t)(hi - lo) * des;
                        em.emit(r);
                    }
                }
            }
        }
    }
    if (em.misaligned) return NEREUS_ERR_INDIVISIBLE;
    return NEREUS_OK;
}

static void finish(nereus_transition_s& t) {
    // execution order: by level, then largest first (stable, so equal tasks keep destination order)
    std::stable_sort(t.rects.begin(), t.rects.end(), [](const Rect& a, const Rect& b) {
        if (a.level != b.level) return a.level < b.level;
        return a.rows * a.width_dst > b.rows * b.width_dst;
    });
    t.bytes_read = t.bytes_written = 0;
    for (const Rect& r : t.rects) {
        t.bytes_written += r.rows * r.width_dst * (uint64_t)r.replicas;
        t.bytes_read += r.rows * (r.width_dst << r.cast);
    }
}

uint64_t tile_table(const nereus_transition_s& t, uint32_t tile_bytes, std::vector<RectDev>& out,
                    std::vector<uint32_t>& first, uint32_t level_end[kMaxLevels]) {
    out.resize(t.rects.size());
    first.resize(t.rects.size() + 1);
    return tile_table_raw(t, tile_bytes, out.data(), first.data(), level_end);
}

uint64_t tile_table_raw(const nereus_transition_s& t, uint32_t tile_bytes, RectDev* out, uint32_t* first,
                        uint32_t level_end[kMaxLevels]) {
    for (int k = 0; k < kMaxLevels; ++k) level_end[k] = 0;
    uint64_t total = 0;
    size_t   i = 0;
    for (const Rect& r : t.rects) {
        RectDev q{};
        q.src_off = r.src_off; q.dst_off = r.dst_off; q.width = r.width_dst;
        q.src_pitch = (uint32_t)r.src_pitch; q.dst_pitch = (uint32_t)r.dst_pitch;
        q.rows = (uint32_t)r.rows;
        q.src_buf = (uint16_t)r.src_buf; q.dst_buf = (uint16_t)r.dst_buf;
        q.level = (uint16_t)r.level; q.cast = (uint16_t)r.cast;
        q.replicas = (uint16_t)r.replicas; q.replica_stride = (uint16_t)r.replica_stride;
        uint64_t ntiles;
        if (r.rows == 1 || r.width_dst >= tile_bytes) {
            q.rows_per_tile = 1;
            q.tile_w = tile_bytes;
            const uint64_t ct = (r.width_dst + tile_bytes - 1) / tile_bytes;
            q.col_tiles = (uint32_t)ct;
            ntiles = ct * r.rows;
        } else {
            q.rows_per_tile = (uint32_t)std::max<uint64_t>(1, tile_bytes / r.width_dst);
            q.tile_w = (uint32_t)r.width_dst;
            q.col_tiles = 1;
            ntiles = (r.rows + q.rows_per_tile - 1) / q.rows_per_tile;
        }
        if (total + ntiles > 0xFFFFFFF0ull) return 0;
        q.first_tile = (uint32_t)total;
        first[i] = (uint32_t)total;
        total += ntiles;
        level_end[r.level] = (uint32_t)total;
        out[i++] = q;
    }
    first[i] = (uint32_t)total;
    for (int k = 1; k < kMaxLevels; ++k) level_end[k] = std::max(level_end[k], level_end[k - 1]);
    return total;
}


void expand_tiles(const RectDev* rects, size_t n_rects, TileRec* out) {
    for (size_t i = 0; i < n_rects; ++i) {
        const RectDev& q = rects[i];
        const uint32_t row_blocks = (q.rows + q.rows_per_tile - 1) / q.rows_per_tile;
        TileRec* o = out + q.first_tile;
        for (uint32_t rb = 0; rb < row_blocks; ++rb) {
            const uint32_t r0 = rb * q.rows_per_tile;
            for (uint32_t cb = 0; cb < q.col_tiles; ++cb) {
                const uint64_t c0 = (uint64_t)cb * q.tile_w;
                TileRec e{};
                e.src_off = q.src_off + (uint64_t)r0 * q.src_pitch + (c0 << q.cast);
                e.dst_off = q.dst_off + (uint64_t)r0 * q.dst_pitch + c0;
                e.src_pitch = q.src_pitch; e.dst_pitch = q.dst_pitch;
                e.rows = std::min(q.rows_per_tile, q.rows - r0);
                e.width = (uint32_t)std::min<uint64_t>(q.tile_w, q.width - c0);
                e.src_buf = q.src_buf; e.dst_buf = q.dst_buf;
                e.replicas = q.replicas; e.replica_stride = q.replica_stride;
                e.level = q.level; e.cast = q.cast;
                *o++ = e;
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------------
// validator
// ---------------------------------------------------------------------------------------------------

namespace {

typedef unsigned __int128 u128;

// Last byte + 1 that a task touches in a buffer, from its first piece.
inline u128 extent(uint64_t off, uint64_t rows, uint64_t pitch, uint64_t width) {
    return (u128)off + (u128)(rows - 1) * pitch + width;
}

// Two destination footprints in one buffer whose bounding intervals overlap: do any of their pieces?
bool pieces_overlap(const Rect& a, const Rect& b) {
    if (a.rows == 1 && b.rows == 1) return true;
    const Rect& lo = a.dst_off <= b.dst_off ? a : b;
    const Rect& hi = a.dst_off <= b.dst_off ? b : a;
    if (lo.rows > 1 && hi.rows > 1 && lo.dst_pitch == hi.dst_pitch) {
        // same period: the later task's pieces sit in the gaps of the earlier one's, or they do not
        const uint64_t d = (hi.dst_off - lo.dst_off) % lo.dst_pitch;
        if (d >= lo.width_dst && d + hi.width_dst <= lo.dst_pitch) return false;
    }
    uint64_t i = 0, j = 0;                                   // exact: merge the two piece sequences
    while (i < a.rows && j < b.rows) {
        const u128 as = (u128)a.dst_off + (u128)i * a.dst_pitch, ae = as + a.width_dst;
        const u128 bs = (u128)b.dst_off + (u128)j * b.dst_pitch, be = bs + b.width_dst;
        if (ae <= bs) ++i; else if (be <= as) ++j; else return true;
    }
    return false;
}

}  // namespace

int validate_table(const nereus_transition_s& t, const RectDev* tiled, const uint32_t* first, uint64_t n_tiles,
                   uint32_t* order) {
    const size_t ns = t.src_bytes.size(), nd = t.dst_bytes.size(), n = t.rects.size();
    if (ns + nd > (size_t)kMaxBuffers || t.n_levels < 1 || t.n_levels > kMaxLevels) return NEREUS_ERR_TABLE;
    if (t.dst_level.size() != nd) return NEREUS_ERR_TABLE;
    int    prev_level = 0;
    size_t n_entries = 0;
    for (size_t i = 0; i < n; ++i) {
        const Rect& r = t.rects[i];
        if (r.level < prev_level || r.level >= t.n_levels) return NEREUS_ERR_TABLE;      // execution order
        prev_level = r.level;
        if ((r.cast != 0 && r.cast != 1) || r.rows == 0 || r.width_dst == 0 || (r.rows >> 32)) return NEREUS_ERR_TABLE;
        if (r.replicas < 1 || r.replicas > kMaxReplicas || r.replica_stride < 0 ||
            (r.replicas > 1 && r.replica_stride < 1)) return NEREUS_ERR_TABLE;
        if (r.src_buf < 0 || (size_t)r.src_buf >= ns + nd) return NEREUS_ERR_TABLE;
        if (r.dst_buf < (int64_t)ns ||
            (size_t)r.dst_buf + (size_t)(r.replicas - 1) * r.replica_stride >= ns + nd) return NEREUS_ERR_TABLE;
        const uint64_t ws = r.width_dst << r.cast;
        if ((r.src_off | r.dst_off | r.width_dst) & 15) return NEREUS_ERR_TABLE;
        if (r.rows > 1) {
            if ((r.src_pitch | r.dst_pitch) & 15) return NEREUS_ERR_TABLE;
            if (r.src_pitch < ws || r.dst_pitch < r.width_dst) return NEREUS_ERR_TABLE;   // pieces would overlap
            if ((r.src_pitch >> 32) || (r.dst_pitch >> 32)) return NEREUS_ERR_TABLE;      // device form holds 32 bits
        }
        const uint64_t sbytes = (size_t)r.src_buf < ns ? t.src_bytes[r.src_buf] : t.dst_bytes[r.src_buf - ns];
        if (extent(r.src_off, r.rows, r.src_pitch, ws) > sbytes) return NEREUS_ERR_TABLE;
        // a chained task reads what an earlier level wrote, never its own level's output
        if ((size_t)r.src_buf >= ns && t.dst_level[r.src_buf - ns] >= r.level) return NEREUS_ERR_TABLE;
        for (int j = 0; j < r.replicas; ++j) {
            const size_t d = (size_t)r.dst_buf - ns + (size_t)j * r.replica_stride;
            if (extent(r.dst_off, r.rows, r.dst_pitch, r.width_dst) > t.dst_bytes[d]) return NEREUS_ERR_TABLE;
            if (t.dst_level[d] != r.level) return NEREUS_ERR_TABLE;
        }
        n_entries += (size_t)r.replicas;
        if (tiled) {
            const RectDev& q = tiled[i];
            if (q.src_off != r.src_off || q.dst_off != r.dst_off || q.width != r.width_dst || q.rows != r.rows ||
                q.src_buf != r.src_buf || q.dst_buf != r.dst_buf || q.level != r.level || q.cast != r.cast ||
                q.replicas != r.replicas || q.replica_stride != r.replica_stride ||
                (r.rows > 1 && (q.src_pitch != r.src_pitch || q.dst_pitch != r.dst_pitch)))
                return NEREUS_ERR_TABLE;
            if (q.rows_per_tile == 0 || q.tile_w == 0 || q.col_tiles == 0 || (q.tile_w & 15)) return NEREUS_ERR_TABLE;
            if (q.col_tiles > 1 && q.rows_per_tile != 1) return NEREUS_ERR_TABLE;
            if ((uint64_t)q.col_tiles * q.tile_w < q.width || (uint64_t)(q.col_tiles - 1) * q.tile_w >= q.width)
                return NEREUS_ERR_TABLE;
            const uint64_t row_blocks = ((uint64_t)q.rows + q.rows_per_tile - 1) / q.rows_per_tile;
            if (q.first_tile != first[i] || (uint64_t)first[i] + row_blocks * q.col_tiles != first[i + 1])
                return NEREUS_ERR_TABLE;
        }
    }
    if (tiled && first[n] != n_tiles) return NEREUS_ERR_TABLE;

    // destinations pairwise disjoint: one entry per (task, replica), sorted by buffer and first byte; an entry is
    // compared with the later ones that start inside its bounding interval
    size_t k = 0;
    for (size_t i = 0; i < n; ++i)
        for (int j = 0; j < t.rects[i].replicas; ++j) order[k++] = (uint32_t)i | ((uint32_t)j << 24);
    auto buf_of = [&t](uint32_t e) {
        const Rect& r = t.rects[e & 0xFFFFFFu];
        return (uint32_t)(r.dst_buf + (int)(e >> 24) * r.replica_stride);
    };
    std::sort(order, order + n_entries, [&](uint32_t x, uint32_t y) {
        const uint32_t bx = buf_of(x), by = buf_of(y);
        if (bx != by) return bx < by;
        return t.rects[x & 0xFFFFFFu].dst_off < t.rects[y & 0xFFFFFFu].dst_off;
    });
    for (size_t a = 0; a < n_entries; ++a) {
        const Rect& ra = t.rects[order[a] & 0xFFFFFFu];
        const u128  end = extent(ra.dst_off, ra.rows, ra.dst_pitch, ra.width_dst);
        for (size_t b = a + 1; b < n_entries && buf_of(order[b]) == buf_of(order[a]); ++b) {
            const Rect& rb = t.rects[order[b] & 0xFFFFFFu];
            if ((u128)rb.dst_off >= end) break;
            if (pieces_overlap(ra, rb)) return NEREUS_ERR_TABLE;
        }
    }
    return NEREUS_OK;
}

}  // namespace nereus

// ---------------------------------------------------------------------------------------------------
// C ABI: descriptor, layout queries, compiler
// ---------------------------------------------------------------------------------------------------

#define NEREUS_GUARD_BEGIN try {
#define NEREUS_GUARD_END   } catch (const std::bad_alloc&) { return NEREUS_ERR_NOMEM; } catch (...) { return NEREUS_ERR_ARG; }

extern "C" {

int nereus_model_desc(int layers, int hidden, int heads, int kv_heads, int ffn, int vocab, int dtype,
                      nereus_model_desc_t* out) {
    NEREUS_GUARD_BEGIN
    if (!out || layers < 1 || hidden < 1 || heads < 1 || kv_heads < 1 || ffn < 1 || vocab < 1) return NEREUS_ERR_ARG;
    if (dtype != NEREUS_BF16 && dtype != NEREUS_FP32) return NEREUS_ERR_ARG;
    if (hidden % heads || heads % kv_heads) return NEREUS_ERR_INDIVISIBLE;
    auto* d = new nereus_model_desc_s{layers, hidden, heads, kv_heads, ffn, vocab, dtype, false, {}};
    build_catalogue(*d);
    *out = d;
    return NEREUS_OK;
    NEREUS_GUARD_END
}

int nereus_model_desc_set_value_head(nereus_model_desc_t d, int out_dim) {
    NEREUS_GUARD_BEGIN
    if (!d) return NEREUS_ERR_ARG;
    if (out_dim != 1) return NEREUS_ERR_UNSUPPORTED;
    d->value_head = true;
    build_catalogue(*d);
    return NEREUS_OK;
    NEREUS_GUARD_END
}

int nereus_model_desc_destroy(nereus_model_desc_t d) {
    if (!d) return NEREUS_ERR_ARG;
    delete d;
    return NEREUS_OK;
}

int nereus_plan_check(nereus_model_desc_t d, nereus_plan_t p) {
    if (!d) return NEREUS_ERR_ARG;
    return check_plan(*d, p);
}

int nereus_plan_num_shards(nereus_model_desc_t d, nereus_plan_t p, int* n) {
    if (!d || !n) return NEREUS_ERR_ARG;
    if (int rc = check_plan(*d, p)) return rc;
    *n = p.tp * p.pp;
    return NEREUS_OK;
}

int nereus_plan_shard_bytes(nereus_model_desc_t d, nereus_plan_t p, int shard, size_t* bytes) {
    NEREUS_GUARD_BEGIN
    if (!d || !bytes) return NEREUS_ERR_ARG;
    if (int rc = check_plan(*d, p)) return rc;
    if (shard < 0 || shard >= p.tp * p.pp) return NEREUS_ERR_ARG;
    StageLayout sl;
    stage_layout(*d, p, shard / p.tp, sl);
    *bytes = (size_t)sl.bytes;
    return NEREUS_OK;
    NEREUS_GUARD_END
}

int nereus_model_num_tensors(nereus_model_desc_t d, int* n) {
    if (!d || !n) return NEREUS_ERR_ARG;
    *n = (int)d->catalogue.size();
    return NEREUS_OK;
}

int nereus_plan_tensor_slice(nereus_model_desc_t d, nereus_plan_t p, int shard, int tensor_id, size_t* offset,
                             size_t* rows, size_t* cols, int* replicated) {
    NEREUS_GUARD_BEGIN
    if (!d || !offset || !rows || !cols) return NEREUS_ERR_ARG;
    if (int rc = check_plan(*d, p)) return rc;
    if (shard < 0 || shard >= p.tp * p.pp || tensor_id < 0 || tensor_id >= (int)d->catalogue.size())
        return NEREUS_ERR_ARG;
    StageLayout sl;
    stage_layout(*d, p, shard / p.tp, sl);
    if (replicated) *replicated = d->catalogue[tensor_id].cut == Cut::Whole;
    if (sl.offset[tensor_id] == kNotHeld) { *offset = 0; *rows = 0; *cols = 0; return NEREUS_OK; }
    int64_t r, c;
    stored_block(d->catalogue[tensor_id], p.tp, p.layout, r, c);
    *offset = (size_t)sl.offset[tensor_id]; *rows = (size_t)r; *cols = (size_t)c;
    return NEREUS_OK;
    NEREUS_GUARD_END
}

int nereus_transition_compile(nereus_model_desc_t d, nereus_plan_t sp, nereus_plan_t dp, nereus_transition_t* out) {
    NEREUS_GUARD_BEGIN
    if (!d || !out) return NEREUS_ERR_ARG;
    if (int rc = check_plan(*d, sp)) return rc;
    if (int rc = check_plan(*d, dp)) return rc;
    const int sdt = plan_dtype(*d, sp), ddt = plan_dtype(*d, dp);
    if (!(sdt == ddt || (sdt == NEREUS_FP32 && ddt == NEREUS_BF16))) return NEREUS_ERR_UNSUPPORTED;
    auto* t = new nereus_transition_s();
    if (int rc = compile_one(*d, sp, dp, 1, *t)) { delete t; return rc; }
    finish(*t);
    *out = t;
    return NEREUS_OK;
    NEREUS_GUARD_END
}

int nereus_transition_compile_replicated(nereus_model_desc_t d, nereus_plan_t sp, nereus_plan_t dp, int replicas,
                                         nereus_transition_t* out) {
    NEREUS_GUARD_BEGIN
    if (!d || !out || replicas < 1 || replicas > kMaxReplicas) return NEREUS_ERR_ARG;
    if (int rc = check_plan(*d, sp)) return rc;
    if (int rc = check_plan(*d, dp)) return rc;
    const int sdt = plan_dtype(*d, sp), ddt = plan_dtype(*d, dp);
    if (!(sdt == ddt || (sdt == NEREUS_FP32 && ddt == NEREUS_BF16))) return NEREUS_ERR_UNSUPPORTED;
    auto* t = new nereus_transition_s();
    if (int rc = compile_one(*d, sp, dp, replicas, *t)) { delete t; return rc; }
    finish(*t);
    *out = t;
    return NEREUS_OK;
    NEREUS_GUARD_END
}

int nereus_transition_compile_state(nereus_model_desc_t d, nereus_plan_t sp, nereus_plan_t dp, int n_opt,
                                    nereus_transition_t* out) {
    NEREUS_GUARD_BEGIN
    if (!d || !out || n_opt < 0 || n_opt > 8) return NEREUS_ERR_ARG;
    nereus_transition_t parts[9] = {nullptr};
    int rc = nereus_transition_compile(d, sp, dp, &parts[0]);
    nereus_plan_t so = sp, dO = dp;
    so.dtype = NEREUS_FP32; dO.dtype = NEREUS_FP32;      // omega: fp32 on both sides, same (tp, pp) and layout
    for (int k = 0; rc == NEREUS_OK && k < n_opt; ++k) rc = nereus_transition_compile(d, so, dO, &parts[1 + k]);
    if (rc == NEREUS_OK) rc = nereus_transition_fuse(parts, 1 + n_opt, 0, out);
    for (int k = 0; k < 9; ++k)
        if (parts[k]) nereus_transition_destroy(parts[k]);
    return rc;
    NEREUS_GUARD_END
}

int nereus_transition_fuse(const nereus_transition_t* parts, int n, int chained, nereus_transition_t* out) {
    NEREUS_GUARD_BEGIN
    if (!parts || n < 1 || !out) return NEREUS_ERR_ARG;
    for (int i = 0; i < n; ++i)
        if (!parts[i] || parts[i]->n_levels != 1) return NEREUS_ERR_ARG;     // fuse takes compiled parts only
    if (chained && n > kMaxLevels) return NEREUS_ERR_UNSUPPORTED;
    auto* t = new nereus_transition_s();
    if (!chained) {
        size_t ns = 0, nd = 0;
        for (int i = 0; i < n; ++i) { ns += parts[i]->src_bytes.size(); nd += parts[i]->dst_bytes.size(); }
        if (ns + nd > (size_t)kMaxBuffers) { delete t; return NEREUS_ERR_UNSUPPORTED; }
        size_t so = 0, dof = 0;
        for (int i = 0; i < n; ++i) {
            const nereus_transition_s& p = *parts[i];
            const int pns = (int)p.src_bytes.size();
            for (Rect r : p.rects) {
                r.src_buf = (int32_t)(so + r.src_buf);
                r.dst_buf = (int32_t)(ns + dof + (r.dst_buf - pns));
                t->rects.push_back(r);
            }
            t->src_bytes.insert(t->src_bytes.end(), p.src_bytes.begin(), p.src_bytes.end());
            t->dst_bytes.insert(t->dst_bytes.end(), p.dst_bytes.begin(), p.dst_bytes.end());
            so += p.src_bytes.size(); dof += p.dst_bytes.size();
        }
        t->dst_level.assign(nd, 0);
        t->dst_read_level.assign(nd, -1);
        t->n_levels = 1;
    } else {
        for (int i = 1; i < n; ++i)
            if (parts[i]->src_bytes != parts[i - 1]->dst_bytes) { delete t; return NEREUS_ERR_MISMATCH; }
        const size_t ns = parts[0]->src_bytes.size();
        size_t nd = 0;
        for (int i = 0; i < n; ++i) nd += parts[i]->dst_bytes.size();
        if (ns + nd > (size_t)kMaxBuffers) { delete t; return NEREUS_ERR_UNSUPPORTED; }
        t->src_bytes = parts[0]->src_bytes;
        size_t prev_base = 0;      // unified index of the buffers level k reads
        size_t dof = 0;            // destinations emitted so far
        for (int i = 0; i < n; ++i) {
            const nereus_transition_s& p = *parts[i];
            const int pns = (int)p.src_bytes.size();
            for (Rect r : p.rects) {
                r.src_buf = (int32_t)(prev_base + r.src_buf);
                r.dst_buf = (int32_t)(ns + dof + (r.dst_buf - pns));
                r.level = i;
                t->rects.push_back(r);
            }
            for (size_t j = 0; j < p.dst_bytes.size(); ++j) {
                t->dst_bytes.push_back(p.dst_bytes[j]);
                t->dst_level.push_back(i);
                t->dst_read_level.push_back(i + 1 < n ? i + 1 : -1);
            }
            prev_base = ns + dof;
            dof += p.dst_bytes.size();
        }
        t->n_levels = n;
    }
    finish(*t);
    *out = t;
    return NEREUS_OK;
    NEREUS_GUARD_END
}

int nereus_transition_num_buffers(nereus_transition_t t, int* n_src, int* n_dst) {
    if (!t || !n_src || !n_dst) return NEREUS_ERR_ARG;
    *n_src = (int)t->src_bytes.size(); *n_dst = (int)t->dst_bytes.size();
    return NEREUS_OK;
}

int nereus_transition_buffer_bytes(nereus_transition_t t, int is_dst, int index, size_t* bytes) {
    if (!t || !bytes || index < 0) return NEREUS_ERR_ARG;
    const std::vector<uint64_t>& v = is_dst ? t->dst_bytes : t->src_bytes;
    if ((size_t)index >= v.size()) return NEREUS_ERR_ARG;
    *bytes = (size_t)v[index];
    return NEREUS_OK;
}

int nereus_transition_bytes(nereus_transition_t t, size_t* read, size_t* written) {
    if (!t || !read || !written) return NEREUS_ERR_ARG;
    *read = (size_t)t->bytes_read; *written = (size_t)t->bytes_written;
    return NEREUS_OK;
}

int nereus_transition_num_rects(nereus_transition_t t, int* n) {
    if (!t || !n) return NEREUS_ERR_ARG;
    *n = (int)t->rects.size();
    return NEREUS_OK;
}

int nereus_transition_get_rect(nereus_transition_t t, int index, nereus_rect_t* out) {
    if (!t || !out || index < 0 || (size_t)index >= t->rects.size()) return NEREUS_ERR_ARG;
    const Rect& r = t->rects[index];
    out->src_buf = r.src_buf; out->dst_buf = r.dst_buf; out->level = r.level; out->cast = r.cast;
    out->src_off = r.src_off; out->dst_off = r.dst_off;
    out->src_pitch = r.src_pitch; out->dst_pitch = r.dst_pitch;
    out->rows = r.rows;
    out->width_bytes_dst = r.width_dst; out->width_bytes_src = r.width_dst << r.cast;
    out->replicas = r.replicas; out->replica_stride = r.replica_stride;
    return NEREUS_OK;
}

int nereus_transition_validate(nereus_transition_t t) {
    NEREUS_GUARD_BEGIN
    if (!t) return NEREUS_ERR_ARG;
    size_t entries = 0;
    for (const Rect& r : t->rects) entries += (size_t)std::max(1, std::min(r.replicas, kMaxReplicas));
    if (t->rects.size() >= (1u << 24)) return NEREUS_ERR_UNSUPPORTED;
    std::vector<uint32_t> order(entries + 1);
    return validate_table(*t, nullptr, nullptr, 0, order.data());
    NEREUS_GUARD_END
}

int nereus_debug_set_rect(nereus_transition_t t, int index, const nereus_rect_t* in) {
    if (!t || !in || index < 0 || (size_t)index >= t->rects.size()) return NEREUS_ERR_ARG;
    if (t->dev.rects) return NEREUS_ERR_UNSUPPORTED;          // only before the table has reached a device
    Rect& r = t->rects[index];
    r.src_buf = in->src_buf; r.dst_buf = in->dst_buf; r.level = in->level; r.cast = in->cast;
    r.src_off = in->src_off; r.dst_off = in->dst_off;
    r.src_pitch = in->src_pitch; r.dst_pitch = in->dst_pitch;
    r.rows = in->rows; r.width_dst = in->width_bytes_dst;
    r.replicas = in->replicas; r.replica_stride = in->replica_stride;
    return NEREUS_OK;
}

int nereus_dag_lower(nereus_dag_t dag, const nereus_model_desc_t* descs, int n_descs, nereus_transition_t* out) {
    NEREUS_GUARD_BEGIN
    if (!dag || !descs || !out || !dag->scheduled || n_descs != (int)dag->stages.size()) return NEREUS_ERR_ARG;
    for (int m = 0; m < n_descs; ++m)
        if (!descs[m]) return NEREUS_ERR_ARG;
    const int n_units = (int)dag->units.size();
    // which units are inputs (never created) and where each unit's shards start in the unified buffer list
    std::vector<int> producer(n_units, -1);
    for (size_t i = 0; i < dag->prims.size(); ++i)
        for (int u : dag->prims[i].dst) producer[u] = (int)i;
    std::vector<int> base(n_units, -1);
    int n_src = 0, n_all = 0;
    for (int u = 0; u < n_units; ++u)
        if (producer[u] < 0) { base[u] = n_src; n_src += dag->units[u].tp * dag->units[u].pp; }
    n_all = n_src;
    for (int u = 0; u < n_units; ++u)
        if (producer[u] >= 0) { base[u] = n_all; n_all += dag->units[u].tp * dag->units[u].pp; }
    if (n_all > kMaxBuffers) return NEREUS_ERR_UNSUPPORTED;

    // dependency levels of the data-moving primitives, renumbered densely
    std::vector<int> used_levels;
    for (const PrimRec& p : dag->prims)
        if (p.op != NEREUS_OP_DESTROY) used_levels.push_back(p.level);
    std::sort(used_levels.begin(), used_levels.end());
    used_levels.erase(std::unique(used_levels.begin(), used_levels.end()), used_levels.end());
    if ((int)used_levels.size() > kMaxLevels) return NEREUS_ERR_UNSUPPORTED;
    auto level_of = [&](const PrimRec& p) {
        return (int)(std::lower_bound(used_levels.begin(), used_levels.end(), p.level) - used_levels.begin());
    };

    auto* t = new nereus_transition_s();
    t->src_bytes.assign(n_src, 0);
    t->src_read_level.assign(n_src, 0);
    t->dst_bytes.assign(n_all - n_src, 0);
    t->dst_level.assign(n_all - n_src, 0);
    t->dst_read_level.assign(n_all - n_src, -1);
    auto plan_of = [](const UnitRec& u) { return nereus_plan_t{u.tp, u.pp, 0, 0}; };
    int rc = NEREUS_OK;
    for (const PrimRec& p : dag->prims) {
        if (p.op == NEREUS_OP_DESTROY) continue;
        const nereus_model_desc_s& d = *descs[p.stage];
        const UnitRec& su = dag->units[p.src[0]];
        const UnitRec& du = dag->units[p.dst[0]];
        const int k = p.op == NEREUS_OP_SPLIT ? (int)p.dst.size() : 1;
        nereus_transition_s part;
        if ((rc = check_plan(d, plan_of(su))) || (rc = check_plan(d, plan_of(du)))) break;
        if ((rc = compile_one(d, plan_of(su), plan_of(du), 1, part))) break;
        const int ns = su.tp * su.pp, nd = du.tp * du.pp, lvl = level_of(p);
        const int sub = su.tp * su.pp;                 // Merge: GPUs per sub-unit = shards per sub-unit
        for (int i = 0; i < ns; ++i)
            for (int u : p.src) {
                if (producer[u] < 0) {
                    t->src_bytes[base[u] + i] = part.src_bytes[i];
                    t->src_read_level[base[u] + i] = std::max(t->src_read_level[base[u] + i], lvl);
                }
                else t->dst_read_level[base[u] - n_src + i] = std::max(t->dst_read_level[base[u] - n_src + i], lvl);
            }
        for (int u : p.dst)
            for (int j = 0; j < nd; ++j) {
                t->dst_bytes[base[u] - n_src + j] = part.dst_bytes[j];
                t->dst_level[base[u] - n_src + j] = lvl;
            }
        for (Rect r : part.rects) {
            const int shard_s = r.src_buf, shard_d = r.dst_buf - ns;
            // Merge cuts target shard j from the sub-unit on the same GPU; Split and Extend read their one source
            const int src_unit = p.op == NEREUS_OP_MERGE ? p.src[shard_d / sub] : p.src[0];
            r.src_buf = base[src_unit] + shard_s;
            r.dst_buf = base[p.dst[0]] + shard_d;
            r.level = lvl;
            if (k > 1) {
                // the k sub-units are created one after another, so their buffers are nd apart
                r.replicas = k;
                r.replica_stride = nd;
            }
            t->rects.push_back(r);
        }
    }
    if (rc) { delete t; return rc; }
    t->n_levels = std::max<int>(1, (int)used_levels.size());
    finish(*t);
    *out = t;
    return NEREUS_OK;
    NEREUS_GUARD_END
}

int nereus_transition_estimate(nereus_transition_t t, double gbytes_per_s, double setup_seconds, double* seconds) {
    if (!t || !seconds || !(gbytes_per_s > 0.0) || !(setup_seconds >= 0.0)) return NEREUS_ERR_ARG;
    // levels are serial; within a level everything streams at the given bandwidth
    double bytes = 0.0;
    for (const Rect& r : t->rects)
        bytes += (double)(r.rows * (r.width_dst << r.cast)) + (double)(r.rows * r.width_dst) * r.replicas;
    *seconds = setup_seconds + bytes / (gbytes_per_s * 1e9);
    return NEREUS_OK;
}

int nereus_admit(double l_tran, double l_step_current, double l_step_target, double gamma, double h_x, int urgent,
                 int* admit, double* payback_steps) {
    if (!admit || !(l_tran >= 0.0) || !(gamma >= 0.0 && gamma <= 1.0) || !(h_x >= 0.0)) return NEREUS_ERR_ARG;
    const double delta_l = l_step_current - l_step_target;
    const double inf = 1.0 / 0.0;
    const double payback = delta_l > 0.0 ? l_tran / delta_l : inf;
    if (payback_steps) *payback_steps = payback;
    *admit = urgent ? 1 : (delta_l > 0.0 && payback <= gamma * h_x && gamma > 0.0 ? 1 : 0);
    return NEREUS_OK;
}

int nereus_horizon_init(nereus_horizon_t* h, double weight) {
    if (!h || !(weight > 0.0 && weight <= 1.0)) return NEREUS_ERR_ARG;
    h->h_steps = 1.0;            // before the first interval is observed
    h->weight = weight;
    h->observed = 0;
    return NEREUS_OK;
}

int nereus_horizon_crossing(nereus_horizon_t* h, double interval_steps) {
    if (!h || !(interval_steps >= 0.0) || !(h->weight > 0.0 && h->weight <= 1.0)) return NEREUS_ERR_ARG;
    h->h_steps = h->observed ? (1.0 - h->weight) * h->h_steps + h->weight * interval_steps : interval_steps;
    h->observed += 1;
    return NEREUS_OK;
}

const char* nereus_strerror(int code) {
    switch (code) {
    case NEREUS_OK:              return "ok";
    case NEREUS_ERR_ARG:         return "invalid argument";
    case NEREUS_ERR_INDIVISIBLE: return "plan does not divide the model, or a piece is not a multiple of 16 bytes";
    case NEREUS_ERR_UNSUPPORTED: return "unsupported dtype pair, too many buffers or levels, or a call that is not allowed here";
    case NEREUS_ERR_ALIAS:       return "a destination buffer overlaps a source or another destination";
    case NEREUS_ERR_CUDA:        return "a CUDA call failed";
    case NEREUS_ERR_NOMEM:       return "out of host memory";
    case NEREUS_ERR_MISMATCH:    return "chained parts do not connect";
    case NEREUS_ERR_ALIGN:       return "a shard pointer is not 16-byte aligned";
    case NEREUS_ERR_INFEASIBLE:  return "the transition DAG cannot be scheduled: an acquisition stays blocked";
    case NEREUS_ERR_TOO_LARGE:   return "the transition has more tasks than the fixed scratch of run_static holds";
    case NEREUS_ERR_TABLE:       return "the task table failed validation: a task leaves its buffers or two tasks collide";
    case NEREUS_ERR_TOO_SMALL:   return "a shard buffer is shorter than the transition requires";
    default:                     return "unknown error";
    }
}

}  // extern "C"
