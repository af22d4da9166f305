// Internal types shared by the layout, the transition compiler and the launcher.  Not installed.
#pragma once

#include <cstdint>
#include <cstddef>
#include <vector>

#include "nereus.h"

namespace nereus {

// ---------------------------------------------------------------------------------------------------
// Model descriptor and the catalogue of stored tensors
// ---------------------------------------------------------------------------------------------------

// How a stored tensor is cut over TP ranks.
enum class Cut : int {
    Whole = 0,   // replicated: every TP rank stores the whole tensor            (norms, value head)
    Rows  = 1,   // dim-0: one or more stacked segments, each cut by rows         (embed, head, qkv, gate_up)
    Cols  = 2,   // dim-1: every row is cut into tp column pieces                 (wo, wdown)
};

// A stored tensor of the catalogue, before any plan is applied.
struct StoredTensor {
    Cut     cut;
    int     nseg;        // Rows: number of stacked segments (1, 2 or 3); otherwise 1
    int64_t seg_rows[3]; // Rows: logical rows of each segment; Whole/Cols: seg_rows[0] = rows
    int64_t seg_unit[3]; // Rows: smallest block of rows a rank may hold (head_dim for K and V, else 0): when a
                         //       rank's share would be smaller, the block is replicated over ranks instead
    int64_t pad_to;      // Rows, one segment: with NEREUS_VOCAB_PADDED the rows are padded to a multiple of
                         //       pad_to * tp before the cut (128 for embed and LM head, else 0)
    int64_t cols;        // logical columns (the contiguous dimension)
    int     layer;       // owning layer, -1 embed (first stage), -2 final norm / head (last stage)
};

}  // namespace nereus

struct nereus_model_desc_s {
    int64_t L, H, nq, nkv, F, V;
    int     dtype;
    bool    value_head;
    std::vector<nereus::StoredTensor> catalogue;   // 6L + 3 entries, in stored-id order
};

namespace nereus {

inline int      elem_size(int dtype) { return dtype == NEREUS_FP32 ? 4 : 2; }
inline int      plan_dtype(const nereus_model_desc_s& d, nereus_plan_t p) { return p.dtype ? p.dtype : d.dtype; }
inline uint64_t round_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

void build_catalogue(nereus_model_desc_s& d);
int  check_plan(const nereus_model_desc_s& d, nereus_plan_t p);

// Byte layout of the shards of one pipeline stage under one plan (identical for all TP ranks of the stage).
struct StageLayout {
    std::vector<uint64_t> offset;   // per stored id; kNotHeld when the stage does not own the tensor
    uint64_t              bytes;    // buffer length
};
constexpr uint64_t kNotHeld = ~0ull;

// Stage that owns stored tensor `id` under a plan with `pp` stages.
int  owning_stage(const nereus_model_desc_s& d, int id, int pp);
void stage_layout(const nereus_model_desc_s& d, nereus_plan_t p, int stage, StageLayout& out);
// Rows x cols (elements) of the block one TP rank of `tp` stores for tensor `t`.
void stored_block(const StoredTensor& t, int tp, int layout, int64_t& rows, int64_t& cols);
// Segment s of a Rows-cut tensor on rank r of t: first logical row, row count, and whether r is the first
// rank holding these rows (false on the later copies of a replicated block).
void segment_share(const StoredTensor& t, int s, int r, int tp, int layout, int64_t& lo, int64_t& n, bool& primary);

// ---------------------------------------------------------------------------------------------------
// Task table
// ---------------------------------------------------------------------------------------------------

// Host form of one rect-copy task.  Widths and pitches in bytes; width_src = width_dst << cast.
struct Rect {
    int32_t  src_buf, dst_buf;   // unified buffer indices: [sources..., destinations...]
    int32_t  level;
    int32_t  cast;
    uint64_t src_off, dst_off;
    uint64_t src_pitch, dst_pitch;
    uint64_t rows;
    uint64_t width_dst;
    int32_t  replicas = 1;       // the piece is written to `replicas` buffers: dst_buf + j * replica_stride
    int32_t  replica_stride = 0;
};

// Device form, 64 bytes.  A rect is cut into tiles of rows_per_tile rows x tile_w bytes (dst side);
// tile g of the table belongs to the rect with first_tile <= g < first_tile of the next rect.
struct alignas(16) RectDev {
    uint64_t src_off, dst_off;
    uint64_t width;          // dst bytes per row piece
    uint32_t src_pitch, dst_pitch;
    uint32_t rows, rows_per_tile;
    uint32_t tile_w;         // dst bytes per column tile
    uint32_t col_tiles;
    uint32_t first_tile;
    uint16_t src_buf, dst_buf;
    uint16_t level, cast;
    uint16_t replicas, replica_stride;
};
static_assert(sizeof(RectDev) == 64, "RectDev must stay 64 bytes");

// One tile, resolved on the host: tables of up to kDirectMaxTiles tiles carry one record per tile, so that a
// claimer reaches its addresses with one load instead of a search through the tile prefix.  48 bytes.
struct alignas(16) TileRec {
    uint64_t src_off, dst_off;   // of the tile, from the start of its source / destination buffers
    uint32_t src_pitch, dst_pitch;
    uint32_t rows, width;        // row pieces in the tile, dst bytes per piece
    uint16_t src_buf, dst_buf;
    uint16_t replicas, replica_stride;
    uint16_t level, cast;
    uint32_t reserved;
};
static_assert(sizeof(TileRec) == 48, "TileRec must stay 48 bytes");

// Control words on the device, one block per device copy of a table.  A run leaves cursor, done and exited at
// zero for the next one (the last block to finish clears them), so a launch needs no reset in front of it and
// may be replayed from a captured graph.  status is sticky: the first failure since it was last read.
struct Ctrl {
    uint32_t cursor;      // tiles claimed dynamically so far
    uint32_t done;        // tiles completed (only maintained for multi-level tables)
    uint32_t exited;      // blocks of the running launch that have finished
    uint32_t status;      // NEREUS_DEV_*
    uint32_t detail;      // tile index that raised the status
    uint32_t reserved[3];
};
static_assert(sizeof(Ctrl) == 32, "Ctrl is one 32-byte sector");

// Optional per-block trace of one run (nereus_transition_trace): when the block started, when it finished, how
// many tiles it moved.  Same layout as nereus_block_trace_t.
struct BlockTrace {
    uint64_t begin_ns, end_ns;   // the GPU's global timer
    uint32_t tiles, block;
};
static_assert(sizeof(BlockTrace) == sizeof(nereus_block_trace_t), "BlockTrace is the public record");

constexpr int kMaxBuffers = 448;      // pointers carried in the kernel's parameter block
constexpr int kMaxLevels  = 8;
constexpr int kMaxReplicas = 16;
constexpr uint32_t kDirectMaxTiles = 1u << 17;   // tables up to this many tiles get per-tile records (6 MiB)

struct Tuning {
    int tile_bytes  = 0;
    int ctas_per_sm = 0;
    int threads     = 0;
    int variant     = 0;
};

struct DeviceTable {                  // one per prepare()
    int       device    = -1;
    RectDev*  rects     = nullptr;
    uint32_t* first     = nullptr;    // n_rects + 1 tile prefix
    TileRec*  tiles     = nullptr;    // n_tiles records, or null for tables beyond kDirectMaxTiles
    BlockTrace* trace   = nullptr;    // one record per block of the launch, or null when tracing is off
    uint32_t  trace_blocks = 0;
    Ctrl*     ctrl      = nullptr;    // the control block
    uint32_t  runs      = 0;          // runs launched on this device copy
    uint32_t  n_tiles   = 0;
    uint32_t  level_end[kMaxLevels] = {0};   // tiles up to and including each level
    int       sm_count  = 0;
    int       tile_bytes = 0, ctas_per_sm = 0, threads = 0, variant = 0;
};

}  // namespace nereus

struct nereus_transition_s {
    std::vector<nereus::Rect> rects;          // execution order
    std::vector<uint64_t>     src_bytes;      // required length of each source buffer
    std::vector<uint64_t>     dst_bytes;      // ... of each destination buffer
    std::vector<int>          src_read_level; // last level that reads source buffer i (empty: level 0)
    std::vector<int>          dst_level;      // level that writes destination buffer j
    std::vector<int>          dst_read_level; // level that reads destination j (chained), -1 if none
    int                       n_levels = 1;
    uint64_t                  bytes_read = 0, bytes_written = 0;
    nereus::Tuning            tuning;
    bool                      trace = false;  // nereus_transition_trace
    nereus::DeviceTable       dev;
    uint64_t                  launches = 0;
};

// ---------------------------------------------------------------------------------------------------
// Transition DAG over EMU primitives
// ---------------------------------------------------------------------------------------------------

#include <set>

namespace nereus {

struct UnitRec {
    int              stage, tp, pp;
    std::vector<int> gpus;
};

struct PrimRec {
    int              op, stage;
    std::vector<int> src, dst;
    std::set<int>    deps, rdeps;
    int              order = -1, level = 0;
};

struct StageRec {
    int                  kind;
    uint64_t             state_bytes;
    std::vector<UnitRec> current, target;
};

}  // namespace nereus

struct nereus_dag_s {
    std::vector<nereus::StageRec> stages;
    std::vector<nereus::UnitRec>  units;
    std::vector<nereus::PrimRec>  prims;
    bool                          planned = false;     // nereus_dag_plan has run: no more stages or units
    bool                          scheduled = false;   // ... and every primitive got its place in the schedule
};

namespace nereus {

// Cuts rects into tiles for a tile size; fills RectDev entries, the prefix and level ends.
// Returns the number of tiles, or 0 with *overflow = true when it exceeds 32 bits.
uint64_t tile_table(const nereus_transition_s& t, uint32_t tile_bytes, std::vector<RectDev>& out,
                    std::vector<uint32_t>& first, uint32_t level_end[kMaxLevels]);

// Same into caller-provided arrays (rects.size() entries and rects.size() + 1 entries): no allocation.
uint64_t tile_table_raw(const nereus_transition_s& t, uint32_t tile_bytes, RectDev* out, uint32_t* first,
                        uint32_t level_end[kMaxLevels]);

// One record per tile from a tiled table (out has room for the table's tile count).
void expand_tiles(const RectDev* rects, size_t n_rects, TileRec* out);

// Host-side check of a table before it reaches the device: every task inside its buffers, the 16-byte rule,
// pitches that keep row pieces apart, buffer indices and levels in range, a chained task reading only what an
// earlier level wrote, destinations of one level pairwise disjoint, and (when `tiled` is given) a tiling that
// covers each task exactly.  `order` is scratch for rects.size() indices.  Allocates nothing.
int validate_table(const nereus_transition_s& t, const RectDev* tiled, const uint32_t* first, uint64_t n_tiles,
                   uint32_t* order);

void set_cuda_error(int e);

}  // namespace nereus
