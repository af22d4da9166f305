// Device side of the EMU reshard for sm_100a: ONE kernel launch walks the task table of a compiled transition
// (the local layout change of Section 6.2 of the Nereus paper) and moves every rect-copy task's bytes from the
// source shards to the destination shards, with an optional fused fp32 -> bf16 round-to-nearest-even cast.
// Pure data movement: the bound is HBM bandwidth, there is no tensor-core work.  Three kernels share the table
// format and the tile bodies; the host picks one per table (resolve_launch).
//
// nereus_walk_vec, persistent, register-staged
//   * grid = SMs x ctas_per_sm persistent blocks; every WARP claims tiles on its own.  Its first tile is its
//     own index in the grid (no atomic on the way to the first load); further tiles come from a global cursor:
//     lane 0 takes the next index with one atomicAdd and broadcasts it by shuffle, and the claim of the next
//     tile is issued before the current tile is copied, so its latency hides behind the copy.  Chained tables
//     claim every tile from the cursor: tiles are then handed out in level order to warps that already run,
//     which is what keeps the level gates free of deadlock whatever else shares the GPU.
//   * a tile index is resolved by one load of its 48-byte record when the table carries per-tile records
//     (tables of up to 2^17 tiles), else to its rect by binary search in the tile-prefix array and then to a
//     row block / column block of that rect by arithmetic; every lane moves 16-byte vectors, 32 lanes x 16 B =
//     512 B contiguous per instruction, kUnroll independent loads in flight per lane before the first store.
//   * tables with several dependency levels (chained transitions): a tile of level k waits, with a poll
//     limit, until every tile of level k-1 has completed; on giving up it records NEREUS_DEV_TIMEOUT and the
//     warp leaves.  A warp publishes its completed tiles once per level (one fence, one atomic), not per
//     tile.  Loads bypass L1 (ld.global.cg) so a level reads what another SM wrote before it.
// nereus_walk_ring, persistent, for large tables: one CTA per SM, a producer warp that claims tiles and issues
//     cp.async.bulk global -> shared copies into a ring of stages, and a consumer warp that issues
//     cp.async.bulk shared -> global stores (tables with a cast: fifteen consumer warps that convert from
//     shared memory and store with plain 16-byte stores); mbarriers track both directions and every wait has
//     a deadline on the global timer and an iteration limit.
// nereus_walk_once, not persistent, for small and medium single-level tables: one warp per tile, the tile's
//     addresses from its record, no cursor, no shared memory.
// In both persistent kernels the last block to finish zeroes the cursor and the counters, so a launch needs no
// reset in front of it and can be replayed from a captured graph.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "nereus_internal.hpp"

using namespace nereus;

namespace nereus {

static thread_local int g_last_cuda_error = 0;
void set_cuda_error(int e) { g_last_cuda_error = e; }

#define NEREUS_CUDA(call)                                               \
    do {                                                                \
        cudaError_t e_ = (call);                                        \
        if (e_ != cudaSuccess) { set_cuda_error((int)e_); (void)cudaGetLastError(); return NEREUS_ERR_CUDA; } \
    } while (0)

struct WalkParams {
    const RectDev*  rects;
    const uint32_t* first;        // n_rects + 1
    const TileRec*  tiles;        // n_tiles records, or null
    Ctrl*           ctrl;
    BlockTrace*     trace;        // one record per block, or null
    uint32_t        n_rects, n_tiles, n_levels;
    uint32_t        level_end[kMaxLevels];
    char*           bufs[kMaxBuffers];
};
static_assert(sizeof(WalkParams) <= 4000, "kernel parameter block too large");

constexpr int      kUnrollRun   = 8;            // 16-byte loads in flight per lane, contiguous runs
constexpr int      kUnrollRect  = 6;            // ... pitched rects (their index math needs registers)
constexpr int      kUnrollCast  = 8;            // ... the cast
constexpr uint32_t kPrefixCache = 2047;         // rects whose tile prefix the vector kernel keeps in shared memory
constexpr uint32_t kGatePolls   = 1u << 21;     // x ~200 ns sleep: gives up after roughly half a second
constexpr uint64_t kWaitNanos   = 500ull * 1000 * 1000;   // deadline of an mbarrier wait, on %globaltimer

// ---------------------------------------------------------------------------------------------------
// device helpers
// ---------------------------------------------------------------------------------------------------

__device__ __forceinline__ uint32_t claim_tiles(Ctrl* ctrl, unsigned lane, uint32_t n) {
    uint32_t g = 0;
    if (lane == 0) g = atomicAdd(&ctrl->cursor, n);
    return __shfl_sync(0xffffffffu, g, 0);
}

// A claim in two halves, so that the atomic's round trip hides behind the work in between: issue it on
// lane 0, broadcast the answer only when it is needed.
__device__ __forceinline__ uint32_t claim_issue(Ctrl* ctrl, unsigned lane, uint32_t n) {
    return lane == 0 ? atomicAdd(&ctrl->cursor, n) : 0u;
}
__device__ __forceinline__ uint32_t claim_take(uint32_t issued) { return __shfl_sync(0xffffffffu, issued, 0); }

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ uint4 ld_stream(const char* p) { return __ldcg(reinterpret_cast<const uint4*>(p)); }
__device__ __forceinline__ void  st_stream(char* p, uint4 v) { __stcs(reinterpret_cast<uint4*>(p), v); }
__device__ __forceinline__ void  st_stream8(char* p, uint2 v) { __stcs(reinterpret_cast<uint2*>(p), v); }

// two fp32 -> packed bf16x2, round to nearest even (the instruction's own rounding: ties to even, overflow to
// +-Inf, subnormals rounded, signed zero kept).  For a NaN the instruction leaves the pattern 0x7FFF in that half,
// which no other input produces (finite values end at 0x7F80 = Inf); the rule of this library is 0x7FC0 for
// every NaN, so such halves are rewritten.  The test is on the packed result: (half & 0x7FFF) + 1 reaches
// 0x8000 exactly for 0x7FFF / 0xFFFF, and the carry cannot leave its half.
__device__ __forceinline__ uint32_t cvt_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ uint32_t nan_halves(uint32_t r) { return ((r & 0x7FFF7FFFu) + 0x00010001u) & 0x80008000u; }
__device__ __forceinline__ uint32_t fix_nan_halves(uint32_t r) {
    const uint32_t n = nan_halves(r);
    if (n & 0x00008000u) r = (r & 0xFFFF0000u) | 0x00007FC0u;
    if (n & 0x80000000u) r = (r & 0x0000FFFFu) | 0x7FC00000u;
    return r;
}
// The same rule without a branch, for the register-staged kernels (a data-dependent branch between their loads
// and stores costs them up to 5%; the ring's converting warps, which are bound by instruction issue, gain 2%
// from testing eight results at once instead).
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r = cvt_bf16x2(lo, hi);
    if (lo != lo) r = (r & 0xFFFF0000u) | 0x00007FC0u;
    if (hi != hi) r = (r & 0x0000FFFFu) | 0x7FC00000u;
    return r;
}

// The three tile bodies below load a batch of vectors once and store it to every destination replica
// (`reps` is 1 except for replicated transitions); D(j) yields replica j's base pointer for the tile.
// Each body runs full batches without predicates; what is left goes one vector at a time (the persistent
// kernel: its tiles are large, tails are rare, registers are scarce) or, with kBatchTail, as ONE predicated
// batch, so that a small tile's last (or only) loads are in flight together instead of one round trip each.

// Bit copy of a contiguous run of `nvec` 16-byte vectors.
template <int kUnroll, bool kBatchTail, class Dst>
__device__ __forceinline__ void copy_run(const char* __restrict__ s, Dst D, uint32_t reps, uint32_t nvec,
                                         unsigned lane) {
    s += lane * 16;
    uint32_t off = lane * 16;
    uint32_t left = nvec;
#pragma unroll 1
    for (; left >= 32 * kUnroll; left -= 32 * kUnroll) {          // full batches: no predicates
        uint4 v[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) v[u] = ld_stream(s + u * 512);
#pragma unroll 1
        for (uint32_t j = 0; j < reps; ++j) {
            char* d = D(j) + off;
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) st_stream(d + u * 512, v[u]);
        }
        s += 512 * kUnroll;
        off += 512 * kUnroll;
    }
    if (!kBatchTail) {
#pragma unroll 1
        for (uint32_t i = lane; i < left; i += 32) {              // ragged tail, one vector at a time
            const uint4 v = ld_stream(s);
#pragma unroll 1
            for (uint32_t j = 0; j < reps; ++j) st_stream(D(j) + off, v);
            s += 512;
            off += 512;
        }
    } else if (left) {                                            // ragged tail: one predicated batch
        uint4 v[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u)
            if (lane + 32 * u < left) v[u] = ld_stream(s + u * 512);
#pragma unroll 1
        for (uint32_t j = 0; j < reps; ++j) {
            char* d = D(j) + off;
#pragma unroll
            for (int u = 0; u < kUnroll; ++u)
                if (lane + 32 * u < left) st_stream(d + u * 512, v[u]);
        }
    }
}

// Bit copy of a pitched tile: `rows` pieces of `vpr` 16-byte vectors each.  Offsets inside a tile fit
// 32 bits (rows_per_tile x pitch is far below 4 GiB).
template <int kUnroll, bool kBatchTail, class Dst>
__device__ __forceinline__ void copy_rect(const char* __restrict__ s, Dst D, uint32_t reps, uint32_t rows,
                                          uint32_t vpr, uint32_t sp, uint32_t dp, unsigned lane) {
    const uint32_t nvec = rows * vpr;
    uint32_t       base = lane;
#pragma unroll 1
    for (; base + 32 * (kUnroll - 1) < nvec; base += 32 * kUnroll) {   // every lane has kUnroll vectors
        uint4    v[kUnroll];
        uint32_t doff[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const uint32_t idx = base + u * 32;
            const uint32_t r = idx / vpr, c = idx - r * vpr;
            doff[u] = r * dp + c * 16;
            v[u] = ld_stream(s + (r * sp + c * 16));
        }
#pragma unroll 1
        for (uint32_t j = 0; j < reps; ++j) {
            char* d = D(j);
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) st_stream(d + doff[u], v[u]);
        }
    }
    if (!kBatchTail) {
#pragma unroll 1
        for (; base < nvec; base += 32) {                              // ragged tail, one vector at a time
            const uint32_t r = base / vpr, c = base - r * vpr;
            const uint4 v = ld_stream(s + (r * sp + c * 16));
#pragma unroll 1
            for (uint32_t j = 0; j < reps; ++j) st_stream(D(j) + (r * dp + c * 16), v);
        }
    } else if (base < nvec) {                                          // ragged tail: one predicated batch
        uint4    v[kUnroll];
        uint32_t doff[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const uint32_t idx = base + u * 32;
            if (idx < nvec) {
                const uint32_t r = idx / vpr, c = idx - r * vpr;
                doff[u] = r * dp + c * 16;
                v[u] = ld_stream(s + (r * sp + c * 16));
            }
        }
#pragma unroll 1
        for (uint32_t j = 0; j < reps; ++j) {
            char* d = D(j);
#pragma unroll
            for (int u = 0; u < kUnroll; ++u)
                if (base + u * 32 < nvec) st_stream(d + doff[u], v[u]);
        }
    }
}

// Cast tile: the unit is 4 elements, 16 bytes of fp32 in and 8 bytes of bf16 out, so that both the loads
// and the stores of a warp instruction stay contiguous.  `upr` = units per row piece.
__device__ __forceinline__ uint2 cast_unit(uint4 v) {
    uint2 o;
    o.x = pack_bf16x2(__uint_as_float(v.x), __uint_as_float(v.y));
    o.y = pack_bf16x2(__uint_as_float(v.z), __uint_as_float(v.w));
    return o;
}

template <int kUnroll, bool kBatchTail, class Dst>
__device__ __forceinline__ void cast_tile(const char* __restrict__ s, Dst D, uint32_t reps, uint32_t rows,
                                          uint32_t upr, uint32_t sp, uint32_t dp, unsigned lane) {
    const uint32_t nunit = rows * upr;
    uint32_t       base = lane;
#pragma unroll 1
    for (; base + 32 * (kUnroll - 1) < nunit; base += 32 * kUnroll) {
        uint2    o[kUnroll];
        uint32_t doff[kUnroll];
        {
            uint4 v[kUnroll];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const uint32_t idx = base + u * 32;
                const uint32_t r = idx / upr, c = idx - r * upr;
                doff[u] = r * dp + c * 8;
                v[u] = ld_stream(s + (r * sp + c * 16));
            }
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) o[u] = cast_unit(v[u]);
        }
#pragma unroll 1
        for (uint32_t j = 0; j < reps; ++j) {
            char* d = D(j);
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) st_stream8(d + doff[u], o[u]);
        }
    }
    if (!kBatchTail) {
#pragma unroll 1
        for (; base < nunit; base += 32) {                             // ragged tail, one unit at a time
            const uint32_t r = base / upr, c = base - r * upr;
            const uint2 o = cast_unit(ld_stream(s + (r * sp + c * 16)));
#pragma unroll 1
            for (uint32_t j = 0; j < reps; ++j) st_stream8(D(j) + (r * dp + c * 8), o);
        }
    } else if (base < nunit) {                                         // ragged tail: one predicated batch
        uint2    o[kUnroll];
        uint32_t doff[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const uint32_t idx = base + u * 32;
            if (idx < nunit) {
                const uint32_t r = idx / upr, c = idx - r * upr;
                doff[u] = r * dp + c * 8;
                o[u] = cast_unit(ld_stream(s + (r * sp + c * 16)));
            }
        }
#pragma unroll 1
        for (uint32_t j = 0; j < reps; ++j) {
            char* d = D(j);
#pragma unroll
            for (int u = 0; u < kUnroll; ++u)
                if (base + u * 32 < nunit) st_stream8(d + doff[u], o[u]);
        }
    }
}

// ---------------------------------------------------------------------------------------------------
// tile index -> addresses
// ---------------------------------------------------------------------------------------------------

struct Tile {
    const char* s;
    uint64_t    d_off;             // byte offset of the tile inside each destination buffer
    uint32_t    dst_buf, reps, rstride;   // destinations: bufs[dst_buf + j * rstride], j < reps
    uint32_t    nr, w, sp, dp;     // row pieces, dst bytes per piece, pitches
    uint32_t    level, cast;
};

// Destination j of a tile.  The pointer table lives in the kernel's parameter block (constant bank).
__device__ __forceinline__ char* tile_dst(const WalkParams& p, uint32_t dst_buf, uint32_t rstride, uint64_t d_off,
                                          uint32_t j) {
    return p.bufs[dst_buf + j * rstride] + d_off;
}

// The rect a claimer resolved last: consecutive claims of one warp usually fall into the same rect (a rect
// has thousands of tiles), so the binary search is skipped while first <= g < next_first.
struct RectRange {
    uint32_t first = 1, next_first = 0;                        // empty range
    uint4    q0, q1, q2, q3;                                   // the rect's 64-byte record
};

// Resolves tile g: binary search for the rect (largest i with first[i] <= g), then row block x column block.
// Returns false when the table does not resolve (corrupted).
// `first_at(i)` reads entry i of the tile-prefix array (from global memory, or from a shared-memory copy).
template <bool kUseRange, class FirstAt>
__device__ __forceinline__ bool resolve_tile(const WalkParams& p, uint32_t g, RectRange& rr, Tile& t,
                                             FirstAt first_at) {
    uint4 q0, q1, q2, q3;
    if (!kUseRange || g < rr.first || g >= rr.next_first) {
        uint32_t lo = 0, hi = p.n_rects;                       // invariant: first[lo] <= g < first[hi]
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) >> 1;
            if (first_at(mid) <= g) lo = mid; else hi = mid;
        }
        const RectDev* rp = p.rects + lo;
        q0 = __ldg(reinterpret_cast<const uint4*>(rp));        // src_off, dst_off
        q1 = __ldg(reinterpret_cast<const uint4*>(rp) + 1);    // width, src_pitch, dst_pitch
        q2 = __ldg(reinterpret_cast<const uint4*>(rp) + 2);    // rows, rows_per_tile, tile_w, col_tiles
        q3 = __ldg(reinterpret_cast<const uint4*>(rp) + 3);    // first_tile, bufs, level|cast, replicas|stride
        if (kUseRange) {
            rr.first = first_at(lo);
            rr.next_first = first_at(lo + 1);
            rr.q0 = q0; rr.q1 = q1; rr.q2 = q2; rr.q3 = q3;
        }
    } else {
        q0 = rr.q0; q1 = rr.q1; q2 = rr.q2; q3 = rr.q3;
    }
    const uint64_t src_off = ((uint64_t)q0.y << 32) | q0.x, dst_off = ((uint64_t)q0.w << 32) | q0.z;
    const uint64_t width   = ((uint64_t)q1.y << 32) | q1.x;
    const uint32_t rows = q2.x, rpt = q2.y, tile_w = q2.z, col_tiles = q2.w;
    const uint32_t first_tile = q3.x;
    const uint32_t src_buf = q3.y & 0xFFFFu, dst_buf = q3.y >> 16;
    t.sp = q1.z; t.dp = q1.w;
    t.level = q3.z & 0xFFFFu; t.cast = q3.z >> 16;
    t.reps = q3.w & 0xFFFFu; t.rstride = q3.w >> 16;
    t.dst_buf = dst_buf;
    if (first_tile > g || src_buf >= (uint32_t)kMaxBuffers || col_tiles == 0 || t.reps == 0 ||
        dst_buf + (t.reps - 1) * t.rstride >= (uint32_t)kMaxBuffers)
        return false;
    const uint32_t k  = g - first_tile;
    const uint32_t rb = k / col_tiles, cb = k - rb * col_tiles;
    const uint32_t r0 = rb * rpt;
    if (r0 >= rows) return false;
    const uint64_t c0 = (uint64_t)cb * tile_w;                 // dst bytes into the row piece
    t.nr = min(rpt, rows - r0);
    t.w  = (uint32_t)min((uint64_t)tile_w, width - c0);
    t.s  = p.bufs[src_buf] + src_off + (uint64_t)r0 * t.sp + (c0 << t.cast);
    t.d_off = dst_off + (uint64_t)r0 * t.dp + c0;
    return true;
}

// Tile g of a table that carries per-tile records: one 48-byte load, no search.
__device__ __forceinline__ bool resolve_direct(const WalkParams& p, uint32_t g, Tile& t) {
    const uint4* q = reinterpret_cast<const uint4*>(p.tiles + g);
    const uint4 a = __ldg(q), b = __ldg(q + 1), c = __ldg(q + 2);
    const uint64_t src_off = ((uint64_t)a.y << 32) | a.x;
    t.d_off = ((uint64_t)a.w << 32) | a.z;
    t.sp = b.x; t.dp = b.y; t.nr = b.z; t.w = b.w;
    const uint32_t src_buf = c.x & 0xFFFFu;
    t.dst_buf = c.x >> 16;
    t.reps = c.y & 0xFFFFu; t.rstride = c.y >> 16;
    t.level = c.z & 0xFFFFu; t.cast = c.z >> 16;
    if (src_buf >= (uint32_t)kMaxBuffers || t.reps == 0 || t.nr == 0 ||
        t.dst_buf + (t.reps - 1) * t.rstride >= (uint32_t)kMaxBuffers)
        return false;
    t.s = p.bufs[src_buf] + src_off;
    return true;
}

__device__ __forceinline__ uint64_t global_nanos() {
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// Tracing (off unless nereus_transition_trace switched it on): a block's first thread notes when the block
// starts and ends, every warp adds the tiles it moved.
__device__ __forceinline__ void trace_begin(BlockTrace* trace) {
    if (trace && threadIdx.x == 0) { trace[blockIdx.x].begin_ns = global_nanos(); trace[blockIdx.x].block = blockIdx.x; }
}
__device__ __forceinline__ void trace_tiles(BlockTrace* trace, uint32_t n, unsigned lane) {
    if (trace && lane == 0 && n) atomicAdd(&trace[blockIdx.x].tiles, n);
}
__device__ __forceinline__ void trace_end(BlockTrace* trace) {           // after the block's closing barrier
    if (trace && threadIdx.x == 0) trace[blockIdx.x].end_ns = global_nanos();
}

__device__ __forceinline__ void raise_status(Ctrl* ctrl, uint32_t status, uint32_t detail) {
    if (atomicCAS(&ctrl->status, (uint32_t)NEREUS_DEV_OK, status) == (uint32_t)NEREUS_DEV_OK) ctrl->detail = detail;
}

// End of a block's work: the last block of the launch to get here leaves the control words as a fresh launch
// expects them.  Every claim and every publication of the block happened before its arrival (the barrier
// orders the block's threads, the fence orders the block against the others), so nothing touches the words
// after they are cleared.  The status word is not cleared: it is the host's to read.
__device__ __forceinline__ void finish_block(Ctrl* ctrl) {
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(&ctrl->exited, 1u) == gridDim.x - 1) {
            __threadfence();
            ctrl->cursor = 0;
            ctrl->done = 0;
            ctrl->exited = 0;
        }
    }
}

// ---------------------------------------------------------------------------------------------------
// the persistent walker, register-staged vector copy
// ---------------------------------------------------------------------------------------------------

__global__ void __launch_bounds__(512, 2) nereus_walk_vec(const __grid_constant__ WalkParams p) {
    const unsigned lane = threadIdx.x & 31;
    Ctrl* const    ctrl = p.ctrl;
    uint32_t       my_done = 0, my_level = 0;                  // tiles completed and not yet published
    uint32_t       open_level = 0;                             // highest level whose gate this warp has passed
    uint32_t       moved = 0;                                  // tiles this warp moved (for the trace)
    RectRange      rr;
    trace_begin(p.trace);

    // tables without per-tile records: the tile prefix is copied to shared memory once per CTA (when it fits),
    // so that resolving a tile costs one trip to memory (the rect record) instead of a chain of dependent ones
    __shared__ uint32_t s_first[kPrefixCache + 1];
    const bool direct = p.tiles != nullptr;
    const bool cached = !direct && p.n_rects <= kPrefixCache;
    if (cached) {
        for (uint32_t i = threadIdx.x; i <= p.n_rects; i += blockDim.x) s_first[i] = __ldg(p.first + i);
        __syncthreads();
    }
    const uint32_t* const sf = s_first;
    auto first_at = [&p, cached, sf](uint32_t i) { return cached ? sf[i] : __ldg(p.first + i); };

    // single-level tables: the first tile of a warp is its own index, the cursor hands out the tiles beyond
    // the grid; chained tables take every tile from the cursor (see the head of this file)
    const uint32_t n_warps = gridDim.x * (blockDim.x >> 5);
    const uint32_t base    = p.n_levels == 1 ? n_warps : 0u;
    const bool     more    = p.n_tiles > base;                 // false: nobody ever touches the cursor
    uint32_t g = p.n_levels == 1 ? blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)
                                 : claim_tiles(ctrl, lane, 1);
    while (g < p.n_tiles) {
        const uint32_t next_issued = more ? claim_issue(ctrl, lane, 1) : 0u;   // in flight while this tile is copied
        Tile t;
        if (!(direct ? resolve_direct(p, g, t) : resolve_tile<false>(p, g, rr, t, first_at))) {
            if (lane == 0) raise_status(ctrl, NEREUS_DEV_BOUNDS, g);
            break;
        }

        if (t.level != my_level) {
            // leaving a level: make this warp's stores visible, publish its tiles, then wait for the level
            // below this tile's to be complete everywhere
            if (my_done) {
                __threadfence();
                __syncwarp();
                if (lane == 0) atomicAdd(&ctrl->done, my_done);
                my_done = 0;
            }
            my_level = t.level;
        }
        if (t.level > open_level) {
            const uint32_t need = p.level_end[t.level - 1];
            bool ok = true;
            if (lane == 0) {
                uint32_t polls = 0;
                while (ld_acquire_u32(&ctrl->done) < need) {
                    if (++polls > kGatePolls) { ok = false; break; }
                    __nanosleep(200);
                }
                if (!ok) raise_status(ctrl, NEREUS_DEV_TIMEOUT, g);
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            __threadfence();
            open_level = t.level;
        }

        const uint32_t dst_buf = t.dst_buf, rstride = t.rstride;
        const uint64_t d_off = t.d_off;
        auto D = [&p, dst_buf, rstride, d_off](uint32_t j) { return tile_dst(p, dst_buf, rstride, d_off, j); };
        if (t.cast) {
            cast_tile<kUnrollCast, false>(t.s, D, t.reps, t.nr, t.w >> 3, t.sp, t.dp, lane);
        } else if (t.nr == 1) {
            copy_run<kUnrollRun, false>(t.s, D, t.reps, t.w >> 4, lane);
        } else {
            copy_rect<kUnrollRect, false>(t.s, D, t.reps, t.nr, t.w >> 4, t.sp, t.dp, lane);
        }
        if (p.n_levels > 1) ++my_done;
        ++moved;
        g = more ? base + claim_take(next_issued) : p.n_tiles;
    }
    if (my_done) {
        __threadfence();
        __syncwarp();
        if (lane == 0) atomicAdd(&ctrl->done, my_done);
    }
    trace_tiles(p.trace, moved, lane);
    finish_block(ctrl);
    trace_end(p.trace);
}

// ---------------------------------------------------------------------------------------------------
// small tables: one warp per tile, no loop
// ---------------------------------------------------------------------------------------------------
//
// A table of a few thousand tiles is over before a persistent grid has warmed up: what counts is the chain of
// dependent memory trips in front of the first load and the number of bytes in flight.  Here a warp's tile is
// its index in the grid and its addresses come with one 48-byte record; there is no cursor, no claim, no
// shared memory and nothing to reset; the hardware's block scheduler does the balancing.  Single-level tables
// with per-tile records and at most kOnceMaxBuffers buffers only (the parameter block stays small).

constexpr int kOnceMaxBuffers = 64;

struct OnceParams {
    const TileRec* tiles;
    Ctrl*          ctrl;
    BlockTrace*    trace;         // one record per block, or null
    uint32_t       n_tiles;
    char*          bufs[kOnceMaxBuffers];
};

__global__ void __launch_bounds__(512, 2) nereus_walk_once(const __grid_constant__ OnceParams p) {
    const unsigned lane = threadIdx.x & 31;
    const uint32_t g = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (g >= p.n_tiles) return;
    if (p.trace && lane == 0) {                      // no barrier in this kernel: first warp in, last warp out
        BlockTrace* tr = p.trace + blockIdx.x;
        if (atomicCAS(reinterpret_cast<unsigned long long*>(&tr->begin_ns), 0ull, (unsigned long long)global_nanos()) == 0ull)
            tr->block = blockIdx.x;
    }
    const uint4* q = reinterpret_cast<const uint4*>(p.tiles + g);
    const uint4 a = __ldg(q), b = __ldg(q + 1), c = __ldg(q + 2);
    const uint32_t src_buf = c.x & 0xFFFFu, dst_buf = c.x >> 16;
    const uint32_t reps = c.y & 0xFFFFu, rstride = c.y >> 16, cast = c.z >> 16;
    if (src_buf >= (uint32_t)kOnceMaxBuffers || reps == 0 || b.z == 0 ||
        dst_buf + (reps - 1) * rstride >= (uint32_t)kOnceMaxBuffers) {
        if (lane == 0) raise_status(p.ctrl, NEREUS_DEV_BOUNDS, g);
        return;
    }
    const char*    s     = p.bufs[src_buf] + (((uint64_t)a.y << 32) | a.x);
    const uint64_t d_off = ((uint64_t)a.w << 32) | a.z;
    auto D = [&p, dst_buf, rstride, d_off](uint32_t j) { return p.bufs[dst_buf + j * rstride] + d_off; };
    if (cast)          cast_tile<kUnrollCast, true>(s, D, reps, b.z, b.w >> 3, b.x, b.y, lane);
    else if (b.z == 1) copy_run<kUnrollRun, true>(s, D, reps, b.w >> 4, lane);
    else               copy_rect<kUnrollRect, true>(s, D, reps, b.z, b.w >> 4, b.x, b.y, lane);
    if (p.trace) {
        __syncwarp();
        if (lane == 0) {
            atomicAdd(&p.trace[blockIdx.x].tiles, 1u);
            atomicMax(reinterpret_cast<unsigned long long*>(&p.trace[blockIdx.x].end_ns), (unsigned long long)global_nanos());
        }
    }
}

// ---------------------------------------------------------------------------------------------------
// the persistent walker, bulk-copy ring (bit-copy tables)
// ---------------------------------------------------------------------------------------------------
//
// Shared memory: n_stages x stage_bytes of data, then per stage one "full" mbarrier (1 arrival + the
// bytes the bulk loads deliver), one "empty" mbarrier (one arrival per consumer warp) and the tile's
// destination record.  Data never passes through registers.

struct StageMeta {
    uint64_t d_off;
    uint32_t nr, w, dp;
    uint32_t kind;          // kStageData, kStageEnd or kStageFlush
    uint16_t dst_buf, reps, rstride, cast;
    uint32_t magic;         // converting ring: ceil(2^32 / (w / 16)), so that a row index is one multiply
    uint32_t reserved;
};
constexpr uint32_t kStageData = 0, kStageEnd = 1, kStageFlush = 2;

constexpr uint32_t kBulkMaxStages = 28;
constexpr uint32_t kCastConsumers = 480;        // cast ring: threads that convert a stage (15 warps)
constexpr uint32_t kBarrierTries  = 1u << 22;   // try_wait attempts before a wait gives up

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait for the phase with the given parity; false when it gave up.  Two limits: a deadline of
// kWaitNanos (half a second) on the global timer, read every 64 attempts once the first few have failed, and
// a cap on the attempts as a backstop should the timer not advance (a try_wait suspends the thread for a time
// the hardware chooses, so the cap alone has no number).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    uint64_t deadline = 0;
    for (uint32_t i = 0; i < kBarrierTries; ++i) {
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
        if ((i & 63u) == 63u) {
            const uint64_t now = global_nanos();
            if (deadline == 0) deadline = now + kWaitNanos;
            else if (now > deadline) return false;
        }
    }
    return false;
}
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const char* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_store(char* dst, uint32_t src_smem, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(dst), "r"(src_smem), "r"(bytes) : "memory");
}

struct Ring {
    unsigned char* data;
    uint64_t*      full;
    uint64_t*      empty;
    StageMeta*     meta;
    uint32_t       stage_bytes, n_stages;
    uint32_t       piece;          // contiguous tiles are issued as bulk copies of this many bytes
    uint32_t       lag;            // stages whose stores may still be reading shared memory
    uint32_t       claim;          // consecutive tiles the producer takes per atomic
};

// cp.async.bulk.wait_group.read takes an immediate
__device__ __forceinline__ void wait_store_reads(uint32_t pending) {
    switch (pending) {
    case 1:  asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); break;
    case 2:  asm volatile("cp.async.bulk.wait_group.read 2;" ::: "memory"); break;
    case 3:  asm volatile("cp.async.bulk.wait_group.read 3;" ::: "memory"); break;
    case 4:  asm volatile("cp.async.bulk.wait_group.read 4;" ::: "memory"); break;
    case 5:  asm volatile("cp.async.bulk.wait_group.read 5;" ::: "memory"); break;
    case 6:  asm volatile("cp.async.bulk.wait_group.read 6;" ::: "memory"); break;
    case 7:  asm volatile("cp.async.bulk.wait_group.read 7;" ::: "memory"); break;
    case 8:  asm volatile("cp.async.bulk.wait_group.read 8;" ::: "memory"); break;
    default: asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); break;
    }
}

// Producer warp: claims R.claim consecutive tiles at a time, resolves them and loads them into the ring.
// kCast: the stage receives the fp32 source bytes (twice the destination bytes).
template <bool kCast>
__device__ __forceinline__ void ring_producer(const WalkParams& p, const Ring& R, unsigned lane) {
    Ctrl* const ctrl = p.ctrl;
    uint32_t    stage = 0, phase = 0, level = 0, moved = 0;
    RectRange   rr;
    // single-level tables: the first batch is the block's own index, the cursor hands out the batches beyond
    // the grid; chained tables take every batch from the cursor
    const uint32_t base = p.n_levels == 1 ? gridDim.x * R.claim : 0u;
    uint32_t    g0 = p.n_levels == 1 ? blockIdx.x * R.claim : claim_tiles(ctrl, lane, R.claim);
    bool        running = true;
    while (running) {
        const bool     last    = g0 >= p.n_tiles;
        const uint32_t next_issued = last ? g0 : claim_issue(ctrl, lane, R.claim);   // hidden behind this batch
        for (uint32_t g = g0; running && g < g0 + R.claim; ++g) {
            const bool end = g >= p.n_tiles;
            Tile t;
            bool ok = true;
            if (!end) {
                // the converting ring (kCast) takes both kinds of tile, the bit-copy ring only its own
                ok = (p.tiles ? resolve_direct(p, g, t)
                              : resolve_tile<true>(p, g, rr, t, [&p](uint32_t i) { return __ldg(p.first + i); })) &&
                     (kCast || t.cast == 0) &&
                     (((uint64_t)t.nr * t.w) << t.cast) <= R.stage_bytes;
                if (!ok && lane == 0) raise_status(ctrl, NEREUS_DEV_BOUNDS, g);
            }
            // a tile of a higher level: first have the consumer publish this CTA's finished tiles (a flush
            // stage), only then wait for the level below to be complete everywhere
            const bool climb = !end && ok && t.level > level;
            for (int pass = climb ? 0 : 1; running && pass < 2; ++pass) {
                // the stage is free once the consumer has finished reading its previous contents
                bool freed = true;
                if (lane == 0) freed = mbar_wait(smem_addr(R.empty + stage), phase ^ 1);
                freed = __shfl_sync(0xffffffffu, freed, 0);
                if (!freed) {
                    if (lane == 0) raise_status(ctrl, NEREUS_DEV_TIMEOUT, g);
                    running = false;
                    break;
                }
                const uint32_t base = smem_addr(R.data + (size_t)stage * R.stage_bytes);
                const uint32_t bar  = smem_addr(R.full + stage);
                if (pass == 0) {
                    if (lane == 0) {
                        R.meta[stage].kind = kStageFlush;
                        mbar_arrive(bar);
                    }
                    if (++stage == R.n_stages) { stage = 0; phase ^= 1; }
                    // dependency gate, bounded
                    bool open = true;
                    if (lane == 0) {
                        // a cast table counts warp-tiles: every tile is published by each of its consumer warps
                        const uint32_t need = p.level_end[t.level - 1] * (kCast ? kCastConsumers / 32 : 1u);
                        uint32_t polls = 0;
                        while (ld_acquire_u32(&ctrl->done) < need) {
                            if (++polls > kGatePolls) { open = false; break; }
                            __nanosleep(200);
                        }
                        if (!open) raise_status(ctrl, NEREUS_DEV_TIMEOUT, g);
                    }
                    open = __shfl_sync(0xffffffffu, open, 0);
                    if (!open) { ok = false; }
                    // what other SMs wrote and published is read below through the async proxy
                    asm volatile("fence.proxy.async.global;" ::: "memory");
                    level = t.level;
                    continue;
                }
                if (end || !ok) {
                    if (lane == 0) {
                        R.meta[stage].kind = kStageEnd;
                        mbar_arrive(bar);
                    }
                    running = false;
                    break;
                }
                const uint32_t ws = t.w << t.cast;                          // source bytes per row piece
                if (lane == 0) {
                    StageMeta& m = R.meta[stage];
                    m.d_off = t.d_off; m.nr = t.nr; m.w = t.w; m.dp = t.dp;
                    m.dst_buf = (uint16_t)t.dst_buf; m.reps = (uint16_t)t.reps; m.rstride = (uint16_t)t.rstride;
                    m.cast = (uint16_t)t.cast;
                    // 16-byte units per row piece; a stage holds fewer than 2^16 of them, so umulhi(idx, magic)
                    // is idx / units exactly (units = 1: the quotient is idx itself, flagged by magic = 0)
                    m.magic = (kCast && t.nr > 1 && (t.w >> 4) > 1) ? 0xFFFFFFFFu / (t.w >> 4) + 1u : 0u;
                    m.kind = kStageData;
                    mbar_arrive_expect_tx(bar, t.nr * ws);
                }
                __syncwarp();
                if (t.nr == 1) {
                    for (uint32_t off = lane * R.piece; off < ws; off += 32 * R.piece)
                        bulk_load(base + off, t.s + off, min(R.piece, ws - off), bar);
                } else {
                    for (uint32_t r = lane; r < t.nr; r += 32)
                        bulk_load(base + r * ws, t.s + (size_t)r * t.sp, ws, bar);
                }
                ++moved;
                if (++stage == R.n_stages) { stage = 0; phase ^= 1; }
            }
        }
        g0 = last ? g0 : base + claim_take(next_issued);
    }
    trace_tiles(p.trace, moved, lane);
}

// Consumer warp of the bit-copy ring: stores full stages with bulk copies, hands them back `lag` stages later.
__device__ __forceinline__ void ring_consumer_copy(const WalkParams& p, const Ring& R, unsigned lane) {
    Ctrl* const ctrl = p.ctrl;
    uint32_t    stage = 0, phase = 0, issued = 0, unpublished = 0;
    while (true) {
        bool ready = true;
        if (lane == 0) ready = mbar_wait(smem_addr(R.full + stage), phase);
        ready = __shfl_sync(0xffffffffu, ready, 0);
        if (!ready) {
            if (lane == 0) raise_status(ctrl, NEREUS_DEV_TIMEOUT, 0xFFFFFFFFu);
            break;
        }
        const StageMeta m = R.meta[stage];
        if (m.kind == kStageEnd) break;
        if (m.kind == kStageFlush) {
            // this CTA leaves a level: all its stores must have landed and be visible device-wide before
            // the tiles are counted as done
            asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
            asm volatile("fence.proxy.async.global;" ::: "memory");
            __threadfence();
            __syncwarp();
            if (lane == 0 && unpublished) atomicAdd(&ctrl->done, unpublished);
            unpublished = 0;
        } else {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            const uint32_t base = smem_addr(R.data + (size_t)stage * R.stage_bytes);
            for (uint32_t j = 0; j < m.reps; ++j) {              // one load, `reps` stores
                char* d = tile_dst(p, m.dst_buf, m.rstride, m.d_off, j);
                if (m.nr == 1) {
                    for (uint32_t off = lane * R.piece; off < m.w; off += 32 * R.piece)
                        bulk_store(d + off, base + off, min(R.piece, m.w - off));
                } else {
                    for (uint32_t r = lane; r < m.nr; r += 32)
                        bulk_store(d + (size_t)r * m.dp, base + r * m.w, m.w);
                }
            }
            ++unpublished;
        }
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");        // a flush commits an empty group
        ++issued;
        if (issued > R.lag) {
            // all but the `lag` newest groups of this lane have finished reading shared memory
            wait_store_reads(R.lag);
            const uint32_t rel = (stage + R.n_stages - R.lag) % R.n_stages;
            __syncwarp();                                             // every lane's stores have read the stage
            if (lane == 0) mbar_arrive(smem_addr(R.empty + rel));
        }
        if (++stage == R.n_stages) { stage = 0; phase ^= 1; }
    }
    // shared memory must outlive the stores that read it; other CTAs may be waiting for this one's tiles
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (p.n_levels > 1 && unpublished) {
        asm volatile("fence.proxy.async.global;" ::: "memory");
        __threadfence();
        __syncwarp();
        if (lane == 0) atomicAdd(&ctrl->done, unpublished);
    }
}


// Consumer warps of the converting ring: read fp32 from the stage, convert, store bf16 with plain 16-byte stores
// (bit-copy tiles of a mixed table: 16 bytes in, 16 bytes out).
// The unit is 8 elements: 32 bytes of shared memory in, 16 bytes out.  Each of the warps publishes its
// own share of a tile, so the completion counter of a cast table counts warp-tiles (15 per tile) and no wait
// between the warps (which could not be bounded) is needed.  Fifteen warps: a lone warp per scheduler would
// be bound by the latency of its own dependent instructions.
__device__ __forceinline__ void ring_consumer_cast(const WalkParams& p, const Ring& R, unsigned ct) {
    Ctrl* const    ctrl = p.ctrl;
    const unsigned lane = ct & 31;
    uint32_t       stage = 0, phase = 0, unpublished = 0;
    while (true) {
        bool ready = true;
        if (lane == 0) ready = mbar_wait(smem_addr(R.full + stage), phase);
        ready = __shfl_sync(0xffffffffu, ready, 0);
        if (!ready) {
            if (ct == 0) raise_status(ctrl, NEREUS_DEV_TIMEOUT, 0xFFFFFFFFu);
            break;
        }
        const StageMeta m = R.meta[stage];
        if (m.kind == kStageEnd) break;
        if (m.kind == kStageFlush) {
            __threadfence();
            __syncwarp();
            if (lane == 0 && unpublished) atomicAdd(&ctrl->done, unpublished);
            unpublished = 0;
        } else {
            // The stage holds the tile's row pieces back to back, so unit idx sits at idx * (bytes per unit) and
            // only its destination needs the row: idx * 16 + row * (pitch - width).  Rows come from one multiply
            // with the reciprocal the producer left in the record (a 32-bit division per unit would be a third
            // of this loop's instructions).
            const unsigned char* src = R.data + (size_t)stage * R.stage_bytes;
            const uint32_t nunit = (m.nr * m.w) >> 4, gap = m.dp - m.w;
            auto row_of = [&m](uint32_t idx) { return m.nr == 1 ? 0u : (m.magic ? __umulhi(idx, m.magic) : idx); };
            if (!m.cast) {
                // a bit-copy tile of a mixed table: 16 bytes per lane straight from the stage
#pragma unroll 2
                for (uint32_t idx = ct; idx < nunit; idx += kCastConsumers) {
                    const uint4 v = *reinterpret_cast<const uint4*>(src + idx * 16);
                    const uint32_t doff = idx * 16 + row_of(idx) * gap;
                    for (uint32_t j = 0; j < m.reps; ++j)
                        st_stream(tile_dst(p, m.dst_buf, m.rstride, m.d_off, j) + doff, v);
                }
            } else {
#pragma unroll 2
                for (uint32_t idx = ct; idx < nunit; idx += kCastConsumers) {
                    const uint4 a = *reinterpret_cast<const uint4*>(src + idx * 32);
                    const uint4 b = *reinterpret_cast<const uint4*>(src + idx * 32 + 16);
                    uint4 o;
                    o.x = cvt_bf16x2(__uint_as_float(a.x), __uint_as_float(a.y));
                    o.y = cvt_bf16x2(__uint_as_float(a.z), __uint_as_float(a.w));
                    o.z = cvt_bf16x2(__uint_as_float(b.x), __uint_as_float(b.y));
                    o.w = cvt_bf16x2(__uint_as_float(b.z), __uint_as_float(b.w));
                    if (nan_halves(o.x) | nan_halves(o.y) | nan_halves(o.z) | nan_halves(o.w)) {   // rare: a NaN among the eight
                        o.x = fix_nan_halves(o.x); o.y = fix_nan_halves(o.y);
                        o.z = fix_nan_halves(o.z); o.w = fix_nan_halves(o.w);
                    }
                    const uint32_t doff = idx * 16 + row_of(idx) * gap;
                    for (uint32_t j = 0; j < m.reps; ++j)
                        st_stream(tile_dst(p, m.dst_buf, m.rstride, m.d_off, j) + doff, o);
                }
            }
            ++unpublished;
        }
        __syncwarp();                                            // this warp is done reading the stage
        if (lane == 0) mbar_arrive(smem_addr(R.empty + stage));
        if (++stage == R.n_stages) { stage = 0; phase ^= 1; }
    }
    if (p.n_levels > 1 && unpublished) {
        __threadfence();
        __syncwarp();
        if (lane == 0) atomicAdd(&ctrl->done, unpublished);
    }
}

template <bool kCast>
__global__ void __launch_bounds__(kCast ? 32 + kCastConsumers : 64, kCast ? 1 : 2)
nereus_walk_ring(const __grid_constant__ WalkParams p, const uint32_t stage_bytes, const uint32_t n_stages,
                 const uint32_t piece, const uint32_t lag, const uint32_t claim) {
    extern __shared__ __align__(128) unsigned char smem[];
    Ring R;
    R.data  = smem;
    R.full  = reinterpret_cast<uint64_t*>(smem + (size_t)stage_bytes * n_stages);
    R.empty = R.full + n_stages;
    R.meta  = reinterpret_cast<StageMeta*>(R.empty + n_stages);
    R.stage_bytes = stage_bytes;
    R.n_stages = n_stages;
    R.piece = piece;
    R.lag = lag;
    R.claim = claim;
    const unsigned lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    trace_begin(p.trace);

    if (threadIdx.x == 0) {
        for (uint32_t i = 0; i < n_stages; ++i) {
            mbar_init(smem_addr(R.full + i), 1);
            mbar_init(smem_addr(R.empty + i), kCast ? kCastConsumers / 32 : 1);     // one arrival per consumer warp
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (warp == 0) ring_producer<kCast>(p, R, lane);
    else if (kCast) ring_consumer_cast(p, R, threadIdx.x - 32);
    else ring_consumer_copy(p, R, lane);
    finish_block(p.ctrl);
    trace_end(p.trace);
}

// ---------------------------------------------------------------------------------------------------
// host: prepare / run / status
// ---------------------------------------------------------------------------------------------------

static void drop_device_table(nereus_transition_s& t) {
    if (t.dev.device >= 0) {
        int cur = -1;
        if (cudaGetDevice(&cur) == cudaSuccess) {
            if (cur != t.dev.device) cudaSetDevice(t.dev.device);
            if (t.dev.rects) cudaFree(t.dev.rects);
            if (t.dev.trace) cudaFree(t.dev.trace);
            if (cur != t.dev.device) cudaSetDevice(cur);
        }
        (void)cudaGetLastError();
    }
    t.dev = DeviceTable();
}

static int env_int(const char* name, int dflt) {
    const char* v = getenv(name);
    return (v && *v) ? atoi(v) : dflt;
}

// Launch shape of one run, from the handle's tuning, the environment and the table.
struct Launch {
    int      variant = 1;           // 1 vector copy, 2 bulk-copy ring, 3 one warp per tile
    bool     cast = false;          // ring only: the table is all cast
    int      tile_bytes = 0, ctas_per_sm = 0, threads = 0;
    uint32_t n_stages = 0;          // bulk ring
    uint32_t piece = 16384, lag = 2, claim = 4;
    size_t   smem = 0;
};

// Which kernel walks a table (nereus_transition_tune and NEREUS_VARIANT override):
//   * single-level tables that write less than 1 GiB through at most kOnceMaxBuffers buffers: one warp per
//     tile (nereus_walk_once); measured on B200 it is the fastest from a few MB up to about 1 GiB;
//   * otherwise tables that write 64 MiB or more: the ring (its per-block start-up costs more than it gains
//     below that); all-bit-copy tables on the bulk-store consumer, anything with a cast in it on the
//     converting consumers (which copy the bit-copy tiles of a mixed table from shared memory as well);
//   * what is left (small chained tables, small tables with very many buffers, large bit-copy tables with 4% or
//     more of their bytes in row pieces below 1 KiB): the persistent vector kernel.
static int resolve_launch(const nereus_transition_s& t, int sms, Launch& L, bool once_fits = true) {
    const int want = t.tuning.variant ? t.tuning.variant : env_int("NEREUS_VARIANT", 0);
    const int asked_tile = t.tuning.tile_bytes ? t.tuning.tile_bytes : env_int("NEREUS_TILE_BYTES", 0);
    L.cast = false;
    for (const Rect& r : t.rects) L.cast = L.cast || r.cast;
    const bool once_ok = once_fits && t.n_levels == 1 &&
                         t.src_bytes.size() + t.dst_bytes.size() <= (size_t)kOnceMaxBuffers;
    if (want)  L.variant = want;
    else if (once_ok && t.bytes_written < (1ull << 30)) L.variant = 3;
    else       L.variant = (t.bytes_written >= (64ull << 20) && asked_tile <= (L.cast ? 24576 : 49152)) ? 2 : 1;
    if (L.variant == 3 && !once_ok) L.variant = 1;
    if (!want && L.variant == 2 && !L.cast && t.n_levels == 1) {
        // Row pieces below 1 KiB travel as one bulk copy each, and at 512 bytes those cost the ring 4 - 5% of a
        // whole 8B table in which they are 8% of the bytes (TP 16: 6.54 TB/s against 6.84 at 1 KiB pieces), while
        // the vector kernel moves them at its usual rate (6.72): it takes such tables.
        uint64_t small = 0;
        for (const Rect& r : t.rects)
            if (r.rows > 1 && r.width_dst < 1024) small += r.rows * r.width_dst * (uint64_t)r.replicas;
        if (small * 25 >= t.bytes_written) L.variant = 1;
    }
    L.ctas_per_sm = t.tuning.ctas_per_sm ? t.tuning.ctas_per_sm : env_int("NEREUS_CTAS_PER_SM", 2);
    L.threads     = t.tuning.threads     ? t.tuning.threads     : env_int("NEREUS_THREADS", L.variant == 3 ? 256 : 384);
    L.tile_bytes  = asked_tile;
    if (L.variant == 2) { L.ctas_per_sm = t.tuning.ctas_per_sm ? t.tuning.ctas_per_sm : 1; L.threads = 64; }
    if (L.ctas_per_sm < 1 || L.ctas_per_sm > 2 || L.threads < 32 || L.threads > 512 || L.threads % 32)
        return NEREUS_ERR_ARG;
    if (L.tile_bytes == 0) {
        // default: 16 KiB per warp tile (32 KiB per ring stage); smaller tiles for small tables, until at least
        // every other claimer gets a tile; a tile stays a multiple of 512 bytes
        L.tile_bytes = L.variant == 2 ? (L.cast ? 24576 : 32768) : 16384;
        const uint64_t claimers = (uint64_t)sms * L.ctas_per_sm * (L.variant == 2 ? 8 : L.threads / 32);
        while (L.variant != 3 && L.tile_bytes / 2 >= 1024 && (L.tile_bytes / 2) % 512 == 0 &&
               t.bytes_written / L.tile_bytes < claimers / 2)
            L.tile_bytes /= 2;
        if (L.variant == 3) {
            // one batch of loads per warp (32 lanes x 8 vectors = 4 KiB); smaller while the table would not
            // give every resident warp (32 per SM at 64 registers) a tile, larger only to stay within the
            // number of tiles that get per-tile records
            L.tile_bytes = 4096;
            while (L.tile_bytes > 1024 && t.bytes_written / L.tile_bytes < (uint64_t)sms * 32) L.tile_bytes /= 2;
            while (t.bytes_written / L.tile_bytes > kDirectMaxTiles * 3ull / 4) L.tile_bytes *= 2;
        }
    }
    if (L.tile_bytes < 512 || L.tile_bytes % 512) return NEREUS_ERR_ARG;
    if (L.variant == 2) {
        if (L.cast) L.ctas_per_sm = 1;
        const size_t budget = (227 * 1024) / L.ctas_per_sm - 1024;          // per CTA
        const size_t stage_bytes = (size_t)L.tile_bytes << (L.cast ? 1 : 0); // a cast stage holds the fp32 source
        if (stage_bytes > budget / 4) return NEREUS_ERR_ARG;
        const size_t per_stage = stage_bytes + 2 * sizeof(uint64_t) + sizeof(StageMeta);
        L.n_stages = (uint32_t)std::min<size_t>(kBulkMaxStages, budget / per_stage);
        L.smem = L.n_stages * per_stage;
        L.piece = (uint32_t)env_int("NEREUS_RING_PIECE", 16384);
        L.lag = (uint32_t)env_int("NEREUS_RING_LAG", std::min(3, (int)L.n_stages - 2));
        L.claim = (uint32_t)env_int("NEREUS_RING_CLAIM", 4);
        if (L.claim < 1 || L.claim > 64) return NEREUS_ERR_ARG;
        if (L.piece < 16 || L.piece % 16 || L.lag < 1 || L.lag > 8 || L.lag + 2 > L.n_stages) return NEREUS_ERR_ARG;
    }
    return NEREUS_OK;
}

// Kernel, launch shape and tiling of a table on a device with `sms` SMs, into arrays of rects.size() and
// rects.size() + 1 entries.  `records`: the caller can carry per-tile records (the allocation-free path
// cannot); a table that was to run one warp per tile but has more tiles than get records falls back to the
// kernels that search the tile prefix, with their own tile size.
static int plan_launch(const nereus_transition_s& t, int sms, bool records, Launch& L, RectDev* rects,
                       uint32_t* first, uint32_t level_end[kMaxLevels], uint64_t& n_tiles) {
    if (int rc = resolve_launch(t, sms, L, records)) return rc;
    n_tiles = tile_table_raw(t, (uint32_t)L.tile_bytes, rects, first, level_end);
    if (L.variant == 3 && (n_tiles == 0 || n_tiles > kDirectMaxTiles)) {
        if (int rc = resolve_launch(t, sms, L, false)) return rc;
        n_tiles = tile_table_raw(t, (uint32_t)L.tile_bytes, rects, first, level_end);
    }
    if (n_tiles == 0 && !t.rects.empty()) return NEREUS_ERR_UNSUPPORTED;      // more than 2^32 tiles
    return NEREUS_OK;
}

// The ring kernels use more dynamic shared memory than a kernel gets by default: opt in once per device (the
// launch itself then makes no other runtime call, which keeps it legal inside a stream capture).
constexpr int kMaxDevices = 64;
static bool g_ring_ready[kMaxDevices];

static int ring_opt_in(int device) {
    if (device < 0 || device >= kMaxDevices) return NEREUS_ERR_UNSUPPORTED;
    if (g_ring_ready[device]) return NEREUS_OK;
    const int most = 227 * 1024;
    NEREUS_CUDA(cudaFuncSetAttribute(nereus_walk_ring<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, most));
    NEREUS_CUDA(cudaFuncSetAttribute(nereus_walk_ring<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, most));
    g_ring_ready[device] = true;
    return NEREUS_OK;
}

static int launch_walk(const Launch& L, int sms, const WalkParams& p, cudaStream_t stream) {
    if (p.n_tiles == 0) return NEREUS_OK;
    if (L.variant == 2) {
        const unsigned grid = std::max(1u, std::min((unsigned)(sms * L.ctas_per_sm), p.n_tiles));
        if (L.cast) {
            nereus_walk_ring<true><<<grid, 32 + kCastConsumers, L.smem, stream>>>(p, (uint32_t)L.tile_bytes * 2, L.n_stages,
                                                                                  L.piece, L.lag, L.claim);
        } else {
            nereus_walk_ring<false><<<grid, 64, L.smem, stream>>>(p, (uint32_t)L.tile_bytes, L.n_stages, L.piece, L.lag, L.claim);
        }
    } else if (L.variant == 3 && p.tiles) {
        OnceParams o;
        o.tiles = p.tiles; o.ctrl = p.ctrl; o.trace = p.trace; o.n_tiles = p.n_tiles;
        for (int k = 0; k < kOnceMaxBuffers; ++k) o.bufs[k] = p.bufs[k];
        const unsigned warps_per_cta = (unsigned)L.threads / 32;
        nereus_walk_once<<<(p.n_tiles + warps_per_cta - 1) / warps_per_cta, L.threads, 0, stream>>>(o);
    } else {
        // (a table asked to run one warp per tile that turned out too large for per-tile records lands here)
        const unsigned warps_per_cta = (unsigned)L.threads / 32;
        unsigned grid = (unsigned)(sms * L.ctas_per_sm);
        grid = std::max(1u, std::min(grid, (p.n_tiles + warps_per_cta - 1) / warps_per_cta));
        nereus_walk_vec<<<grid, L.threads, 0, stream>>>(p);
    }
    NEREUS_CUDA(cudaGetLastError());
    return NEREUS_OK;
}

static int prepare(nereus_transition_s& t) {
    int device = 0;
    NEREUS_CUDA(cudaGetDevice(&device));
    if (t.dev.device == device && t.dev.rects) return NEREUS_OK;
    drop_device_table(t);

    int sms = 0;
    NEREUS_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    if (int rc = ring_opt_in(device)) return rc;
    DeviceTable dv;
    dv.device = device;
    dv.sm_count = sms;
    Launch L;
    std::vector<RectDev>  rects(t.rects.size());
    std::vector<uint32_t> first(t.rects.size() + 1);
    uint64_t n_tiles = 0;
    if (int rc = plan_launch(t, sms, true, L, rects.data(), first.data(), dv.level_end, n_tiles)) return rc;
    dv.tile_bytes = L.tile_bytes; dv.ctas_per_sm = L.ctas_per_sm; dv.threads = L.threads; dv.variant = L.variant;
    dv.n_tiles = (uint32_t)n_tiles;

    // nothing reaches the device that the host has not checked against the declared buffer sizes
    if (t.rects.size() >= (1u << 24)) return NEREUS_ERR_UNSUPPORTED;
    size_t entries = 0;
    for (const Rect& r : t.rects) entries += (size_t)std::max(1, std::min(r.replicas, kMaxReplicas));
    std::vector<uint32_t> order(entries + 1);
    if (int rc = validate_table(t, rects.data(), first.data(), n_tiles, order.data())) return rc;

    std::vector<TileRec> tiles;
    if (n_tiles <= kDirectMaxTiles) {
        tiles.resize(n_tiles);
        expand_tiles(rects.data(), rects.size(), tiles.data());
    }

    // one allocation: [rects | first | tiles | ctrl]
    const size_t rects_b = round_up(rects.size() * sizeof(RectDev), 256);
    const size_t first_b = round_up(first.size() * sizeof(uint32_t), 256);
    const size_t tiles_b = round_up(tiles.size() * sizeof(TileRec), 256);
    const size_t ctrl_b  = round_up(sizeof(Ctrl), 256);
    char* base = nullptr;
    NEREUS_CUDA(cudaMalloc(&base, rects_b + first_b + tiles_b + ctrl_b));
    dv.rects = reinterpret_cast<RectDev*>(base);
    dv.first = reinterpret_cast<uint32_t*>(base + rects_b);
    dv.tiles = tiles.empty() ? nullptr : reinterpret_cast<TileRec*>(base + rects_b + first_b);
    dv.ctrl  = reinterpret_cast<Ctrl*>(base + rects_b + first_b + tiles_b);
    cudaError_t e = cudaMemcpy(dv.rects, rects.data(), rects.size() * sizeof(RectDev), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(dv.first, first.data(), first.size() * sizeof(uint32_t), cudaMemcpyHostToDevice);
    if (e == cudaSuccess && !tiles.empty())
        e = cudaMemcpy(dv.tiles, tiles.data(), tiles.size() * sizeof(TileRec), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemset(dv.ctrl, 0, ctrl_b);
    if (e != cudaSuccess) { cudaFree(base); set_cuda_error((int)e); (void)cudaGetLastError(); return NEREUS_ERR_CUDA; }
    if (t.trace) {
        // one record per block of the launch this table will get
        const uint32_t warps = (uint32_t)L.threads / 32;
        dv.trace_blocks = L.variant == 3 ? (dv.n_tiles + warps - 1) / warps : (uint32_t)(sms * L.ctas_per_sm);
        dv.trace_blocks = std::max(1u, dv.trace_blocks);
        e = cudaMalloc(&dv.trace, (size_t)dv.trace_blocks * sizeof(BlockTrace));
        if (e == cudaSuccess) e = cudaMemset(dv.trace, 0, (size_t)dv.trace_blocks * sizeof(BlockTrace));
        if (e != cudaSuccess) {
            cudaFree(base);
            if (dv.trace) cudaFree(dv.trace);
            set_cuda_error((int)e); (void)cudaGetLastError();
            return NEREUS_ERR_CUDA;
        }
    }
    t.dev = dv;
    return NEREUS_OK;
}

static void fill_params(const nereus_transition_s& t, const void* const* src_ptrs, void* const* dst_ptrs,
                        WalkParams& p) {
    p.n_rects = (uint32_t)t.rects.size();
    p.n_levels = (uint32_t)t.n_levels;
    const size_t ns = t.src_bytes.size(), nd = t.dst_bytes.size();
    for (size_t i = 0; i < ns; ++i) p.bufs[i] = (char*)const_cast<void*>(src_ptrs[i]);
    for (size_t j = 0; j < nd; ++j) p.bufs[ns + j] = (char*)dst_ptrs[j];
    for (size_t k = ns + nd; k < (size_t)kMaxBuffers; ++k) p.bufs[k] = nullptr;
}

static bool overlap(const char* a, uint64_t na, const char* b, uint64_t nb) {
    return a < b + nb && b < a + na;
}

static int check_buffers(const nereus_transition_s& t, const void* const* src, void* const* dst) {
    const size_t ns = t.src_bytes.size(), nd = t.dst_bytes.size();
    for (size_t i = 0; i < ns; ++i) {
        if (!src[i]) return NEREUS_ERR_ARG;
        if ((uintptr_t)src[i] & 15) return NEREUS_ERR_ALIGN;
    }
    for (size_t j = 0; j < nd; ++j) {
        if (!dst[j]) return NEREUS_ERR_ARG;
        if ((uintptr_t)dst[j] & 15) return NEREUS_ERR_ALIGN;
    }
    for (size_t j = 0; j < nd; ++j) {
        const char* dj = (const char*)dst[j];
        // a destination may overlap an original source only if it is written after the source's last reader
        for (size_t i = 0; i < ns; ++i) {
            const int last_read = t.src_read_level.empty() ? 0 : t.src_read_level[i];
            if (t.dst_level[j] <= last_read && overlap(dj, t.dst_bytes[j], (const char*)src[i], t.src_bytes[i]))
                return NEREUS_ERR_ALIAS;
        }
        for (size_t k = j + 1; k < nd; ++k) {
            if (!overlap(dj, t.dst_bytes[j], (const char*)dst[k], t.dst_bytes[k])) continue;
            // two destinations may share memory only when the earlier one has been consumed before the
            // later one is written
            const size_t a = t.dst_level[j] <= t.dst_level[k] ? j : k, b = (a == j) ? k : j;
            if (t.dst_level[a] == t.dst_level[b]) return NEREUS_ERR_ALIAS;
            if (t.dst_read_level[a] < 0 || t.dst_level[b] <= t.dst_read_level[a]) return NEREUS_ERR_ALIAS;
        }
    }
    return NEREUS_OK;
}

// The status word is sticky on the device (first failure wins); reading it hands it to the host and clears it.
static int read_and_clear_status(Ctrl* ctrl, int* device_status) {
    Ctrl c;
    NEREUS_CUDA(cudaMemcpy(&c, ctrl, sizeof(Ctrl), cudaMemcpyDeviceToHost));
    if (c.status != (uint32_t)NEREUS_DEV_OK)
        NEREUS_CUDA(cudaMemset(&ctrl->status, 0, 2 * sizeof(uint32_t)));      // status and detail
    *device_status = (int)c.status;
    return NEREUS_OK;
}

}  // namespace nereus

extern "C" {

int nereus_transition_tune(nereus_transition_t t, int tile_bytes, int ctas_per_sm, int threads, int variant) {
    if (!t || tile_bytes < 0 || ctas_per_sm < 0 || threads < 0 || variant < 0 || variant > 3) return NEREUS_ERR_ARG;
    if (tile_bytes && (tile_bytes < 512 || tile_bytes % 512)) return NEREUS_ERR_ARG;
    if (ctas_per_sm > 2 || threads > 512 || threads % 32) return NEREUS_ERR_ARG;
    t->tuning.tile_bytes = tile_bytes; t->tuning.ctas_per_sm = ctas_per_sm;
    t->tuning.threads = threads; t->tuning.variant = variant;
    drop_device_table(*t);
    return NEREUS_OK;
}

int nereus_transition_num_tiles(nereus_transition_t t, uint64_t* tiles, int* levels) {
    try {
        if (!t || !tiles || !levels) return NEREUS_ERR_ARG;
        if (t->dev.rects) { *tiles = t->dev.n_tiles; *levels = t->n_levels; return NEREUS_OK; }
        // not prepared: what a 148-SM device would get
        std::vector<RectDev> rects(t->rects.size()); std::vector<uint32_t> first(t->rects.size() + 1);
        uint32_t le[kMaxLevels];
        Launch L;
        uint64_t n = 0;
        if (int rc = plan_launch(*t, 148, true, L, rects.data(), first.data(), le, n)) return rc;
        *tiles = n;
        *levels = t->n_levels;
        return NEREUS_OK;
    } catch (const std::bad_alloc&) { return NEREUS_ERR_NOMEM; }
}

int nereus_transition_get_tiles(nereus_transition_t t, uint64_t first, uint64_t count, nereus_rect_t* out) {
    try {
        if (!t || !out) return NEREUS_ERR_ARG;
        // the tiling of the prepared table, else what a 148-SM device would get
        std::vector<RectDev> rects(t->rects.size()); std::vector<uint32_t> prefix(t->rects.size() + 1);
        uint32_t le[kMaxLevels];
        Launch L;
        uint64_t n = 0;
        if (t->dev.rects) {
            if (int rc = resolve_launch(*t, t->dev.sm_count, L, t->dev.variant == 3)) return rc;
            n = tile_table_raw(*t, (uint32_t)t->dev.tile_bytes, rects.data(), prefix.data(), le);
        } else if (int rc = plan_launch(*t, 148, true, L, rects.data(), prefix.data(), le, n)) {
            return rc;
        }
        if (first > n || count > n - first) return NEREUS_ERR_ARG;
        if (n > (1u << 24)) return NEREUS_ERR_TOO_LARGE;              // an inspection call, not for 2^32 tiles
        std::vector<TileRec> tiles(n);
        expand_tiles(rects.data(), rects.size(), tiles.data());
        for (uint64_t k = 0; k < count; ++k) {
            const TileRec& e = tiles[first + k];
            nereus_rect_t& o = out[k];
            o.src_buf = e.src_buf; o.dst_buf = e.dst_buf; o.level = e.level; o.cast = e.cast;
            o.src_off = e.src_off; o.dst_off = e.dst_off;
            o.src_pitch = e.src_pitch; o.dst_pitch = e.dst_pitch;
            o.rows = e.rows; o.width_bytes_dst = e.width; o.width_bytes_src = (uint64_t)e.width << e.cast;
            o.replicas = e.replicas; o.replica_stride = e.replica_stride;
        }
        return NEREUS_OK;
    } catch (const std::bad_alloc&) { return NEREUS_ERR_NOMEM; }
}

int nereus_transition_launch_info(nereus_transition_t t, int* variant, int* tile_bytes, int* grid, int* threads) {
    try {
        if (!t || !variant || !tile_bytes || !grid || !threads) return NEREUS_ERR_ARG;
        const int sms = t->dev.rects ? t->dev.sm_count : 148;
        Launch L;
        uint64_t n_tiles = t->dev.n_tiles;
        if (t->dev.rects) {
            if (int rc = resolve_launch(*t, sms, L, t->dev.variant == 3)) return rc;
        } else {
            std::vector<RectDev> rects(t->rects.size()); std::vector<uint32_t> first(t->rects.size() + 1);
            uint32_t le[kMaxLevels];
            if (int rc = plan_launch(*t, sms, true, L, rects.data(), first.data(), le, n_tiles)) return rc;
        }
        const int warps = L.threads / 32;
        *grid = L.variant == 3 ? (int)((n_tiles + warps - 1) / warps) : sms * L.ctas_per_sm;   // one warp per tile
        *variant = L.variant; *tile_bytes = L.tile_bytes;
        *threads = L.variant == 2 ? (L.cast ? 32 + (int)kCastConsumers : 64) : L.threads;
        return NEREUS_OK;
    } catch (const std::bad_alloc&) { return NEREUS_ERR_NOMEM; }
}

int nereus_transition_prepare(nereus_transition_t t) {
    try {
        if (!t) return NEREUS_ERR_ARG;
        return prepare(*t);
    } catch (const std::bad_alloc&) { return NEREUS_ERR_NOMEM; }
}

int nereus_transition_run(nereus_transition_t t, const void* const* src_ptrs, void* const* dst_ptrs,
                          void* cuda_stream) {
    try {
        if (!t || !src_ptrs || !dst_ptrs) return NEREUS_ERR_ARG;
        if (int rc = check_buffers(*t, src_ptrs, dst_ptrs)) return rc;
        if (int rc = prepare(*t)) return rc;
        const DeviceTable& dv = t->dev;
        cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);

        Launch L;                       // the same answer prepare got (it falls back when per-tile records do not fit)
        if (int rc = resolve_launch(*t, dv.sm_count, L, dv.variant == 3)) return rc;
        if (L.variant != dv.variant || L.tile_bytes != dv.tile_bytes) return NEREUS_ERR_ARG;
        WalkParams p;
        // the control words need no reset: every launch leaves them zeroed for the next one
        p.rects = dv.rects; p.first = dv.first; p.tiles = dv.tiles; p.ctrl = dv.ctrl; p.trace = dv.trace;
        p.n_tiles = dv.n_tiles;
        if (dv.trace)               // tracing: every run starts from an empty trace
            NEREUS_CUDA(cudaMemsetAsync(dv.trace, 0, (size_t)dv.trace_blocks * sizeof(BlockTrace), stream));
        // NEREUS_DEBUG_GATE_BIAS (tests only): raises what a dependency gate waits for, so that it can never
        // open and the bounded wait must give up with NEREUS_DEV_TIMEOUT
        const uint32_t gate_bias = (uint32_t)env_int("NEREUS_DEBUG_GATE_BIAS", 0);
        for (int k = 0; k < kMaxLevels; ++k) p.level_end[k] = dv.level_end[k] + gate_bias;
        fill_params(*t, src_ptrs, dst_ptrs, p);

        if (int rc = launch_walk(L, dv.sm_count, p, stream)) return rc;
        t->dev.runs += 1;
        if (dv.n_tiles > 0) t->launches += 1;
        return NEREUS_OK;
    } catch (const std::bad_alloc&) { return NEREUS_ERR_NOMEM; }
}

int nereus_transition_run_sized(nereus_transition_t t, const void* const* src_ptrs, const size_t* src_sizes,
                                void* const* dst_ptrs, const size_t* dst_sizes, void* cuda_stream) {
    if (!t || !src_ptrs || !dst_ptrs || !src_sizes || !dst_sizes) return NEREUS_ERR_ARG;
    // the table was checked against the sizes it declares; here the caller's buffers are checked against those
    for (size_t i = 0; i < t->src_bytes.size(); ++i)
        if (src_sizes[i] < t->src_bytes[i]) return NEREUS_ERR_TOO_SMALL;
    for (size_t j = 0; j < t->dst_bytes.size(); ++j)
        if (dst_sizes[j] < t->dst_bytes[j]) return NEREUS_ERR_TOO_SMALL;
    return nereus_transition_run(t, src_ptrs, dst_ptrs, cuda_stream);
}

int nereus_transition_status(nereus_transition_t t, int* device_status) {
    if (!t || !device_status) return NEREUS_ERR_ARG;
    if (!t->dev.rects) { *device_status = NEREUS_DEV_OK; return NEREUS_OK; }
    if (t->dev.runs == 0) { *device_status = NEREUS_DEV_OK; return NEREUS_OK; }
    return read_and_clear_status(t->dev.ctrl, device_status);
}

int nereus_transition_trace(nereus_transition_t t, int enable) {
    if (!t) return NEREUS_ERR_ARG;
    t->trace = enable != 0;
    drop_device_table(*t);
    return NEREUS_OK;
}

int nereus_transition_trace_read(nereus_transition_t t, nereus_block_trace_t* out, int cap, int* n) {
    if (!t || !out || !n || cap < 0) return NEREUS_ERR_ARG;
    if (!t->dev.trace || (uint32_t)cap < t->dev.trace_blocks) return NEREUS_ERR_ARG;
    NEREUS_CUDA(cudaMemcpy(out, t->dev.trace, (size_t)t->dev.trace_blocks * sizeof(BlockTrace), cudaMemcpyDeviceToHost));
    *n = (int)t->dev.trace_blocks;
    return NEREUS_OK;
}

int nereus_transition_launches(nereus_transition_t t, uint64_t* n) {
    if (!t || !n) return NEREUS_ERR_ARG;
    *n = t->launches;
    return NEREUS_OK;
}

int nereus_transition_destroy(nereus_transition_t t) {
    if (!t) return NEREUS_ERR_ARG;
    drop_device_table(*t);
    delete t;
    return NEREUS_OK;
}

int nereus_last_cuda_error(void) { return g_last_cuda_error; }

}  // extern "C"

// ---------------------------------------------------------------------------------------------------
// run without any allocation: the task table lives in a fixed device array
// ---------------------------------------------------------------------------------------------------
//
// Some callers cannot allocate device memory at the moment they need a transition: an engine that handed
// all of HBM to its own pool (a serving process with a pre-sized KV cache, a trainer whose caching
// allocator owns the device) has nothing left for cudaMalloc to give, and at a near-capacity safe boundary
// the allocation that prepare() makes may simply fail.  For them the table and the control words sit in
// this file-scope array, which every process that loads the library holds on every GPU it touches until
// it exits.

namespace nereus {

constexpr int    kStaticMaxRects    = NEREUS_STATIC_MAX_RECTS;
constexpr int    kStaticMaxEntries  = 4 * kStaticMaxRects;            // (task, replica) pairs the check can sort
constexpr size_t kStaticRectBytes   = (size_t)kStaticMaxRects * sizeof(RectDev);              // 256 KiB
constexpr size_t kStaticFirstBytes  = ((size_t)kStaticMaxRects + 1 + 63) / 64 * 64 * sizeof(uint32_t);
constexpr size_t kStaticScratchBytes = kStaticRectBytes + kStaticFirstBytes + 256;            // ~272 KiB

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kStaticMaxDevices = kMaxDevices;
static unsigned char* g_static_ptr[kStaticMaxDevices];   // device address of the array, per device
static int            g_static_sms[kStaticMaxDevices];

// Host staging of the tiled table: plain file-scope arrays (part of the library's image, so no thread's first
// call allocates anything), shared by all threads under a lock that is held until the runtime has taken the
// bytes.
static std::mutex g_static_lock;
static RectDev    g_static_rects[kStaticMaxRects];
static uint32_t   g_static_first[kStaticMaxRects + 1];
static uint32_t   g_static_order[kStaticMaxEntries + 1];

// Once per device, with that device current: the array's name is only a host-side handle of the symbol;
// the address a kernel can use comes from cudaGetSymbolAddress.
static int static_scratch(int device, unsigned char** ptr, int* sms) {
    if (device < 0 || device >= kStaticMaxDevices) return NEREUS_ERR_UNSUPPORTED;
    if (!g_static_ptr[device]) {
        unsigned char* p = nullptr;
        NEREUS_CUDA(cudaGetSymbolAddress((void**)&p, g_static_scratch));
        if (int rc = ring_opt_in(device)) return rc;
        int n = 0;
        NEREUS_CUDA(cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, device));
        g_static_sms[device] = n;
        g_static_ptr[device] = p;
    }
    *ptr = g_static_ptr[device];
    *sms = g_static_sms[device];
    return NEREUS_OK;
}

static Ctrl* static_ctrl(unsigned char* scratch) {
    return reinterpret_cast<Ctrl*>(scratch + kStaticRectBytes + kStaticFirstBytes);
}

}  // namespace nereus

extern "C" int nereus_transition_run_static(nereus_transition_t t, const void* const* src_ptrs,
                                            void* const* dst_ptrs, void* cuda_stream) try {
    if (!t || !src_ptrs || !dst_ptrs) return NEREUS_ERR_ARG;
    const size_t n_rects = t->rects.size();
    if (n_rects > (size_t)kStaticMaxRects) return NEREUS_ERR_TOO_LARGE;
    size_t entries = 0;
    for (const Rect& r : t->rects) entries += (size_t)std::max(1, std::min(r.replicas, kMaxReplicas));
    if (entries > (size_t)kStaticMaxEntries) return NEREUS_ERR_TOO_LARGE;
    if (int rc = check_buffers(*t, src_ptrs, dst_ptrs)) return rc;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    // the table is uploaded from host arrays that the next call overwrites: a captured copy of them would
    // replay whatever table came last, so the call is refused while the stream is being captured
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    NEREUS_CUDA(cudaStreamIsCapturing(stream, &capturing));
    if (capturing != cudaStreamCaptureStatusNone) return NEREUS_ERR_UNSUPPORTED;

    std::lock_guard<std::mutex> hold(g_static_lock);
    int device = 0;
    NEREUS_CUDA(cudaGetDevice(&device));
    unsigned char* scratch = nullptr;
    int sms = 0;
    if (int rc = static_scratch(device, &scratch, &sms)) return rc;

    Launch L;
    WalkParams p;
    uint64_t n_tiles = 0;      // no room for per-tile records in the fixed array: the kernels that search the prefix
    if (int rc = plan_launch(*t, sms, false, L, g_static_rects, g_static_first, p.level_end, n_tiles)) return rc;
    if (int rc = validate_table(*t, g_static_rects, g_static_first, n_tiles, g_static_order)) return rc;

    RectDev*  d_rects = reinterpret_cast<RectDev*>(scratch);
    uint32_t* d_first = reinterpret_cast<uint32_t*>(scratch + kStaticRectBytes);
    Ctrl*     d_ctrl  = static_ctrl(scratch);
    // The array keeps whatever the previous call left: overwrite the table and zero the cursor and the two
    // counters (a launch leaves them zeroed, but nothing here relies on how the last one ended).  The status
    // word stays: it is sticky until nereus_static_status reads it.  The copies come from pageable memory:
    // the runtime has taken the bytes by the time each call returns, so the lock may then be released.
    NEREUS_CUDA(cudaMemcpyAsync(d_rects, g_static_rects, n_rects * sizeof(RectDev), cudaMemcpyHostToDevice, stream));
    NEREUS_CUDA(cudaMemcpyAsync(d_first, g_static_first, (n_rects + 1) * sizeof(uint32_t), cudaMemcpyHostToDevice, stream));
    NEREUS_CUDA(cudaMemsetAsync(d_ctrl, 0, 3 * sizeof(uint32_t), stream));

    p.rects = d_rects; p.first = d_first; p.tiles = nullptr; p.ctrl = d_ctrl; p.trace = nullptr;
    p.n_tiles = (uint32_t)n_tiles;
    const uint32_t gate_bias = (uint32_t)env_int("NEREUS_DEBUG_GATE_BIAS", 0);     // tests of the failure path only
    for (int k = 0; k < kMaxLevels; ++k) p.level_end[k] += gate_bias;
    fill_params(*t, src_ptrs, dst_ptrs, p);
    if (int rc = launch_walk(L, sms, p, stream)) return rc;
    if (n_tiles > 0) t->launches += 1;
    return NEREUS_OK;
} catch (...) {
    return NEREUS_ERR_UNSUPPORTED;      // the lock could not be taken; nothing here allocates, so nothing else throws
}

extern "C" int nereus_static_status(int* device_status) {
    if (!device_status) return NEREUS_ERR_ARG;
    int device = 0;
    NEREUS_CUDA(cudaGetDevice(&device));
    if (device < 0 || device >= kStaticMaxDevices) return NEREUS_ERR_UNSUPPORTED;
    if (!g_static_ptr[device]) { *device_status = NEREUS_DEV_OK; return NEREUS_OK; }   // no static run here yet
    return read_and_clear_status(static_ctrl(g_static_ptr[device]), device_status);
}
