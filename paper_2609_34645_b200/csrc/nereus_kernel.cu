// Device side of the EMU reshard for sm_100a: one persistent kernel walks the task table of a compiled
// transition (the local layout change of Section 6.2 of the Nereus paper) and moves every rect-copy task's
// bytes from the source shards to the destination shards, with an optional fused fp32 -> bf16
// round-to-nearest-even cast.  Pure data movement: the bound is HBM bandwidth, there is no tensor-core work.
//
// Execution model
//   * grid = SMs x ctas_per_sm persistent blocks; every WARP claims tiles on its own: lane 0 takes the next
//     tile index from a global cursor with one atomicAdd and broadcasts it by shuffle; the claim of the next
//     tile is issued before the current tile is copied, so its latency hides behind the copy.
//   * a tile index is resolved to its rect by binary search in the tile-prefix array, then to a row block /
//     column block of that rect by arithmetic; every lane moves 16-byte vectors, 32 lanes x 16 B = 512 B
//     contiguous per instruction, kUnroll independent loads in flight per lane before the first store.
//   * tables with several dependency levels (chained transitions): a tile of level k waits, with a poll
//     limit, until every tile of level k-1 has completed; on giving up it records NEREUS_DEV_TIMEOUT and the
//     warp leaves.  Loads bypass L1 (ld.global.cg) so a level reads what another SM wrote before it.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
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
    Ctrl*           ctrl;
    uint32_t        n_rects, n_tiles, n_levels;
    uint32_t        level_end[kMaxLevels];
    char*           bufs[kMaxBuffers];
};
static_assert(sizeof(WalkParams) <= 4000, "kernel parameter block too large");

constexpr int      kUnrollRun   = 8;            // 16-byte loads in flight per lane, contiguous runs
constexpr int      kUnrollRect  = 8;            // ... pitched rects and the cast
constexpr uint32_t kGatePolls   = 1u << 21;     // x ~200 ns sleep: gives up after roughly half a second

// ---------------------------------------------------------------------------------------------------
// device helpers
// ---------------------------------------------------------------------------------------------------

__device__ __forceinline__ uint32_t claim_tile(Ctrl* ctrl, unsigned lane) {
    uint32_t g = 0;
    if (lane == 0) g = atomicAdd(&ctrl->cursor, 1u);
    return __shfl_sync(0xffffffffu, g, 0);
}

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ uint4 ld_stream(const char* p) { return __ldcg(reinterpret_cast<const uint4*>(p)); }
__device__ __forceinline__ void  st_stream(char* p, uint4 v) { __stcs(reinterpret_cast<uint4*>(p), v); }
__device__ __forceinline__ void  st_stream8(char* p, uint2 v) { __stcs(reinterpret_cast<uint2*>(p), v); }

// two fp32 -> packed bf16x2, round to nearest even; NaN (any payload, either sign) -> 0x7FC0
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    if (lo != lo) r = (r & 0xFFFF0000u) | 0x00007FC0u;
    if (hi != hi) r = (r & 0x0000FFFFu) | 0x7FC00000u;
    return r;
}

// Bit copy of a contiguous run of `nvec` 16-byte vectors.
template <int kUnroll>
__device__ __forceinline__ void copy_run(const char* __restrict__ s, char* __restrict__ d, uint32_t nvec,
                                         unsigned lane) {
    s += lane * 16;
    d += lane * 16;
    uint32_t left = nvec;
#pragma unroll 1
    for (; left >= 32 * kUnroll; left -= 32 * kUnroll) {          // full batches: no predicates
        uint4 v[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) v[u] = ld_stream(s + u * 512);
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) st_stream(d + u * 512, v[u]);
        s += 512 * kUnroll;
        d += 512 * kUnroll;
    }
#pragma unroll 1
    for (uint32_t i = lane; i < left; i += 32) {                  // ragged tail, one vector at a time
        st_stream(d, ld_stream(s));
        s += 512;
        d += 512;
    }
}

// Bit copy of a pitched tile: `rows` pieces of `vpr` 16-byte vectors each.  Offsets inside a tile fit
// 32 bits (rows_per_tile x pitch is far below 4 GiB).
template <int kUnroll>
__device__ __forceinline__ void copy_rect(const char* __restrict__ s, char* __restrict__ d, uint32_t rows,
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
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) st_stream(d + doff[u], v[u]);
    }
#pragma unroll 1
    for (; base < nvec; base += 32) {                                  // ragged tail
        const uint32_t r = base / vpr, c = base - r * vpr;
        st_stream(d + (r * dp + c * 16), ld_stream(s + (r * sp + c * 16)));
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

template <int kUnroll>
__device__ __forceinline__ void cast_tile(const char* __restrict__ s, char* __restrict__ d, uint32_t rows,
                                          uint32_t upr, uint32_t sp, uint32_t dp, unsigned lane) {
    const uint32_t nunit = rows * upr;
    uint32_t       base = lane;
#pragma unroll 1
    for (; base + 32 * (kUnroll - 1) < nunit; base += 32 * kUnroll) {
        uint4    v[kUnroll];
        uint32_t doff[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const uint32_t idx = base + u * 32;
            const uint32_t r = idx / upr, c = idx - r * upr;
            doff[u] = r * dp + c * 8;
            v[u] = ld_stream(s + (r * sp + c * 16));
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) st_stream8(d + doff[u], cast_unit(v[u]));
    }
#pragma unroll 1
    for (; base < nunit; base += 32) {
        const uint32_t r = base / upr, c = base - r * upr;
        st_stream8(d + (r * dp + c * 8), cast_unit(ld_stream(s + (r * sp + c * 16))));
    }
}

// ---------------------------------------------------------------------------------------------------
// the persistent walker (register-staged vector copy)
// ---------------------------------------------------------------------------------------------------

__global__ void __launch_bounds__(512, 2) nereus_walk_vec(const __grid_constant__ WalkParams p) {
    const unsigned lane = threadIdx.x & 31;
    Ctrl* const    ctrl = p.ctrl;

    uint32_t g = claim_tile(ctrl, lane);
    while (g < p.n_tiles) {
        const uint32_t g_next = claim_tile(ctrl, lane);      // in flight while this tile is copied

        // tile -> rect: largest i with first[i] <= g
        uint32_t lo = 0, hi = p.n_rects;                       // invariant: first[lo] <= g < first[hi]
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) >> 1;
            if (__ldg(p.first + mid) <= g) lo = mid; else hi = mid;
        }
        const RectDev* rp = p.rects + lo;
        const uint4 q0 = __ldg(reinterpret_cast<const uint4*>(rp));          // src_off, dst_off
        const uint4 q1 = __ldg(reinterpret_cast<const uint4*>(rp) + 1);      // width, src_pitch, dst_pitch
        const uint4 q2 = __ldg(reinterpret_cast<const uint4*>(rp) + 2);      // rows, rows_per_tile, tile_w, col_tiles
        const uint4 q3 = __ldg(reinterpret_cast<const uint4*>(rp) + 3);      // first_tile, bufs, level|cast
        const uint64_t src_off = ((uint64_t)q0.y << 32) | q0.x, dst_off = ((uint64_t)q0.w << 32) | q0.z;
        const uint64_t width   = ((uint64_t)q1.y << 32) | q1.x;
        const uint32_t sp = q1.z, dp = q1.w;
        const uint32_t rows = q2.x, rpt = q2.y, tile_w = q2.z, col_tiles = q2.w;
        const uint32_t first_tile = q3.x;
        const uint32_t src_buf = q3.y & 0xFFFFu, dst_buf = q3.y >> 16;
        const uint32_t level = q3.z & 0xFFFFu, cast = q3.z >> 16;

        if (first_tile > g || src_buf >= (uint32_t)kMaxBuffers || dst_buf >= (uint32_t)kMaxBuffers) {
            if (lane == 0) { atomicCAS(&ctrl->status, NEREUS_DEV_OK, NEREUS_DEV_BOUNDS); ctrl->detail = g; }
            return;
        }

        // dependency gate
        if (level > 0) {
            const uint32_t need = p.level_end[level - 1];
            uint32_t polls = 0;
            bool ok = true;
            if (lane == 0) {
                while (ld_acquire_u32(&ctrl->done) < need) {
                    if (++polls > kGatePolls) { ok = false; break; }
                    __nanosleep(200);
                }
                if (!ok) { atomicCAS(&ctrl->status, NEREUS_DEV_OK, NEREUS_DEV_TIMEOUT); ctrl->detail = g; }
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) return;
            __threadfence();
        }

        // tile -> row block x column block
        const uint32_t t  = g - first_tile;
        const uint32_t rb = t / col_tiles, cb = t - rb * col_tiles;
        const uint32_t r0 = rb * rpt;
        const uint32_t nr = min(rpt, rows - r0);
        const uint64_t c0 = (uint64_t)cb * tile_w;                     // dst bytes into the row piece
        const uint32_t w  = (uint32_t)min((uint64_t)tile_w, width - c0);
        const char* s = p.bufs[src_buf] + src_off + (uint64_t)r0 * sp + (c0 << cast);
        char*       d = p.bufs[dst_buf] + dst_off + (uint64_t)r0 * dp + c0;

        if (cast) {
            cast_tile<kUnrollRect>(s, d, nr, w >> 3, sp, dp, lane);
        } else if (nr == 1) {
            copy_run<kUnrollRun>(s, d, w >> 4, lane);
        } else {
            copy_rect<kUnrollRect>(s, d, nr, w >> 4, sp, dp, lane);
        }

        if (p.n_levels > 1) {
            __threadfence();
            __syncwarp();
            if (lane == 0) atomicAdd(&ctrl->done, 1u);
        }
        g = g_next;
    }
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

static int prepare(nereus_transition_s& t) {
    int device = 0;
    NEREUS_CUDA(cudaGetDevice(&device));
    if (t.dev.device == device && t.dev.rects) return NEREUS_OK;
    drop_device_table(t);

    int sms = 0;
    NEREUS_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));

    DeviceTable dv;
    dv.device = device;
    dv.sm_count = sms;
    dv.tile_bytes  = t.tuning.tile_bytes  ? t.tuning.tile_bytes  : env_int("NEREUS_TILE_BYTES", 16384);
    dv.ctas_per_sm = t.tuning.ctas_per_sm ? t.tuning.ctas_per_sm : env_int("NEREUS_CTAS_PER_SM", 2);
    dv.threads     = t.tuning.threads     ? t.tuning.threads     : env_int("NEREUS_THREADS", 512);
    dv.variant     = t.tuning.variant     ? t.tuning.variant     : env_int("NEREUS_VARIANT", 1);
    if (dv.tile_bytes < 512 || dv.tile_bytes % 512 || dv.ctas_per_sm < 1 || dv.ctas_per_sm > 2 ||
        dv.threads < 32 || dv.threads > 512 || dv.threads % 32)
        return NEREUS_ERR_ARG;

    std::vector<RectDev>  rects;
    std::vector<uint32_t> first;
    const uint64_t n_tiles = tile_table(t, (uint32_t)dv.tile_bytes, rects, first, dv.level_end);
    if (n_tiles == 0 && !t.rects.empty()) return NEREUS_ERR_UNSUPPORTED;
    dv.n_tiles = (uint32_t)n_tiles;

    // one allocation: [rects | first | ctrl]
    const size_t rects_b = round_up(rects.size() * sizeof(RectDev), 256);
    const size_t first_b = round_up(first.size() * sizeof(uint32_t), 256);
    char* base = nullptr;
    NEREUS_CUDA(cudaMalloc(&base, rects_b + first_b + 256));
    dv.rects = reinterpret_cast<RectDev*>(base);
    dv.first = reinterpret_cast<uint32_t*>(base + rects_b);
    dv.ctrl  = reinterpret_cast<Ctrl*>(base + rects_b + first_b);
    cudaError_t e = cudaMemcpy(dv.rects, rects.data(), rects.size() * sizeof(RectDev), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(dv.first, first.data(), first.size() * sizeof(uint32_t), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemset(dv.ctrl, 0, 256);
    if (e != cudaSuccess) { cudaFree(base); set_cuda_error((int)e); (void)cudaGetLastError(); return NEREUS_ERR_CUDA; }
    t.dev = dv;
    return NEREUS_OK;
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
        // a destination may overlap an original source only if it is written after level 0 has read it
        for (size_t i = 0; i < ns; ++i)
            if (t.dst_level[j] == 0 && overlap(dj, t.dst_bytes[j], (const char*)src[i], t.src_bytes[i]))
                return NEREUS_ERR_ALIAS;
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

}  // namespace nereus

extern "C" {

int nereus_transition_tune(nereus_transition_t t, int tile_bytes, int ctas_per_sm, int threads, int variant) {
    if (!t || tile_bytes < 0 || ctas_per_sm < 0 || threads < 0 || variant < 0) return NEREUS_ERR_ARG;
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
        std::vector<RectDev> rects; std::vector<uint32_t> first; uint32_t le[kMaxLevels];
        const int tb = t->dev.rects ? t->dev.tile_bytes
                                    : (t->tuning.tile_bytes ? t->tuning.tile_bytes : env_int("NEREUS_TILE_BYTES", 16384));
        *tiles = tile_table(*t, (uint32_t)tb, rects, first, le);
        *levels = t->n_levels;
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

        WalkParams p;
        p.rects = dv.rects; p.first = dv.first; p.ctrl = dv.ctrl;
        p.n_rects = (uint32_t)t->rects.size(); p.n_tiles = dv.n_tiles; p.n_levels = (uint32_t)t->n_levels;
        for (int k = 0; k < kMaxLevels; ++k) p.level_end[k] = dv.level_end[k];
        const size_t ns = t->src_bytes.size(), nd = t->dst_bytes.size();
        for (size_t i = 0; i < ns; ++i) p.bufs[i] = (char*)const_cast<void*>(src_ptrs[i]);
        for (size_t j = 0; j < nd; ++j) p.bufs[ns + j] = (char*)dst_ptrs[j];
        for (size_t k = ns + nd; k < (size_t)kMaxBuffers; ++k) p.bufs[k] = nullptr;

        NEREUS_CUDA(cudaMemsetAsync(dv.ctrl, 0, sizeof(Ctrl), stream));
        if (dv.n_tiles > 0) {
            const unsigned warps_needed = dv.n_tiles;
            unsigned grid = (unsigned)(dv.sm_count * dv.ctas_per_sm);
            const unsigned warps_per_cta = (unsigned)dv.threads / 32;
            grid = std::max(1u, std::min(grid, (warps_needed + warps_per_cta - 1) / warps_per_cta));
            nereus_walk_vec<<<grid, dv.threads, 0, stream>>>(p);
            NEREUS_CUDA(cudaGetLastError());
            t->launches += 1;
        }
        return NEREUS_OK;
    } catch (const std::bad_alloc&) { return NEREUS_ERR_NOMEM; }
}

int nereus_transition_status(nereus_transition_t t, int* device_status) {
    if (!t || !device_status) return NEREUS_ERR_ARG;
    if (!t->dev.rects) { *device_status = NEREUS_DEV_OK; return NEREUS_OK; }
    Ctrl c;
    NEREUS_CUDA(cudaMemcpy(&c, t->dev.ctrl, sizeof(Ctrl), cudaMemcpyDeviceToHost));
    *device_status = (int)c.status;
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

constexpr int    kStaticMaxRects    = 4096;
constexpr size_t kStaticRectBytes   = (size_t)kStaticMaxRects * sizeof(RectDev);              // 256 KiB
constexpr size_t kStaticFirstBytes  = ((size_t)kStaticMaxRects + 1 + 63) / 64 * 64 * sizeof(uint32_t);
constexpr size_t kStaticScratchBytes = kStaticRectBytes + kStaticFirstBytes + 256;            // ~272 KiB

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kStaticMaxDevices = 64;
static unsigned char* g_static_ptr[kStaticMaxDevices];   // device address of the array, per device
static int            g_static_sms[kStaticMaxDevices];

// Once per device, with that device current: the array's name is only a host-side handle of the symbol;
// the address a kernel can use comes from cudaGetSymbolAddress.
static int static_scratch(int device, unsigned char** ptr, int* sms) {
    if (device < 0 || device >= kStaticMaxDevices) return NEREUS_ERR_UNSUPPORTED;
    if (!g_static_ptr[device]) {
        unsigned char* p = nullptr;
        NEREUS_CUDA(cudaGetSymbolAddress((void**)&p, g_static_scratch));
        int n = 0;
        NEREUS_CUDA(cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, device));
        g_static_sms[device] = n;
        g_static_ptr[device] = p;
    }
    *ptr = g_static_ptr[device];
    *sms = g_static_sms[device];
    return NEREUS_OK;
}

}  // namespace nereus

extern "C" int nereus_transition_run_static(nereus_transition_t t, const void* const* src_ptrs,
                                            void* const* dst_ptrs, void* cuda_stream) {
    try {
        if (!t || !src_ptrs || !dst_ptrs) return NEREUS_ERR_ARG;
        if (t->rects.size() > (size_t)kStaticMaxRects) return NEREUS_ERR_TOO_LARGE;
        if (int rc = check_buffers(*t, src_ptrs, dst_ptrs)) return rc;
        int device = 0;
        NEREUS_CUDA(cudaGetDevice(&device));
        unsigned char* scratch = nullptr;
        int sms = 0;
        if (int rc = static_scratch(device, &scratch, &sms)) return rc;
        cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);

        const int tile_bytes  = t->tuning.tile_bytes  ? t->tuning.tile_bytes  : env_int("NEREUS_TILE_BYTES", 16384);
        const int ctas_per_sm = t->tuning.ctas_per_sm ? t->tuning.ctas_per_sm : env_int("NEREUS_CTAS_PER_SM", 2);
        const int threads     = t->tuning.threads     ? t->tuning.threads     : env_int("NEREUS_THREADS", 512);
        if (tile_bytes < 512 || tile_bytes % 512 || ctas_per_sm < 1 || ctas_per_sm > 2 || threads < 32 ||
            threads > 512 || threads % 32)
            return NEREUS_ERR_ARG;

        WalkParams p;
        std::vector<RectDev>  rects;        // host memory only
        std::vector<uint32_t> first;
        const uint64_t n_tiles = tile_table(*t, (uint32_t)tile_bytes, rects, first, p.level_end);
        if (n_tiles == 0 && !t->rects.empty()) return NEREUS_ERR_UNSUPPORTED;

        RectDev*  d_rects = reinterpret_cast<RectDev*>(scratch);
        uint32_t* d_first = reinterpret_cast<uint32_t*>(scratch + kStaticRectBytes);
        Ctrl*     d_ctrl  = reinterpret_cast<Ctrl*>(scratch + kStaticRectBytes + kStaticFirstBytes);
        // the array keeps whatever the previous call left: overwrite the table, zero the control words
        NEREUS_CUDA(cudaMemcpyAsync(d_rects, rects.data(), rects.size() * sizeof(RectDev), cudaMemcpyHostToDevice, stream));
        NEREUS_CUDA(cudaMemcpyAsync(d_first, first.data(), first.size() * sizeof(uint32_t), cudaMemcpyHostToDevice, stream));
        NEREUS_CUDA(cudaMemsetAsync(d_ctrl, 0, sizeof(Ctrl), stream));

        p.rects = d_rects; p.first = d_first; p.ctrl = d_ctrl;
        p.n_rects = (uint32_t)t->rects.size(); p.n_tiles = (uint32_t)n_tiles; p.n_levels = (uint32_t)t->n_levels;
        const size_t ns = t->src_bytes.size(), nd = t->dst_bytes.size();
        for (size_t i = 0; i < ns; ++i) p.bufs[i] = (char*)const_cast<void*>(src_ptrs[i]);
        for (size_t j = 0; j < nd; ++j) p.bufs[ns + j] = (char*)dst_ptrs[j];
        for (size_t k = ns + nd; k < (size_t)kMaxBuffers; ++k) p.bufs[k] = nullptr;
        if (n_tiles > 0) {
            const unsigned warps_per_cta = (unsigned)threads / 32;
            unsigned grid = (unsigned)(sms * ctas_per_sm);
            grid = std::max(1u, std::min(grid, ((unsigned)n_tiles + warps_per_cta - 1) / warps_per_cta));
            nereus_walk_vec<<<grid, threads, 0, stream>>>(p);
            NEREUS_CUDA(cudaGetLastError());
            t->launches += 1;
        }
        return NEREUS_OK;
    } catch (const std::bad_alloc&) { return NEREUS_ERR_NOMEM; }
}
