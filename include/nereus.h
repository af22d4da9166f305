/*
 * nereus.h -- C ABI of the B200-native EMU reshard.
 *
 * One model-stage's parameter shards theta = {theta_i}, i = 1..tp*pp (the EMU of Section 5 of the Nereus
 * paper) are carried from a source (TP, PP) layout to a target (TP, PP) layout on ONE GPU, every virtual
 * TP/PP rank's shard being a separate device buffer.  This is the local layout change that the paper's Split
 * and Merge primitives perform next to their collectives (Section 6.2, "DAG Execution and Safety" and
 * "Resharding--transport interplay"); it re-cuts and moves the state and leaves the logical state untouched
 * (Section 6.2, "Preserving training semantics").  An optional fp32 -> bf16 round-to-nearest-even cast is
 * fused into the move for the training -> generation weight sync between the actor's two model-stages
 * (Section 5, EMU definition).
 *
 * The paper fixes none of the tensor-level layout; this header does (see "Layout contract").
 *
 * Conventions
 *   - Every function returns an int: NEREUS_OK (0) or a negative NEREUS_ERR_* code.  Nothing throws, aborts
 *     or prints.  Output arguments are written only on success.
 *   - "host" / "device" next to a pointer says where the pointed-to memory lives.
 *   - The library never allocates, frees or keeps shard memory; the caller owns every shard buffer.  A
 *     handle owns only its task table (host copy, plus one device copy per nereus_transition_prepare).
 *   - Handles are not thread-safe; use one handle from one thread at a time.
 *
 * Layout contract
 *   model    L layers, hidden H, nq query heads, nkv KV heads (nkv | nq), head_dim hd = H / nq, FFN F,
 *            vocabulary V, Llama-style: untied embedding, RMSNorm weights only, no biases.
 *   logical tensors, row-major [out, in]:
 *            embed [V,H]; per layer ln1 [H], wq [nq*hd,H], wk [nkv*hd,H], wv [nkv*hd,H], wo [H,nq*hd],
 *            ln2 [H], wgate [F,H], wup [F,H], wdown [H,F]; ln_f [H]; head [V,H] (or a value head [1,H]).
 *   plan     (tp, pp, dtype).  Pipeline stage p owns layers [p*L/pp, (p+1)*L/pp) (when pp does not divide L the
 *            first L mod pp stages own one layer more than the others); embed lives on stage 0,
 *            ln_f and the head on stage pp-1.  Shard index = p*tp + r (TP rank r fastest).
 *   TP rank r of t stores
 *            embed, LM head   rows [r*V/t, (r+1)*V/t)                        (vocabulary-parallel)
 *            qkv              one fused block [Q_r ; K_r ; V_r]: the rows of q heads [r*nq/t, (r+1)*nq/t),
 *                             then of kv heads [r*nkv/t, (r+1)*nkv/t) of wk, then the same of wv (so a
 *                             rank's q heads are exactly the GQA groups of its kv heads)
 *            wo               columns [r*nq*hd/t, (r+1)*nq*hd/t), stored contiguously as [H, nq*hd/t]
 *            gate_up          one fused block [G_r ; U_r], each F/t rows
 *            wdown            columns [r*F/t, (r+1)*F/t), stored as [H, F/t]
 *            ln1, ln2, ln_f, value head   the whole tensor on every TP rank of the owning stage
 *   shard buffer packing: [embed], then per local layer ln1, qkv, wo, ln2, gate_up, wdown, then
 *            [ln_f, head]; every stored tensor starts on a 256-byte boundary; the buffer length is the end
 *            of the last tensor rounded up to 256 bytes.  Padding bytes are never read and never written.
 *   stored tensor ids (argument tensor_id below): 0 = embed; 1 + 6*l + k for layer l and
 *            k = 0 ln1, 1 qkv, 2 wo, 3 ln2, 4 gate_up, 5 wdown; 1 + 6*L = ln_f; 2 + 6*L = head.
 *   layout variants (nereus_plan_t.layout) reorder the rows inside qkv and gate_up, see the flags below.
 *   tp > nkv (nkv | tp): every kv head is replicated on tp/nkv consecutive ranks; rank r stores head
 *            r / (tp/nkv), the one its q heads attend to; as a source only the first copy of a head is read.
 *   required: tp | nkv or nkv | tp, tp | nq, tp | F, tp | V (unless padded), pp <= L, and every contiguous piece
 *            a transition moves must start on and span a multiple of 16 bytes on both sides (for the cast: 8
 *            elements).
 */
#ifndef NEREUS_H_
#define NEREUS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define NEREUS_OK                 0
#define NEREUS_ERR_ARG           -1   /* null pointer, negative or zero size, index out of range          */
#define NEREUS_ERR_INDIVISIBLE   -2   /* a divisibility or 16-byte rule of the layout contract fails       */
#define NEREUS_ERR_UNSUPPORTED   -3   /* dtype pair other than same->same or fp32->bf16; more buffers than */
                                      /* one launch can address; a call that is not allowed in this state  */
#define NEREUS_ERR_ALIAS         -4   /* a destination buffer overlaps a source or another destination     */
#define NEREUS_ERR_CUDA          -5   /* a CUDA call failed; see nereus_last_cuda_error                    */
#define NEREUS_ERR_NOMEM         -6   /* host allocation failed                                            */
#define NEREUS_ERR_MISMATCH      -7   /* parts of a chained fuse do not connect (buffer count or sizes)    */
#define NEREUS_ERR_ALIGN         -8   /* a shard pointer is not 16-byte aligned                            */
#define NEREUS_ERR_TOO_LARGE     -9   /* more tasks than the fixed scratch of nereus_transition_run_static */
/* -10 is NEREUS_ERR_INFEASIBLE, declared with the transition DAG below */
#define NEREUS_ERR_TABLE         -11  /* the task table failed the host-side check that precedes every upload */
#define NEREUS_ERR_TOO_SMALL     -12  /* a buffer handed to nereus_transition_run_sized is shorter than required */

/* device status word (nereus_transition_status) */
#define NEREUS_DEV_OK             0
#define NEREUS_DEV_BOUNDS         1   /* a claimed tile did not resolve to a task: corrupted table         */
#define NEREUS_DEV_TIMEOUT        2   /* a wait inside the kernel gave up: a dependency gate after about   */
                                      /* 0.5 s of polling, a shared-memory barrier after 0.5 s on the GPU's */
                                      /* global timer (with a cap of 2^22 attempts behind it)              */

typedef enum { NEREUS_BF16 = 1, NEREUS_FP32 = 2 } nereus_dtype_t;

typedef struct nereus_model_desc_s* nereus_model_desc_t;   /* opaque, host */
typedef struct nereus_transition_s* nereus_transition_t;   /* opaque, host; owns the task table */

/* Order of the rows inside a rank's fused blocks (which heads and rows a rank holds never changes):
 *   NEREUS_QKV_GROUPED          for each kv head of the rank: its q heads, its k head, its v head (the order
 *                               Megatron-style trainers keep), instead of [all Q ; all K ; all V]
 *   NEREUS_GATE_UP_INTERLEAVED  g0, u0, g1, u1, ... row by row (what some fused SwiGLU kernels read), instead
 *                               of [all gate ; all up]
 * A transition may convert between layouts, e.g. grouped fp32 training weights to blocked bf16 for generation.
 *   NEREUS_VOCAB_PADDED         the vocabulary dimension of embed and LM head is padded up to a multiple of
 *                               128*tp before it is cut (what Megatron-style trainers do): rank r stores
 *                               V_pad/tp rows; rows past V are padding, never read and never written; V need
 *                               not divide by tp under this flag
 */
#define NEREUS_QKV_GROUPED          1
#define NEREUS_GATE_UP_INTERLEAVED  2
#define NEREUS_VOCAB_PADDED         4

/* A (TP, PP) layout.  dtype 0 means "the descriptor's dtype"; layout is a mask of the flags above. */
typedef struct { int tp; int pp; int dtype; int layout; } nereus_plan_t;

/* One rect-copy task of a compiled transition, for inspection and tests.  Buffer indices address the
 * concatenation [src_ptrs..., dst_ptrs...] that nereus_transition_run receives ("unified index").
 * The task copies `rows` pieces; piece i is `width_bytes_dst` bytes at dst_off + i*dst_pitch and comes
 * from `width_bytes_src` bytes at src_off + i*src_pitch (twice as many when cast = 1). */
typedef struct {
    int32_t  src_buf, dst_buf;      /* unified buffer indices */
    int32_t  level;                 /* dependency level: tasks of level k run after all of level k-1 */
    int32_t  cast;                  /* 1: fp32 -> bf16 RNE, 0: bit copy */
    uint64_t src_off, dst_off;      /* bytes from the start of the buffer */
    uint64_t src_pitch, dst_pitch;  /* bytes between consecutive pieces */
    uint64_t rows;
    uint64_t width_bytes_src, width_bytes_dst;
    int32_t  replicas;              /* the piece is written `replicas` times: to buffers dst_buf + j*replica_stride */
    int32_t  replica_stride;
} nereus_rect_t;

/* ---- model descriptor (EMU field M and the shapes of theta; Section 5) -------------------------------- */

/* Describes a Llama-style decoder.  dtype is the element type of plans whose dtype field is 0.
 * Errors: ARG (non-positive size, bad dtype, null out), INDIVISIBLE (heads does not divide hidden, or
 * kv_heads does not divide heads). */
int nereus_model_desc(int layers, int hidden, int heads, int kv_heads, int ffn, int vocab, int dtype,
                      nereus_model_desc_t* out);
/* Replaces the LM head [V,H] by a value head [out_dim,H], out_dim = 1 (critic / reward model-stages).
 * The value head is replicated over TP.  Errors: ARG, UNSUPPORTED (out_dim != 1). */
int nereus_model_desc_set_value_head(nereus_model_desc_t desc, int out_dim);
int nereus_model_desc_destroy(nereus_model_desc_t desc);

/* ---- layout queries (theta_i, i = p*tp + r; Section 5) ------------------------------------------------ */

/* Checks the layout contract's divisibility rules for one plan.  Errors: ARG, INDIVISIBLE, UNSUPPORTED. */
int nereus_plan_check(nereus_model_desc_t desc, nereus_plan_t plan);
int nereus_plan_num_shards(nereus_model_desc_t desc, nereus_plan_t plan, int* n);            /* tp*pp */
int nereus_plan_shard_bytes(nereus_model_desc_t desc, nereus_plan_t plan, int shard, size_t* bytes);
/* Number of stored tensor ids, 6*L + 3. */
int nereus_model_num_tensors(nereus_model_desc_t desc, int* n);
/* Where `shard` keeps stored tensor `tensor_id`: byte offset, and the stored block's rows x cols in
 * elements (row-major, cols contiguous).  rows = cols = 0 when the shard's stage does not own the tensor.
 * replicated = 1 for tensors that every TP rank of the stage holds whole. */
int nereus_plan_tensor_slice(nereus_model_desc_t desc, nereus_plan_t plan, int shard, int tensor_id,
                             size_t* offset, size_t* rows, size_t* cols, int* replicated);

/* ---- transition compiler (the change Delta_M = (E_M -> E*_M) of Section 6.1, at tensor granularity) ---- */

/* Compiles src -> dst for one model-stage into rect-copy tasks by intersecting every destination slice
 * with the source slices directly (no intermediate layout).  Host work only.
 * Errors: ARG, INDIVISIBLE, UNSUPPORTED (dtype pair, too many buffers), NOMEM. */
int nereus_transition_compile(nereus_model_desc_t desc, nereus_plan_t src, nereus_plan_t dst,
                              nereus_transition_t* out);
/* Same, with `replicas` identical destination units (1..16): every source byte is read once and written
 * `replicas` times.  This is the data movement of Extend (Section 5.2(c): replicate a unit onto new GPUs,
 * rank-aligned, each shard sent once; use src == dst) and of a Split that yields k replica units (Section
 * 5.2(a)).  run() takes replicas * tp*pp destination pointers, replica-major: unit 0's shards, unit 1's, ...
 * Errors: as nereus_transition_compile, plus ARG (replicas out of range). */
int nereus_transition_compile_replicated(nereus_model_desc_t desc, nereus_plan_t src, nereus_plan_t dst,
                                         int replicas, nereus_transition_t* out);
/* The EMU's full state (theta, omega) in one table: the parameters src -> dst as above, plus `n_opt`
 * optimizer tensors per parameter (Adam: 2), held in fp32 and sharded exactly like the parameters (Section 5
 * gives omega the layout of theta).  run() takes, on either side, the parameter shards followed by the
 * shards of optimizer tensor 0, then of tensor 1, ...; optimizer shards have the sizes of an fp32 plan with
 * the same tp and pp.  Optimizer state is never cast.  Errors: as nereus_transition_compile, ARG (n_opt < 0). */
int nereus_transition_compile_state(nereus_model_desc_t desc, nereus_plan_t src, nereus_plan_t dst, int n_opt,
                                    nereus_transition_t* out);
/* Fuses n compiled transitions into one task table that one launch executes (the readiness rule of Section
 * 6.2: work whose predecessors are done may run side by side, nothing starts before its predecessors end).
 *   chained = 0: the parts are independent model-stages.  run() takes the concatenation of the parts'
 *                source arrays and the concatenation of their destination arrays.  One level.
 *   chained = 1: part k+1 reads what part k wrote: its source buffers ARE part k's destination buffers
 *                (same count and sizes, else MISMATCH).  run() takes part 0's sources and the concatenation
 *                of all parts' destinations; part k is dependency level k.
 * The parts stay valid and independent of the fused handle.  Errors: ARG, MISMATCH, UNSUPPORTED, NOMEM. */
int nereus_transition_fuse(const nereus_transition_t* parts, int n, int chained, nereus_transition_t* out);
int nereus_transition_destroy(nereus_transition_t t);

/* Number of source / destination buffers run() expects, and the minimum length of each. */
int nereus_transition_num_buffers(nereus_transition_t t, int* n_src, int* n_dst);
int nereus_transition_buffer_bytes(nereus_transition_t t, int is_dst, int index, size_t* bytes);
/* Algorithmic bytes one run reads and writes (sum over tasks; replicated tensors once per replica). */
int nereus_transition_bytes(nereus_transition_t t, size_t* read, size_t* written);
/* The task table, in execution order (level, then largest first). */
int nereus_transition_num_rects(nereus_transition_t t, int* n);
int nereus_transition_get_rect(nereus_transition_t t, int index, nereus_rect_t* out);
/* Tiles one run claims, and dependency levels. */
int nereus_transition_num_tiles(nereus_transition_t t, uint64_t* tiles, int* levels);
/* Tiles [first, first + count) of the tiling one run walks, in claim order, each as the task it amounts to
 * (`rows` pieces of `width_bytes_dst` bytes at its own offsets): what a claimer of tile g moves.  These are
 * the per-tile records that tables of up to 2^17 tiles carry to the device.  `out` (host) holds `count`
 * entries.  For inspection and tests.  Errors: ARG (range), TOO_LARGE (more than 2^24 tiles), NOMEM. */
int nereus_transition_get_tiles(nereus_transition_t t, uint64_t first, uint64_t count, nereus_rect_t* out);
/* Checks the task table on the host, as nereus_transition_prepare and nereus_transition_run_static do before
 * anything reaches a device (Section 6.2, "Safe concurrent execution": a buffer is only read or written inside
 * its declared extent and nothing writes where another task of the same step writes): every task lies inside
 * nereus_transition_buffer_bytes of its source and of each destination replica, offsets, widths and pitches
 * follow the 16-byte rule, a pitch is at least a width, buffer indices and levels are in range and in
 * execution order, a chained task reads only what an earlier level wrote, and the destinations of all tasks
 * are pairwise disjoint.  Errors: ARG, NEREUS_ERR_TABLE, NOMEM. */
int nereus_transition_validate(nereus_transition_t t);
/* Test hook: overwrites task `index` of a table that has not been uploaded yet, without any check, so that the
 * validator can be shown a corrupted table.  Errors: ARG, UNSUPPORTED (the table is already on a device). */
int nereus_debug_set_rect(nereus_transition_t t, int index, const nereus_rect_t* task);

/* Launch tuning; 0 keeps the default of a field.  tile_bytes: target bytes per tile (multiple of 512).
 * ctas_per_sm, threads: the persistent kernels' grid = SMs * ctas_per_sm blocks of `threads` threads; kernel 3
 * takes `threads` only (its grid follows the tile count).
 * variant: which kernel walks the table.
 *   0  default: kernel 3 for single-level tables that write less than 1 GiB through at most 64 buffers;
 *      otherwise kernel 2 for tables that write 64 MiB or more and kernel 1 below that; kernel 1 also for large
 *      bit-copy tables with 4% or more of their bytes in row pieces shorter than 1 KiB (each such piece is one
 *      bulk copy in kernel 2, which costs it more than the register path)
 *   1  persistent register-staged vector copy: a warp per tile, tiles claimed from a cursor (16 KiB tiles,
 *      smaller for small tables until every other warp finds work)
 *   2  persistent bulk-copy ring through shared memory (32 KiB per stage; 24 KiB when the table contains a
 *      cast: the stage then holds the fp32 source).  A stage must fit four times into the shared memory of
 *      an SM, else ARG at prepare
 *   3  one warp per tile without a loop, addresses from per-tile records (4 KiB tiles, down to 1 KiB for
 *      tables too small to give every resident warp a tile, larger as needed to stay within 2^17 tiles);
 *      asked for on a chained table, on more than 64 buffers or on more than 2^17 tiles it falls back to 1
 * Drops the device copy of the table (the next prepare/run uploads it again).  Errors: ARG. */
int nereus_transition_tune(nereus_transition_t t, int tile_bytes, int ctas_per_sm, int threads, int variant);

/* The launch shape the next run on the current device will use (after nereus_transition_prepare; before it,
 * what a 148-SM device would get): the kernel that runs (1, 2 or 3 as above, after any fall-back), tile
 * bytes, grid, block. */
int nereus_transition_launch_info(nereus_transition_t t, int* variant, int* tile_bytes, int* grid, int* threads);

/* ---- execution (the local layout change of Section 6.2) ---------------------------------------------- */

/* Checks the task table (nereus_transition_validate, plus the tiling) and uploads it to the current device
 * (cudaMalloc + synchronous copy).  Optional: run() does it on first use.  Call it ahead of time to keep
 * allocation out of a timed or captured region.  Tables of up to 2^17 tiles also get one 48-byte record per
 * tile, which saves the kernel the search for a tile's task.  Errors: ARG, UNSUPPORTED, NEREUS_ERR_TABLE, CUDA. */
int nereus_transition_prepare(nereus_transition_t t);
/* Enqueues the whole transition on `cuda_stream` (a cudaStream_t; NULL = the default stream) as one
 * kernel launch and returns without synchronising.
 *   src_ptrs (host array of device pointers): source shard i = p*tp + r; read-only during the run.
 *   dst_ptrs (host array of device pointers): destination shards; every byte of every stored tensor is
 *            written exactly once, padding is untouched.
 * Both arrays are copied before the call returns.  Every pointer must be 16-byte aligned and address at
 * least nereus_transition_buffer_bytes bytes.  Sources stay live until the stream reaches the end of the
 * run (Section 6.2: source buffers live until their readers complete).
 * A prepared run enqueues nothing but the kernel: the control words are left zeroed by every launch (the last
 * block to finish clears them), so the launch may be captured into a CUDA graph and replayed, each replay
 * moving whatever the buffers hold by then.
 * Errors: ARG (null), ALIGN, ALIAS, CUDA, and what prepare reports.  Runs of the same handle must not overlap
 * on the device. */
int nereus_transition_run(nereus_transition_t t, const void* const* src_ptrs, void* const* dst_ptrs,
                          void* cuda_stream);
/* The same, with the lengths in bytes of the caller's buffers (host arrays, one entry per pointer): a buffer
 * shorter than nereus_transition_buffer_bytes is refused with NEREUS_ERR_TOO_SMALL before anything is enqueued.
 * Together with the check of the table against those required lengths (nereus_transition_validate, run by
 * prepare) this bounds every access of the kernel by what the caller really holds.  Errors: as run, TOO_SMALL. */
int nereus_transition_run_sized(nereus_transition_t t, const void* const* src_ptrs, const size_t* src_sizes,
                                void* const* dst_ptrs, const size_t* dst_sizes, void* cuda_stream);
/* Environment variables read by prepare() and by every run(): NEREUS_TILE_BYTES, NEREUS_CTAS_PER_SM,
 * NEREUS_THREADS, NEREUS_VARIANT (defaults of the tuning fields; a run whose kernel or tile size no longer is
 * what the table was prepared with returns ARG: call nereus_transition_tune to re-prepare), NEREUS_RING_PIECE,
 * NEREUS_RING_LAG, NEREUS_RING_CLAIM (ring internals), and, for tests of the failure path only,
 * NEREUS_DEBUG_GATE_BIAS: a count added to what every dependency gate waits for, so that
 * the gate cannot open; the waits then run into their poll limit (about half a second), the run ends with
 * device status NEREUS_DEV_TIMEOUT and the destinations of the gated levels stay unwritten. */

/* Reads the device status word (NEREUS_DEV_*): the first failure of any run of this handle since the word was
 * last read, NEREUS_DEV_OK if there was none; a failure that has been read is cleared.  The caller must have
 * synchronised the stream first; this call copies a few bytes from the device synchronously. */
int nereus_transition_status(nereus_transition_t t, int* device_status);
/* Kernels this handle has launched since it was created (one per run). */
int nereus_transition_launches(nereus_transition_t t, uint64_t* n);

/* Per-block trace of a run, for looking at load balance (who got how many tiles, how far apart the blocks
 * finish): the tool this library offers where the paper's framework instrumentation provides kernel times
 * (Section 4.1, monitor phase).  nereus_transition_trace(t, 1) switches it on (and drops the device copy of the
 * table, like nereus_transition_tune); every run then zeroes the trace (one small memset in front of the
 * kernel, so a traced run is not what one times) and every block records the GPU's global timer when it starts
 * and when it finishes and the number of tiles it moved.  nereus_transition_trace_read copies the records of
 * the last run to `out` (host, `cap` entries; *n gets the number of blocks) after the caller has synchronised.
 * Errors: ARG (also: tracing is off, cap too small), CUDA. */
typedef struct { uint64_t begin_ns, end_ns; uint32_t tiles, block; } nereus_block_trace_t;
int nereus_transition_trace(nereus_transition_t t, int enable);
int nereus_transition_trace_read(nereus_transition_t t, nereus_block_trace_t* out, int cap, int* n);

/* ---- cost side: the transition estimate and the admission gate (Sections 4.3 and 6) ------------------- */

/* L_tran of a compiled transition: in the paper the critical-path cost is a function of the bytes moved, the
 * bandwidth of the link and the time to set communicators up (Section 6); on one GPU the link is HBM and the
 * set-up is the launch.  Levels run
 * one after another, so seconds = setup_seconds + sum over levels of (bytes read + written) / bandwidth.
 * gbytes_per_s: the sustained reshard bandwidth (e.g. a value bench.py measured); must be > 0.
 * Errors: ARG. */
int nereus_transition_estimate(nereus_transition_t t, double gbytes_per_s, double setup_seconds, double* seconds);

/* The profitability gate, Eq. 2 of Section 4.3: with delta_l = l_step_current - l_step_target (seconds per
 * step), an executable opportunistic transition is admitted iff delta_l > 0 and
 * l_tran / delta_l <= gamma * h_x, the payback period in steps against a fraction gamma in [0, 1] of the
 * horizon h_x (steps until the triggering signal's next threshold crossing; the smallest one when several
 * signals trigger).  urgent != 0 waives profitability (the urgent path).  gamma = 0 therefore admits only
 * urgent transitions.  *admit gets 0 or 1, *payback_steps (optional) the ratio, +inf when delta_l <= 0.
 * Errors: ARG (negative cost, gamma outside [0, 1], negative horizon, null admit). */
int nereus_admit(double l_tran, double l_step_current, double l_step_target, double gamma, double h_x,
                 int urgent, int* admit, double* payback_steps);

/* H_x: an exponential moving average of the intervals (in steps) between threshold crossings of one signal,
 * updated at crossings only; one step before the first interval is observed (Section 4.3).  The paper does
 * not give the averaging weight; `weight` in (0, 1] is the share of the newest interval (this build's
 * default reading: 0.5).  The first observed interval replaces the initial value. */
typedef struct { double h_steps; double weight; int observed; } nereus_horizon_t;
int nereus_horizon_init(nereus_horizon_t* h, double weight);
int nereus_horizon_crossing(nereus_horizon_t* h, double interval_steps);

/* ---- transition DAG over EMU primitives (Section 6.1) -------------------------------------------------- */

/* Host-side planner.  Each model-stage M brings its current collection E_M and its target collection E*_M
 * (units = (tp, pp, GPU list in shard order p*tp + r)); nereus_dag_plan turns every change Delta_M into a
 * local DAG in the paper's default order Split -> Destroy -> Extend -> Merge and combines the local DAGs
 * into one global DAG:
 *   - T_sub = (gcd(tp, tp*), gcd(pp, pp*)), the largest layout both sides split into; Split(EMU, T_sub) makes
 *     k = tp*pp / |T_sub| replica units on the unit's own GPUs, sub-unit j on GPUs [j*|T_sub|, (j+1)*|T_sub|);
 *   - the target units' GPUs are cut into slots the same way; a slot that already holds a sub-unit (same
 *     GPUs, same order) keeps it; every other sub-unit is redundant and gets a Destroy; every other slot is
 *     filled by an Extend from the lowest-numbered kept sub-unit that shares no GPU with the slot (else the
 *     lowest-numbered such sub-unit at all: Extend copies onto a disjoint GPU set), and a unit that an Extend
 *     still reads is destroyed only after it; Merge fuses a target unit's slots;
 *   - resources are bytes of GPU memory: a unit keeps state_bytes / (tp*pp) on each of its GPUs, every GPU
 *     has gpu_capacity bytes; Split / Extend / Merge need room for what they create, Split / Destroy / Merge
 *     free what they consume when they complete;
 *   - the schedule takes ready primitives releasing-before-acquiring, then in stage order generation ->
 *     inference -> training, then by model-stage and primitive index; because ready primitives run
 *     concurrently, a primitive that only fits thanks to memory another primitive freed gets a
 *     resource-dependency edge to it (newest release first); a blocked acquisition selects an executable
 *     Destroy that frees one of its GPUs and does not depend on it; if there is none the plan is infeasible.
 * Everything above the first item of each bullet is this build's reading of Section 6.1. */
typedef struct nereus_dag_s* nereus_dag_t;
#define NEREUS_GENERATION 0
#define NEREUS_INFERENCE  1
#define NEREUS_TRAINING   2
#define NEREUS_OP_SPLIT   0
#define NEREUS_OP_DESTROY 1
#define NEREUS_OP_EXTEND  2
#define NEREUS_OP_MERGE   3
#define NEREUS_ERR_INFEASIBLE   -10   /* an acquisition stays blocked: the target plan fails the feasibility check */

typedef struct {
    int32_t op, stage;                 /* NEREUS_OP_*, model-stage index */
    int32_t n_src, n_dst;              /* units read / created */
    int32_t n_deps, n_resource_deps;   /* state edges / resource-dependency edges (primitive indices) */
    int32_t order;                     /* position in the serial schedule */
    int32_t level;                     /* longest path from a root: primitives of one level may run together */
} nereus_prim_t;

int nereus_dag_create(nereus_dag_t* out);
int nereus_dag_destroy(nereus_dag_t dag);
/* Adds a model-stage; kind = NEREUS_GENERATION / INFERENCE / TRAINING, state_bytes = one replica's state. */
int nereus_dag_add_stage(nereus_dag_t dag, int kind, uint64_t state_bytes, int* stage);
/* Adds a unit to a stage's current (is_target = 0) or target collection; gpus (host) has tp*pp entries. */
int nereus_dag_add_unit(nereus_dag_t dag, int stage, int is_target, int tp, int pp, const int* gpus);
/* Plans.  gpu_capacity 0 = unlimited.  Errors: ARG (a stage without units, mixed layouts inside a collection,
 * a layout T_sub does not divide), UNSUPPORTED (a target slot that overlaps every unit it could be copied
 * from without coinciding with one), NEREUS_ERR_INFEASIBLE. */
int nereus_dag_plan(nereus_dag_t dag, uint64_t gpu_capacity);
int nereus_dag_num_units(nereus_dag_t dag, int* n);          /* current units first, then created ones */
int nereus_dag_unit(nereus_dag_t dag, int unit, int* stage, int* tp, int* pp, int* gpus, int gpus_cap);
int nereus_dag_num_prims(nereus_dag_t dag, int* n);
int nereus_dag_prim(nereus_dag_t dag, int prim, nereus_prim_t* out);
/* Copies the primitive's lists; each pointer may be NULL, else it must hold the matching count. */
int nereus_dag_prim_lists(nereus_dag_t dag, int prim, int* src, int* dst, int* deps, int* resource_deps);

/* Lowers a planned DAG to ONE task table that one launch executes (the readiness rule of Section 6.2 becomes
 * dependency levels): every data-moving primitive becomes the
 * tasks of a transition between its units' layouts and takes its DAG level as dependency level.
 *   Split(u -> k units of T_sub)   u's layout -> T_sub, read once, written to the k sub-units
 *   Extend(s -> n)                 T_sub -> T_sub copy of s into n
 *   Merge(subs -> v)               T_sub -> v's layout; target shard i is cut from the sub-unit that sits on
 *                                  the same GPU, i.e. subs[i / |T_sub|] (local slicing of replicated state)
 *   Destroy                        no device work
 * descs[m] describes model-stage m (its dtype is the state's dtype; plans use layout 0).  run() then takes as
 * src_ptrs the shards of the current units, unit by unit in unit order, and as dst_ptrs the shards of every
 * created unit (sub-units, extended units, target units) in unit order; a destroyed unit's memory may be
 * reused for a unit created after the last primitive that reads it.
 * Errors: ARG (not planned, or planned without success: an infeasible DAG has no schedule to lower),
 * UNSUPPORTED (more than 8 data-moving levels or too many buffers), and whatever
 * nereus_transition_compile reports for a layout. */
int nereus_dag_lower(nereus_dag_t dag, const nereus_model_desc_t* descs, int n_descs, nereus_transition_t* out);

/* ---- execution without allocation --------------------------------------------------------------------- */

/* The paper has no counterpart of this entry point; it exists for callers that cannot allocate device
 * memory when a transition is due: a process that gave all of HBM to its own pool (a server with a
 * pre-sized KV cache, a trainer whose caching allocator owns the device) has nothing left for cudaMalloc,
 * and at a near-capacity boundary the table upload of nereus_transition_prepare may fail.
 *
 * Same contract, arguments and result as nereus_transition_run, but it calls no cudaMalloc, cudaFree or any
 * other allocating routine, on the device or on the host heap, and never touches the handle's device copy:
 * the task table and the control words go into one fixed array in the library's device image,
 * NEREUS_STATIC_MAX_RECTS tasks at most (about 272 KiB, held on every GPU the process uses until it exits),
 * and the host side stages the table in fixed arrays of the library's own image.  The table is checked
 * (as by nereus_transition_validate) and copied there on `cuda_stream` by every call (two small
 * cudaMemcpyAsync and a 12-byte memset ahead of the kernel).
 *   - A transition with more tasks (nereus_transition_num_rects), or with more than 4 * NEREUS_STATIC_MAX_RECTS
 *     (task, replica) pairs, is refused with NEREUS_ERR_TOO_LARGE.
 *   - The first call on a device does the set-up for that device: it looks the array's device address up
 *     (cudaGetSymbolAddress), reads the SM count and opts the kernels into their shared memory.  Make that
 *     first call before any stream capture begins.  While `cuda_stream` is being captured every call is
 *     refused with NEREUS_ERR_UNSUPPORTED: the
 *     table is uploaded from host arrays that the next call overwrites, so a captured upload would replay
 *     whichever table came last.
 *   - The uploads read pageable host memory: the runtime takes the bytes before each copy call returns, and
 *     to do so it may wait for earlier work of the stream.  Unlike nereus_transition_run the call can
 *     therefore block for as long as the stream's backlog.
 *   - All handles and all calls on one device share the array, which keeps the previous call's contents
 *     until the next one overwrites it: two calls whose work overlaps on the GPU (different streams, or
 *     different threads) race on it.  Issue them on one stream, or order them with events.  (Host threads
 *     are serialised by a lock around the staging arrays; that does not order their work on the GPU.)
 *   - nereus_transition_status does not see these runs: their status word lives in the shared array; read
 *     it with nereus_static_status. */
#define NEREUS_STATIC_MAX_RECTS 4096
int nereus_transition_run_static(nereus_transition_t t, const void* const* src_ptrs, void* const* dst_ptrs,
                                 void* cuda_stream);
/* Device status (NEREUS_DEV_*) of the static runs on the current device: the first failure since the word was
 * last read (NEREUS_DEV_OK if none, or if no static run was made on this device); reading clears it.  The
 * caller must have synchronised the stream of those runs.  Allocates nothing; copies a few bytes from the
 * device synchronously.  Like the entry point it serves, it has no counterpart in the paper. */
int nereus_static_status(int* device_status);

const char* nereus_strerror(int code);
/* cudaError_t of the last failed CUDA call made by this library on the calling thread (0 if none). */
int nereus_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* NEREUS_H_ */
