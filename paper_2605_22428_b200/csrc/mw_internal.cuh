// Internal declarations shared by the translation units of libmw.so.  Not part of the C ABI.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "mw.h"

#define MW_TILE 256          // tokens per plan tile = threads per plan block
#define MW_SMALL_T_MAX 1024  // largest T the single-block plan handles

// Per-plan accumulators filled by atomics; double buffered by plan parity so that the
// buffer of the next plan is cleared by the current one and no separate memset is needed.
struct mw_acc {
    unsigned long long valid_slots;  // expert slots that named a valid expert on a valid rank
    unsigned int self_only;          // tokens whose only destination is the source rank itself
    int status;                      // first data-dependent error seen while planning
};

// Running counts of the plans made on a context, kept on the device and advanced by the plan kernels themselves.
struct mw_plan_state {
    uint32_t plans;      // plans completed (the next plan's epoch is this + 1)
    uint32_t tickets;    // tile tickets handed out by all multi-kernel plans so far
    uint32_t bars;       // grid-barrier arrivals made by all fused plans so far
};

// Device workspace (all pointers into one slab owned by the context).
struct mw_dev {
    // public plan arrays (exposed through mw_plan_view)
    uint64_t *token_mask;
    int32_t *token_ndest, *token_group, *token_mw_row, *mw_row_token, *group_offsets;
    uint64_t *group_mask;
    int32_t *rank_offsets, *rank_tokens, *dest_rank, *dest_pos;
    mw_totals *totals;
    // internal plan arrays
    int32_t *token_slot;     // [Tm]      hash slot of the token's bitmap
    int32_t *token_leader;   // [Tm]      smallest token index with the same bitmap, -1 if empty
    int32_t *token_gcount;   // [Tm]      size of the token's group
    int32_t *gid_at;         // [Tm]      group id, stored at the leader's index
    int32_t *goff_at;        // [Tm]      group offset, stored at the leader's index
    int32_t *row_ndest;      // [Tm]      |D| of the token in MultiWrite send row j
    int32_t *row_dest_rank;  // [Kd, Tm]  destination ranks of send row j (entry i of row j at i * Tm + j)
    int32_t *row_dest_pos;   // [Kd, Tm]  slots of send row j
    int32_t *row_dest_flat;  // [Kd, Tm]  row of the compact receive area for each destination of send row j, -1 pad
    // group-major receive order (mw_order.cu)
    int32_t *gm_rank, *gm_offset;   // [Tm, Kd] destination ranks of group g / first slot of its block in each region
    int32_t *dest_pos_gm;           // [Tm, Kd] slot of token t in the region of its i-th destination, group-major order
    int32_t *row_dest_pos_gm;       // [Kd, Tm] the same per send row, plane layout
    int32_t *row_dest_flat_gm;      // [Kd, Tm] row of the compact receive area per send row and destination
    int32_t *gm_tile_sum;           // [max_tiles, R] rows each tile of 256 groups adds to each region
    unsigned long long *gm_tile_rec;   // [32, R] the same as (call number, value) records, for the one-kernel route
    int32_t *ex_tile_cnt;           // [max_tiles, E] tokens of each tile that selected each expert (nullptr: too large)
    // scratch
    unsigned long long *slot_key;                  // [HS] open-addressed table keyed by bitmap: (hash tag, first token)
    int32_t *slot_leader, *slot_count;             // [HS] smallest token index / number of tokens with that bitmap
    unsigned long long *tile_state;                // [max_tiles, NC] look-back records
    unsigned long long *tile_agg;                  // [max_tiles] (members << 32 | leaders) of each tile, fused plan
    unsigned int *ticket;                          // tile ticket counter
    unsigned int *gbar;                            // arrival counter of the fused plan's grid barriers
    unsigned int *copy_ctr;                        // [2] work-ticket and finished-warp counters of the copy kernels
    mw_acc *acc;                                   // [2]
    unsigned int *gave_up;                         // set by a plan whose wait gave up; later plans refuse to run until mw_reset
    mw_plan_state *plan_state;                     // running counts of the plans (epoch, tickets, barrier arrivals)
};

// What the data path needs to know about one plan: where its arrays are and what was planned into them.
struct mw_slot {
    mw_dev d;               // the slot's arrays (the scratch pointers are the same in both slots)
    int32_t planned_T;      // T of the plan held by the slot, -1 if none
    const void *prefetched; // rows that plan's launch brought into L2 (null: none)
    uint32_t plan_epoch;    // value of mw_ctx::epoch when that plan was issued
};

struct mw_ctx {
    mw_config cfg;
    int W, Kd, HS, NC, max_tiles;
    int sm_count;
    int max_smem_optin;
    int l2_bytes;
    // The current plan slot (the one mw_pack / mw_deliver / ... read), spelled out as members;
    // `other` is the second slot, which mw_plan_next fills while the current one is in use.
    mw_dev d;
    int32_t planned_T;      // T of the latest plan, -1 before the first
    const void *prefetched; // rows the latest plan launch brought into L2 (null: none)
    uint32_t plan_epoch;    // epoch of the current slot's plan
    mw_slot other;
    int next_pending;       // `other` holds a plan issued by mw_plan_next that mw_plan_swap has not taken yet
    cudaStream_t plan_stream;            // library-owned stream of mw_plan_next (highest priority, non-blocking)
    cudaEvent_t ev_submitted, ev_planned; // caller's stream -> plan stream; plan stream -> caller's stream
    int plans_on_side_stream;            // the latest plan launch went to plan_stream and ev_planned marks its end
    void *slab;
    size_t scratch_bytes;   // the part of the slab mw_reset re-initialises starts at scratch_begin
    uint8_t *scratch_begin;
    uint32_t epoch;         // plans issued so far: tells on the host which plan a slot holds (the kernels keep their own counts)
    int32_t spin_limit;     // polls a look-back waits for a predecessor's record before it gives up
    int32_t bar_spin_limit; // polls a block waits at a grid barrier
    int32_t copy_wait_limit;// polls (about 1 us each) the bulk-copy engine waits for a load
    uint32_t test_skew;     // MW_TEST_SKEW_* bits applied to the next launch (mw_test_skew_waits)
    int poisoned;           // a wait gave up: host counters and device scratch may be out of step until mw_reset
    uint32_t gm_epoch;      // epoch of the plan the group-major arrays were made from (0: none)
    uint32_t gm_calls;      // mw_group_major calls so far (tags the per-tile records of the one-kernel route)
    int32_t relay_src, relay_P;   // relay_P > 0: plans map every rank to its next hop as seen from rank relay_src (servers of relay_P ranks)
    int64_t launches;
    // host staging (MW_FLAG_HOST_STAGING)
    int32_t *st_ids, *st_e2r;
    uint8_t *st_x, *st_send, *st_recv;
    int64_t st_recv_rows;
};

// Next hop of a write from rank `src` to rank r when ranks form servers of P consecutive ranks: a destination in
// the source's own server is reached directly, any other through the rank with the source's index in its server.
__host__ __device__ inline int mw_next_hop(int r, int src, int P)
{
    return (r / P == src / P) ? r : (r / P) * P + src % P;
}

// Calls that use the device refuse a context in which a device-side wait has given up (see mw_reset).
#define MW_REFUSE_IF_POISONED(ctx) do { if ((ctx)->poisoned) return MW_ERR_TIMEOUT; } while (0)

// Ordinary launch; with `overlap` the kernel's blocks may be scheduled while the previous kernel of
// the stream drains (programmatic dependent launch).  Such a kernel must execute
// grid_dependency_wait() before it touches global memory that an earlier kernel reads or writes.
template <class... KArgs, class... Args>
inline cudaError_t mw_launch(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool overlap,
                             Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

#ifdef __CUDACC__
// Blocks until every kernel this launch depends on has completed and its writes are visible.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Allows the next kernel of the stream to start being scheduled.
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
// All ones if a == b, else zero.  Written as one opaque instruction on purpose: from `if ((r >> 6) == w) m[w] |= bit`
// with w a constant of an unrolled loop the compiler derives m[r >> 6], an array indexed by a run-time value,
// and moves the bitmap to local memory, where every read-modify-write costs a trip through the memory pipeline
// (measured on B200: 2.6 us for the eight expert ids of a token with four bitmap words, against 0.2 us from registers).
__device__ __forceinline__ uint64_t equal_mask64(int a, int b)
{
    uint32_t m;
    asm("set.eq.u32.s32 %0, %1, %2;" : "=r"(m) : "r"(a), "r"(b));
    return ((uint64_t)m << 32) | m;
}
// Hash step for the table keyed by bitmap (one call per 64-bit word): the golden-ratio combine followed by a
// 64-bit finaliser, both public-domain constants.
__device__ __forceinline__ uint64_t mix64(uint64_t h, uint64_t v)
{
    h ^= v + 0x9e3779b97f4a7c15ull + (h << 6) + (h >> 2);
    h ^= h >> 33; h *= 0xff51afd7ed558ccdull; h ^= h >> 29;
    return h;
}
// Word w of a bitmap held in registers.  Indexing the array with the variable of a loop that the compiler does
// not unroll (a loop over words around a loop over set bits) moves the whole array to local memory, and every
// access then costs a trip through the memory pipeline; a chain of selects keeps the words in registers.
template <int WT>
__device__ __forceinline__ uint64_t bitmap_word(const uint64_t (&m)[WT], int w)
{
    uint64_t v = m[0];
#pragma unroll
    for (int i = 1; i < WT; ++i) v = (w == i) ? m[i] : v;
    return v;
}
#endif

// ---- plan (mw_plan.cu) ----
// `rows` (may be null): the hidden rows [T, row_bytes] the pack step will read; they are brought into L2 while the plan runs
int mw_plan_launch(mw_ctx *ctx, const int32_t *topk_ids, const int32_t *expert_to_rank, int32_t T, const void *rows, cudaStream_t st);
int mw_plan_smem_setup(mw_ctx *ctx);
// Plans into the current slot on the context's own planning stream, ordered after everything submitted to `user`
// so far; the caller makes its stream wait for ctx->ev_planned before it uses the plan (mw_api.cu).
int mw_plan_on_side_stream(mw_ctx *ctx, const int32_t *topk_ids, const int32_t *expert_to_rank, int32_t T, cudaStream_t user);

// ---- single-launch small-batch path (mw_small.cu) ----
bool mw_small_applies(const mw_ctx *ctx, int32_t T, int layout);
int mw_small_setup(mw_ctx *ctx);
int mw_small_launch(mw_ctx *ctx, const int32_t *topk_ids, const int32_t *expert_to_rank, int32_t T, const void *x,
                    void *send_buf, int64_t send_capacity_rows, void *recv_base, int64_t recv_stride_bytes,
                    int64_t recv_capacity_rows, cudaStream_t st);

// ---- group-major order and expert index (mw_order.cu) ----
int mw_order_smem_setup(mw_ctx *ctx);

// ---- row copies (mw_copy.cu) ----
enum mw_copy_mode {
    MW_CP_PACK_MW = 0,      // send[j] = x[mw_row_token[j]]
    MW_CP_SCATTER = 1,      // dst(region, slot) = src[row] for every destination of the row
    MW_CP_DELIVER_UC = 2,   // region(r)[i] = send[rank_offsets[r] + i]
    MW_CP_AG_PACK_MW = 3,   // send[i] = shard[i]
    MW_CP_AG_DELIVER_MW = 4,// region(d)[i] = send[i] for every d of the window
    MW_CP_AG_PACK_UC = 5,   // send[i][d] = shard[i] for every d of the window except rank i itself
    MW_CP_AG_DELIVER_UC = 6,// region(d)[i] = send[i][d] (own shard: taken from shards)
    MW_CP_PAIR_DIRECT = 7,  // paired AllGather: direct segment of shard r to every member of r's domain
    MW_CP_PAIR_SEND = 8,    // relayed segment of shard r to its partner's relay area (and to r itself)
    MW_CP_PAIR_FORWARD = 9, // partner forwards the relayed segment to the other members of r's domain
    MW_CP_DISPATCH_MW = 10, // pack and deliver in one pass: x[mw_row_token[j]] -> send[j] and every destination of row j
    MW_CP_DISPATCH_UC = 11, // x[mw_row_token[j]] -> its unicast send slots and every destination of row j
    MW_CP_AG_FUSED_MW = 12, // AllGather pack and deliver in one pass: shard i -> send[i] and region(d)[i] for the window
    MW_CP_AG_FUSED_UC = 13  // shard i -> send[i][d] (d != i) and region(d)[i] for the window
};

struct mw_copy_args {
    int mode;
    const uint8_t *src;        // source rows (x, send buffer or shards)
    const uint8_t *src2;       // AllGather unicast deliver: the shards (own copy is local)
    uint8_t *dst;              // destination base
    uint8_t *const *dst_ptrs;  // deliver: device array [R] of region base addresses (then dst and dst_stride are unused), or null
    uint8_t *dst2;             // paired AllGather, relayed segment: the receive area (own copy), dst being the relay area;
                               // fused dispatch: the send buffer
    int64_t row_bytes;         // bytes per row (B, or the shard size)
    int64_t dst_stride;        // bytes between receive regions; 0 = compact
    int64_t capacity_rows;     // rows the destination may hold (per region when strided)
    int64_t capacity2_rows;    // fused dispatch: rows the send buffer (dst2) may hold
    int64_t host_rows;         // row count known on the host (-1: read from totals)
    int rows_from;             // 0: host_rows, 1: totals->T_nonempty, 2: totals->total_dest
    int32_t chunk_bytes;       // bytes moved per work item (multiple of 16)
    int32_t chunks_per_row;
    int stages;                // bulk-copy pipeline depth per warp
    int batch;                 // consecutive items claimed per work ticket
    int keep_in_l2;            // destination rows are read again soon: do not mark them evict-first
    int src_in_l2;             // fused dispatch: the source rows were prefetched into L2 by the plan launch
    int loose_bound;           // host_rows may be far above the row count: take the persistent grid, which pays nothing for absent rows
    int src_not_recent;        // SCATTER without a source index whose rows were not written by the launch just before
    int wait_limit;            // bulk-copy engine: polls (about 1 us each) before a wait for a load gives up
    int expect_extra;          // bulk-copy engine, test hook: bytes added to the announced size of every load
    unsigned int *work_ctr;    // [2] ticket counter, finished-warp counter (both zero between launches)
    int Kd, R, dst_begin, dst_count;
    int pair_n, pair_copies;   // paired AllGather: ranks per domain, copies of the relayed segment on the pair link
    int64_t shard_bytes, seg_off;   // paired AllGather: whole shard size, offset of the segment being moved
    const int32_t *src_index;  // PACK_MW: mw_row_token
    const int32_t *ndst;       // SCATTER: destinations per row
    const int32_t *d_rank;     // SCATTER: [Kd, d_stride] destination ranks, entry i of row j at i * d_stride + j
    const int32_t *d_pos;      // SCATTER: [Kd, d_stride] slots
    const int32_t *d_flat;     // SCATTER, compact destination: [Kd, d_stride] destination row, -1 pad
    int64_t d_stride;          // rows per descriptor plane (max_tokens)
    const int32_t *rank_offsets;
    mw_totals *totals;         // device accounting (row counts, status)
};

int mw_copy_launch(mw_ctx *ctx, mw_copy_args a, cudaStream_t st);
int mw_copy_smem_setup(mw_ctx *ctx);
