// Receiver-side layouts derived from the latest plan.  Declared in include/mw.h.
//
// Group-major receive order (paper, Section 4.3.1: MultiWrite(S, M, B_S) writes one source buffer into one
// target buffer B_i per destination; Section 4.3.2: the call takes an array of remote buffer addresses): the
// region of rank r is laid out group by group, so that group g is exactly one such call, from the contiguous
// slice send[group_offsets[g] ..) into one contiguous block per destination.  The block starts are a per-rank
// exclusive prefix sum, over groups in id order, of the sizes of the groups that contain the rank.
//
// Expert index (Section 2.3.2: a token goes to the nodes hosting its experts): per expert, the ascending list
// of its tokens and of their slots in the region of the expert's rank.  A per-expert exclusive prefix sum over
// tokens, done as a bit matrix (expert x token of the tile) plus per-tile counts.
//
// Both are small integer passes over the plan (kilobytes to a few megabytes); they run as a few short kernels
// of one block per 256 groups / tokens and are bound by launch and memory latency, not by bandwidth.
#include <string.h>

#include "mw_internal.cuh"

namespace {

constexpr int kTile = MW_TILE;

__device__ __forceinline__ bool bit_of(const uint64_t *mask, int r) { return (mask[r >> 6] >> (r & 63)) & 1ull; }

struct GmArgs {
    mw_dev d;
    int R, W, Kd, Tm, T;
    int tiles;                 // tiles launched (covers every possible G)
};

// Per tile of 256 groups and per rank: rows the tile's groups add to the rank's region.
__global__ void __launch_bounds__(kTile) k_gm_sum(GmArgs a)
{
    extern __shared__ uint64_t sm64[];
    uint64_t *mask = sm64;                          // [kTile, W]
    int *size = (int *)(mask + (size_t)kTile * a.W);  // [kTile]
    if (a.d.totals->status == MW_ERR_TIMEOUT) return;
    const int G = (int)a.d.totals->G;
    const int g0 = blockIdx.x * kTile;
    const int n = min(kTile, G - g0);
    if (n <= 0) {
        for (int r = threadIdx.x; r < a.R; r += kTile) a.d.gm_tile_sum[(size_t)blockIdx.x * a.R + r] = 0;
        return;
    }
    for (int i = threadIdx.x; i < n * a.W; i += kTile) mask[i] = a.d.group_mask[(size_t)g0 * a.W + i];
    if (threadIdx.x < n) size[threadIdx.x] = a.d.group_offsets[g0 + threadIdx.x + 1] - a.d.group_offsets[g0 + threadIdx.x];
    __syncthreads();
    // one warp per rank; lane l covers groups [8 l, 8 l + 8) of the tile
    const int lane = threadIdx.x & 31;
    for (int r = threadIdx.x >> 5; r < a.R; r += kTile / 32) {
        int sum = 0;
        for (int j = lane * 8; j < min(lane * 8 + 8, n); ++j)
            if (bit_of(mask + (size_t)j * a.W, r)) sum += size[j];
        sum = __reduce_add_sync(0xffffffffu, sum);
        if (lane == 0) a.d.gm_tile_sum[(size_t)blockIdx.x * a.R + r] = sum;
    }
}

// Exclusive prefix over the tiles, per rank, in place (one thread per rank; tiles are few).
__global__ void __launch_bounds__(kTile) k_gm_scan(GmArgs a)
{
    const int r = blockIdx.x * kTile + threadIdx.x;
    if (r >= a.R) return;
    int run = 0;
    for (int t = 0; t < a.tiles; ++t) {
        const int v = a.d.gm_tile_sum[(size_t)t * a.R + r];
        a.d.gm_tile_sum[(size_t)t * a.R + r] = run;
        run += v;
    }
}

// Per tile: the warp of rank r walks the tile's groups in order and hands every group that contains r its block.
__global__ void __launch_bounds__(kTile) k_gm_fill(GmArgs a)
{
    extern __shared__ uint64_t sm64[];
    uint64_t *mask = sm64;
    int *size = (int *)(mask + (size_t)kTile * a.W);
    if (a.d.totals->status == MW_ERR_TIMEOUT) return;
    const int G = (int)a.d.totals->G;
    const int g0 = blockIdx.x * kTile;
    const int n = min(kTile, G - g0);
    if (n <= 0) return;
    for (int i = threadIdx.x; i < n * a.W; i += kTile) mask[i] = a.d.group_mask[(size_t)g0 * a.W + i];
    if (threadIdx.x < n) {
        size[threadIdx.x] = a.d.group_offsets[g0 + threadIdx.x + 1] - a.d.group_offsets[g0 + threadIdx.x];
        for (int i = 0; i < a.Kd; ++i) {
            a.d.gm_rank[(size_t)(g0 + threadIdx.x) * a.Kd + i] = -1;
            a.d.gm_offset[(size_t)(g0 + threadIdx.x) * a.Kd + i] = -1;
        }
    }
    __syncthreads();
    // one warp per rank; lane l covers groups [8 l, 8 l + 8): an exclusive scan over the lanes gives each its start
    const int lane = threadIdx.x & 31;
    for (int r = threadIdx.x >> 5; r < a.R; r += kTile / 32) {
        int sum = 0;
        for (int j = lane * 8; j < min(lane * 8 + 8, n); ++j)
            if (bit_of(mask + (size_t)j * a.W, r)) sum += size[j];
        int incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int v = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += v; }
        int run = a.d.gm_tile_sum[(size_t)blockIdx.x * a.R + r] + incl - sum;
        for (int j = lane * 8; j < min(lane * 8 + 8, n); ++j) {
            const uint64_t *m = mask + (size_t)j * a.W;
            if (!bit_of(m, r)) continue;
            int i = __popcll(m[r >> 6] & ((1ull << (r & 63)) - 1));      // index of r among the group's destinations
            for (int w = 0; w < (r >> 6); ++w) i += __popcll(m[w]);
            a.d.gm_rank[(size_t)(g0 + j) * a.Kd + i] = r;
            a.d.gm_offset[(size_t)(g0 + j) * a.Kd + i] = run;
            run += size[j];
        }
    }
}

// Per token: its slots in group-major order, and the same per send row in plane layout for the deliver kernel.
__global__ void __launch_bounds__(kTile) k_gm_tokens(GmArgs a)
{
    if (a.d.totals->status == MW_ERR_TIMEOUT) return;
    const int t = blockIdx.x * kTile + threadIdx.x;
    if (t >= a.T) return;
    const int g = a.d.token_group[t];
    const int row = a.d.token_mw_row[t];
    const int within = g >= 0 ? row - a.d.group_offsets[g] : 0;
    for (int i = 0; i < a.Kd; ++i) {
        const int r = g >= 0 ? a.d.gm_rank[(size_t)g * a.Kd + i] : -1;
        const int pos = r >= 0 ? a.d.gm_offset[(size_t)g * a.Kd + i] + within : -1;
        a.d.dest_pos_gm[(size_t)t * a.Kd + i] = pos;
        if (g >= 0) {
            a.d.row_dest_pos_gm[(size_t)i * a.Tm + row] = pos;
            a.d.row_dest_flat_gm[(size_t)i * a.Tm + row] = r >= 0 ? a.d.rank_offsets[r] + pos : -1;
        }
    }
}

// ---- expert index -----------------------------------------------------------------------------------
struct ExArgs {
    mw_dev d;
    const int32_t *ids, *e2r;
    int32_t *offsets, *token, *slot;
    int T, K, E, R, Kd, tiles;
};

// bits[e * 8 + w]: which tokens of warp w of this tile selected expert e (valid expert on a valid rank)
__device__ __forceinline__ void expert_bits(const ExArgs &a, uint32_t *bits, int t)
{
    for (int i = threadIdx.x; i < a.E * 8; i += kTile) bits[i] = 0;
    __syncthreads();
    if (t < a.T) {
        for (int k = 0; k < a.K; ++k) {
            const int e = a.ids[(size_t)t * a.K + k];
            if (e < 0 || e >= a.E) continue;
            const int r = a.e2r[e];
            if (r < 0 || r >= a.R) continue;
            atomicOr(bits + (size_t)e * 8 + (threadIdx.x >> 5), 1u << (threadIdx.x & 31));
        }
    }
    __syncthreads();
}

__global__ void __launch_bounds__(kTile) k_ex_count(ExArgs a)
{
    extern __shared__ uint32_t sm32[];
    expert_bits(a, sm32, blockIdx.x * kTile + threadIdx.x);
    for (int e = threadIdx.x; e < a.E; e += kTile) {
        int c = 0;
#pragma unroll
        for (int w = 0; w < 8; ++w) c += __popc(sm32[(size_t)e * 8 + w]);
        a.d.ex_tile_cnt[(size_t)blockIdx.x * a.E + e] = c;
    }
}

// One block: per expert the exclusive prefix over the tiles (in place), then the exclusive prefix over experts.
__global__ void __launch_bounds__(1024) k_ex_scan(ExArgs a)
{
    __shared__ int warp_tot[32];
    __shared__ int carry_s;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    for (int e0 = 0; e0 < a.E; e0 += 1024) {
        const int e = e0 + threadIdx.x;
        int total = 0;
        if (e < a.E) {
            for (int t = 0; t < a.tiles; ++t) {
                const int v = a.d.ex_tile_cnt[(size_t)t * a.E + e];
                a.d.ex_tile_cnt[(size_t)t * a.E + e] = total;
                total += v;
            }
        }
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        int incl = total;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int n = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += n; }
        if (lane == 31) warp_tot[warp] = incl;
        __syncthreads();
        int before = carry_s, all = 0;
        for (int w = 0; w < 32; ++w) { if (w < warp) before += warp_tot[w]; all += warp_tot[w]; }
        if (e < a.E) a.offsets[e] = before + incl - total;
        __syncthreads();
        if (threadIdx.x == 0) carry_s += all;
        __syncthreads();
    }
    if (threadIdx.x == 0) a.offsets[a.E] = carry_s;
}

__global__ void __launch_bounds__(kTile) k_ex_fill(ExArgs a)
{
    extern __shared__ uint32_t sm32[];
    const int t = blockIdx.x * kTile + threadIdx.x;
    expert_bits(a, sm32, t);
    const int P = a.offsets[a.E];
    // tails: every index of the two lists at or beyond P is covered by some thread of the grid
    for (int64_t i = (int64_t)blockIdx.x * kTile + threadIdx.x; i < (int64_t)a.T * a.K; i += (int64_t)gridDim.x * kTile)
        if (i >= P) { a.token[i] = -1; a.slot[i] = -1; }
    if (t >= a.T) return;
    const int warp = threadIdx.x >> 5;
    const uint32_t below = (1u << (threadIdx.x & 31)) - 1;
    for (int k = 0; k < a.K; ++k) {
        const int e = a.ids[(size_t)t * a.K + k];
        if (e < 0 || e >= a.E) continue;
        const int r = a.e2r[e];
        if (r < 0 || r >= a.R) continue;
        bool first = true;                                     // an expert named twice by a token counts once
        for (int j = 0; j < k; ++j) first &= (a.ids[(size_t)t * a.K + j] != e);
        if (!first) continue;
        int pos = a.offsets[e] + a.d.ex_tile_cnt[(size_t)blockIdx.x * a.E + e];
        for (int w = 0; w < warp; ++w) pos += __popc(sm32[(size_t)e * 8 + w]);
        pos += __popc(sm32[(size_t)e * 8 + warp] & below);
        int slot = -1;
        for (int i = 0; i < a.Kd; ++i)
            if (a.d.dest_rank[(size_t)t * a.Kd + i] == r) slot = a.d.dest_pos[(size_t)t * a.Kd + i];
        a.token[pos] = t;
        a.slot[pos] = slot;
    }
}

size_t gm_smem(const mw_ctx *ctx) { return (size_t)kTile * ctx->W * 8 + (size_t)kTile * 4; }
size_t ex_smem(const mw_ctx *ctx) { return (size_t)ctx->cfg.E * 32; }

}  // namespace

int mw_order_smem_setup(mw_ctx *ctx)
{
    const size_t ex = ex_smem(ctx);
    if (ex > 48 * 1024 && ex + 1024 <= (size_t)ctx->max_smem_optin) {
        if (cudaFuncSetAttribute(k_ex_count, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ex) != cudaSuccess ||
            cudaFuncSetAttribute(k_ex_fill, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ex) != cudaSuccess)
            return MW_ERR_CUDA;
    }
    return MW_OK;
}

extern "C" int mw_group_major(mw_ctx *ctx, mw_group_major_view *view, void *stream)
{
    if (!ctx) return MW_ERR_INVALID_ARG;
    MW_REFUSE_IF_POISONED(ctx);
    if (ctx->planned_T < 0) return MW_ERR_NO_PLAN;
    if (view) {
        view->group_dest_rank = ctx->d.gm_rank; view->group_dest_offset = ctx->d.gm_offset;
        view->dest_pos_gm = ctx->d.dest_pos_gm; view->Kd = ctx->Kd; view->reserved = 0;
    }
    ctx->gm_epoch = ctx->plan_epoch;
    const int T = ctx->planned_T;
    if (T == 0) return MW_OK;
    GmArgs a;
    a.d = ctx->d; a.R = ctx->cfg.R; a.W = ctx->W; a.Kd = ctx->Kd; a.Tm = ctx->cfg.max_tokens; a.T = T;
    a.tiles = (T + kTile - 1) / kTile;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t smem = gm_smem(ctx);
    k_gm_sum<<<a.tiles, kTile, smem, st>>>(a);
    k_gm_scan<<<(a.R + kTile - 1) / kTile, kTile, 0, st>>>(a);
    k_gm_fill<<<a.tiles, kTile, smem, st>>>(a);
    k_gm_tokens<<<a.tiles, kTile, 0, st>>>(a);
    ctx->launches += 4;
    return cudaGetLastError() == cudaSuccess ? MW_OK : MW_ERR_CUDA;
}

extern "C" int mw_deliver_group_major(mw_ctx *ctx, const void *send_buf, void *recv_base, int64_t recv_stride_bytes,
                                      int64_t recv_capacity_rows, void *stream)
{
    if (!ctx || !send_buf || !recv_base || recv_stride_bytes < 0 || recv_capacity_rows < 0) return MW_ERR_INVALID_ARG;
    MW_REFUSE_IF_POISONED(ctx);
    if (ctx->planned_T < 0 || ctx->gm_epoch != ctx->plan_epoch) return MW_ERR_NO_PLAN;
    if (((uintptr_t)send_buf & 15u) || ((uintptr_t)recv_base & 15u) || recv_stride_bytes % 16) return MW_ERR_ALIGNMENT;
    if (recv_stride_bytes && recv_capacity_rows * ctx->cfg.row_bytes > recv_stride_bytes) return MW_ERR_CAPACITY;
    mw_copy_args a;
    memset(&a, 0, sizeof(a));
    a.mode = MW_CP_SCATTER;
    a.src = (const uint8_t *)send_buf;
    a.dst = (uint8_t *)recv_base;
    a.row_bytes = ctx->cfg.row_bytes;
    a.dst_stride = recv_stride_bytes;
    a.capacity_rows = recv_capacity_rows;
    a.rows_from = 1;
    a.host_rows = ctx->planned_T;
    a.Kd = ctx->Kd; a.R = ctx->cfg.R;
    a.ndst = ctx->d.row_ndest;
    a.d_rank = ctx->d.row_dest_rank;            // the destination ranks do not depend on the order
    a.d_pos = ctx->d.row_dest_pos_gm;
    a.d_flat = ctx->d.row_dest_flat_gm;
    a.d_stride = ctx->cfg.max_tokens;
    a.rank_offsets = ctx->d.rank_offsets;
    a.totals = ctx->d.totals;
    return mw_copy_launch(ctx, a, (cudaStream_t)stream);
}

extern "C" int mw_expert_index(mw_ctx *ctx, const int32_t *topk_ids, const int32_t *expert_to_rank, int32_t *expert_offsets,
                               int32_t *expert_token, int32_t *expert_slot, void *stream)
{
    if (!ctx || !expert_to_rank || !expert_offsets || !expert_token || !expert_slot) return MW_ERR_INVALID_ARG;
    MW_REFUSE_IF_POISONED(ctx);
    if (ctx->planned_T < 0) return MW_ERR_NO_PLAN;
    const int T = ctx->planned_T;
    if (T > 0 && !topk_ids) return MW_ERR_INVALID_ARG;
    if (!ctx->d.ex_tile_cnt || ex_smem(ctx) + 1024 > (size_t)ctx->max_smem_optin) return MW_ERR_CAPACITY;
    ExArgs a;
    a.d = ctx->d; a.ids = topk_ids; a.e2r = expert_to_rank;
    a.offsets = expert_offsets; a.token = expert_token; a.slot = expert_slot;
    a.T = T; a.K = ctx->cfg.K; a.E = ctx->cfg.E; a.R = ctx->cfg.R; a.Kd = ctx->Kd;
    a.tiles = (T + kTile - 1) / kTile;
    cudaStream_t st = (cudaStream_t)stream;
    if (T > 0) k_ex_count<<<a.tiles, kTile, ex_smem(ctx), st>>>(a);
    k_ex_scan<<<1, 1024, 0, st>>>(a);
    if (T > 0) k_ex_fill<<<a.tiles, kTile, ex_smem(ctx), st>>>(a);
    ctx->launches += T > 0 ? 3 : 1;
    return cudaGetLastError() == cudaSuccess ? MW_OK : MW_ERR_CUDA;
}
