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
// Both are small integer passes over the plan (kilobytes to a few megabytes), bound by launch and memory latency,
// not by bandwidth.  Up to 32 tiles of 256 groups / tokens the group-major arrays take one kernel (every tile publishes
// its per-rank sums and adds up those of the tiles before it) and the expert index two (per-tile counts, then everything
// else, every block summing the earlier tiles' counts by itself); beyond that, a scan kernel sits in between.
#include <string.h>

#include "mw_internal.cuh"

namespace {

constexpr int kTile = MW_TILE;

__device__ __forceinline__ bool bit_of(const uint64_t *mask, int r) { return (mask[r >> 6] >> (r & 63)) & 1ull; }

struct GmArgs {
    mw_dev d;
    int R, W, Kd, Tm, T;
    int tiles;                 // tiles launched (covers every possible G)
    int stash;                 // k_gm_fill keeps the tile's (rank, block start) rows in shared memory as well (Kd <= 16)
    uint32_t call;             // number of this mw_group_major call on the context (tags the per-tile records, never 0)
    uint32_t wait_call;        // tag a tile expects in the records of the tiles before it (= call, unless a test skews it)
    int spin_limit;            // polls before a tile gives up waiting for an earlier tile's record
};

// Per tile of 256 groups and per rank: rows the tile's groups add to the rank's region.
__global__ void __launch_bounds__(kTile) k_gm_sum(GmArgs a)
{
    extern __shared__ uint64_t sm64[];
    uint64_t *mask = sm64;                          // [kTile, W]
    int *size = (int *)(mask + (size_t)kTile * a.W);  // [kTile]
    const int status = a.d.totals->status, G = (int)a.d.totals->G;      // both before the first branch: one round trip
    if (status == MW_ERR_TIMEOUT) return;
    const int g0 = blockIdx.x * kTile;
    const int n = min(kTile, G - g0);
    if (n <= 0) {
        for (int r = threadIdx.x; r < a.R; r += kTile) a.d.gm_tile_sum[(size_t)blockIdx.x * a.R + r] = 0;
        return;
    }
    for (int i = threadIdx.x; i < n * a.W; i += kTile) mask[i] = a.d.group_mask[(size_t)g0 * a.W + i];
    if (threadIdx.x < n) size[threadIdx.x] = a.d.group_offsets[g0 + threadIdx.x + 1] - a.d.group_offsets[g0 + threadIdx.x];
    __syncthreads();
    // one warp per rank; lane l covers groups l, l + 32, ... of the tile (neighbouring lanes read neighbouring bitmaps:
    // with eight consecutive groups per lane the shared-memory reads of a warp fell into two banks)
    const int lane = threadIdx.x & 31;
    for (int r = threadIdx.x >> 5; r < a.R; r += kTile / 32) {
        int sum = 0;
        for (int j = lane; j < n; j += 32)
            if (bit_of(mask + (size_t)j * a.W, r)) sum += size[j];
        sum = __reduce_add_sync(0xffffffffu, sum);
        if (lane == 0) a.d.gm_tile_sum[(size_t)blockIdx.x * a.R + r] = sum;
    }
}

// Exclusive prefix over the tiles, per rank, in place (one thread per rank; tiles are few).
__global__ void __launch_bounds__(kTile) k_gm_scan(GmArgs a)
{
    grid_launch_dependents();
    const int r = blockIdx.x * kTile + threadIdx.x;
    if (r >= a.R) return;
    int run = 0;
    for (int t = 0; t < a.tiles; ++t) {
        const int v = a.d.gm_tile_sum[(size_t)t * a.R + r];
        a.d.gm_tile_sum[(size_t)t * a.R + r] = run;
        run += v;
    }
}

constexpr int kFillThreads = 1024;  // k_gm_fill: 32 warps share the ranks of the tile (the per-rank walk is a chain of warp scans)
constexpr int kFuseTiles = 32;     // up to this many tiles every block adds up the earlier tiles' counts itself

// Per tile of 256 groups: the warp of rank r walks the tile's groups in order and hands every group that contains r
// its block of the region; then the block's threads take the send rows of those groups (they are consecutive) and
// give every member token its slots, per token and per send row (plane layout, for the deliver kernel).
// SCANNED: gm_tile_sum already holds the exclusive prefix over tiles (k_gm_sum and k_gm_scan ran before).  Otherwise
// this is the only kernel: every tile first publishes its own per-rank sums as one 64-bit record each (call number,
// value), then adds up the records of the tiles before it, waiting (with a limit) for those not yet there; a tile
// only waits for tiles with a smaller block index, and at most kFuseTiles blocks exist, all resident.
// The block with index b also marks the tokens [256 b, 256 b + 256) that have no destination.
template <bool SCANNED>
__global__ void __launch_bounds__(kFillThreads) k_gm_fill(GmArgs a)
{
    extern __shared__ uint64_t sm64[];
    uint64_t *mask = sm64;
    int *size = (int *)(mask + (size_t)kTile * a.W);
    int *before_s = size + kTile;                         // [R]
    int *region_s = before_s + a.R;                       // [R + 1] region starts of the plan
    int *rank_s = region_s + a.R + 1;                     // [kTile, Kd] (stash) destination ranks of the tile's groups
    int *start_s = rank_s + (a.stash ? kTile * a.Kd : 0); // [kTile, Kd] (stash) start of each group's block in that region
    __shared__ int gstart[kTile + 1];
    if (!SCANNED) grid_dependency_wait();    // launched as a programmatic dependent: only its start-up overlaps the kernel before it
    if (a.d.totals->status == MW_ERR_TIMEOUT) return;
    {   // tokens without destinations belong to no group: their slots are -1
        const int t = blockIdx.x * kTile + threadIdx.x;
        if (threadIdx.x < kTile && t < a.T && a.d.token_group[t] < 0)
            for (int i = 0; i < a.Kd; ++i) a.d.dest_pos_gm[(size_t)t * a.Kd + i] = -1;
    }
    const int G = (int)a.d.totals->G;
    const int g0 = blockIdx.x * kTile;
    const int n = min(kTile, G - g0);
    if (n <= 0) return;
    for (int i = threadIdx.x; i < n * a.W; i += kFillThreads) mask[i] = a.d.group_mask[(size_t)g0 * a.W + i];
    if (threadIdx.x < n) gstart[threadIdx.x] = a.d.group_offsets[g0 + threadIdx.x];
    if (threadIdx.x == 0) gstart[n] = a.d.group_offsets[g0 + n];
    __syncthreads();
    for (int r = threadIdx.x; r <= a.R; r += kFillThreads) region_s[r] = a.d.rank_offsets[r];
    // the token of this thread's first send row (the member-token part below starts with it)
    const int first_row = gstart[0] + threadIdx.x;
    const int first_token = first_row < gstart[n] ? a.d.mw_row_token[first_row] : -1;
    if (threadIdx.x < n) {
        size[threadIdx.x] = gstart[threadIdx.x + 1] - gstart[threadIdx.x];
        for (int i = 0; i < a.Kd; ++i) {
            a.d.gm_rank[(size_t)(g0 + threadIdx.x) * a.Kd + i] = -1;
            a.d.gm_offset[(size_t)(g0 + threadIdx.x) * a.Kd + i] = -1;
            if (a.stash) rank_s[threadIdx.x * a.Kd + i] = -1;
        }
    }
    const int lane = threadIdx.x & 31;
    if (SCANNED) {
        // Everything above needs the plan only and has run while the scan of the per-tile sums was still at work.
        grid_dependency_wait();
        for (int r = threadIdx.x; r < a.R; r += kFillThreads) before_s[r] = a.d.gm_tile_sum[(size_t)blockIdx.x * a.R + r];
    } else {
        __syncthreads();                                  // bitmaps and sizes are in shared memory
        // this tile's rows per region: one warp per rank, lanes stride the groups; published at once
        for (int r = threadIdx.x >> 5; r < a.R; r += kFillThreads / 32) {
            int sum = 0;
            for (int j = lane; j < n; j += 32)
                if (bit_of(mask + (size_t)j * a.W, r)) sum += size[j];
            sum = __reduce_add_sync(0xffffffffu, sum);
            if (lane == 0)
                *(volatile unsigned long long *)(a.d.gm_tile_rec + (size_t)blockIdx.x * a.R + r) =
                    ((unsigned long long)a.call << 32) | (uint32_t)sum;
        }
        // rows the earlier tiles put into every region: all ranks at once, eight records per round trip
        for (int r = threadIdx.x; r < a.R; r += kFillThreads) {
            int before = 0;
            bool gave_up = false;
            for (int t0 = 0; t0 < (int)blockIdx.x && !gave_up; t0 += 8) {
                unsigned long long v[8];
#pragma unroll
                for (int u = 0; u < 8; ++u)
                    v[u] = t0 + u < (int)blockIdx.x ? *(volatile unsigned long long *)(a.d.gm_tile_rec + (size_t)(t0 + u) * a.R + r)
                                                    : ((unsigned long long)a.wait_call << 32);
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    int spins = 0;
                    while ((uint32_t)(v[u] >> 32) != a.wait_call) {           // not this call's record yet
                        if (++spins > a.spin_limit) { gave_up = true; break; }
                        __nanosleep(64);
                        v[u] = *(volatile unsigned long long *)(a.d.gm_tile_rec + (size_t)(t0 + u) * a.R + r);
                    }
                    before += (int)(uint32_t)v[u];
                }
            }
            if (gave_up) atomicCAS(&a.d.totals->status, 0, MW_ERR_TIMEOUT);
            before_s[r] = before;
        }
    }
    __syncthreads();
    // one warp per rank, 32 groups of the tile per round (lane l takes group 32 k + l, so neighbouring lanes read
    // neighbouring bitmaps): an exclusive scan over the lanes gives each group that contains r the start of its block
    for (int r = threadIdx.x >> 5; r < a.R; r += kFillThreads / 32) {
        int run = before_s[r];
        for (int j0 = 0; j0 < n; j0 += 32) {
            const int j = j0 + lane;
            const uint64_t *m = mask + (size_t)j * a.W;
            const bool has = j < n && bit_of(m, r);
            const int mine = has ? size[j] : 0;
            int incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const int v = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += v; }
            if (has) {
                int i = __popcll(m[r >> 6] & ((1ull << (r & 63)) - 1));  // index of r among the group's destinations
                for (int w = 0; w < (r >> 6); ++w) i += __popcll(m[w]);
                a.d.gm_rank[(size_t)(g0 + j) * a.Kd + i] = r;
                a.d.gm_offset[(size_t)(g0 + j) * a.Kd + i] = run + incl - mine;
                if (a.stash) { rank_s[j * a.Kd + i] = r; start_s[j * a.Kd + i] = run + incl - mine; }
            }
            run += __shfl_sync(0xffffffffu, incl, 31);
        }
    }
    __syncthreads();                                      // the tile's gm_rank / gm_offset rows are complete (and visible to the block)
    // member tokens: send rows [gstart[0], gstart[n]) belong to the tile's groups, in group order
    for (int row = gstart[0] + threadIdx.x; row < gstart[n]; row += kFillThreads) {
        int lo = 0, hi = n;                               // group of the row: the last j with gstart[j] <= row
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (gstart[mid] <= row) lo = mid; else hi = mid;
        }
        const int g = g0 + lo, within = row - gstart[lo];
        const int t = row == first_row ? first_token : a.d.mw_row_token[row];
        // eight destinations at a time: all loads first, then the stores (a store in between would hold the next loads back,
        // since the compiler must assume that the arrays overlap)
        for (int i0 = 0; i0 < a.Kd; i0 += 8) {
            int r[8], pos[8], region[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const bool in = i0 + u < a.Kd;
                r[u] = !in ? -1 : a.stash ? rank_s[lo * a.Kd + i0 + u] : a.d.gm_rank[(size_t)g * a.Kd + i0 + u];
                pos[u] = (!in || r[u] < 0) ? -1 : a.stash ? start_s[lo * a.Kd + i0 + u] : a.d.gm_offset[(size_t)g * a.Kd + i0 + u];
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) region[u] = r[u] >= 0 ? region_s[r[u]] : 0;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                if (i0 + u >= a.Kd) break;
                const int p = r[u] >= 0 ? pos[u] + within : -1;
                a.d.dest_pos_gm[(size_t)t * a.Kd + i0 + u] = p;
                a.d.row_dest_pos_gm[(size_t)(i0 + u) * a.Tm + row] = p;
                a.d.row_dest_flat_gm[(size_t)(i0 + u) * a.Tm + row] = r[u] >= 0 ? region[u] + p : -1;
            }
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
        for (int k0 = 0; k0 < a.K; k0 += 8) {                  // eight independent loads at a time, twice
            int e[8], r[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) e[u] = k0 + u < a.K ? a.ids[(size_t)t * a.K + k0 + u] : -1;
#pragma unroll
            for (int u = 0; u < 8; ++u) r[u] = (e[u] >= 0 && e[u] < a.E) ? a.e2r[e[u]] : -1;
#pragma unroll
            for (int u = 0; u < 8; ++u)
                if (r[u] >= 0 && r[u] < a.R) atomicOr(bits + (size_t)e[u] * 8 + (threadIdx.x >> 5), 1u << (threadIdx.x & 31));
        }
    }
    __syncthreads();
}

__global__ void __launch_bounds__(kTile) k_ex_count(ExArgs a)
{
    extern __shared__ uint32_t sm32[];
    grid_launch_dependents();      // k_ex_fill may build its bit matrix meanwhile
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
    grid_launch_dependents();
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

// FUSED: ex_tile_cnt holds the raw per-tile counts; every block adds up the tiles before it and scans the experts
// itself (block 0 also writes expert_offsets).  Otherwise k_ex_scan has already done both.
template <bool FUSED>
__global__ void __launch_bounds__(kTile) k_ex_fill(ExArgs a)
{
    extern __shared__ uint32_t sm32[];
    __shared__ int warp_tot[kTile / 32];
    __shared__ int carry_s;
    int *start = (int *)(sm32 + (size_t)a.E * 8);          // [E] (FUSED) first list position of this tile's tokens per expert
    const int t = blockIdx.x * kTile + threadIdx.x;
    expert_bits(a, sm32, t);
    grid_dependency_wait();        // the counts of the kernel before this one are needed from here on
    int P;
    if (FUSED) {
        if (threadIdx.x == 0) carry_s = 0;
        __syncthreads();
        for (int e0 = 0; e0 < a.E; e0 += kTile) {
            const int e = e0 + threadIdx.x;
            int total = 0, before = 0;
            if (e < a.E)
                for (int b = 0; b < a.tiles; ++b) {
                    const int v = a.d.ex_tile_cnt[(size_t)b * a.E + e];
                    if (b < (int)blockIdx.x) before += v;
                    total += v;
                }
            const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
            int incl = total;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const int n = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += n; }
            if (lane == 31) warp_tot[warp] = incl;
            __syncthreads();
            int excl = carry_s + incl - total, all = 0;
            for (int w = 0; w < kTile / 32; ++w) { if (w < warp) excl += warp_tot[w]; all += warp_tot[w]; }
            if (e < a.E) {
                start[e] = excl + before;
                if (blockIdx.x == 0) a.offsets[e] = excl;
            }
            __syncthreads();
            if (threadIdx.x == 0) carry_s += all;
            __syncthreads();
        }
        P = carry_s;
        if (blockIdx.x == 0 && threadIdx.x == 0) a.offsets[a.E] = P;
    } else {
        P = a.offsets[a.E];
    }
    // tails: every index of the two lists at or beyond P is covered by some thread of the grid
    for (int64_t i = (int64_t)blockIdx.x * kTile + threadIdx.x; i < (int64_t)a.T * a.K; i += (int64_t)gridDim.x * kTile)
        if (i >= P) { a.token[i] = -1; a.slot[i] = -1; }
    if (t >= a.T) return;
    const int warp = threadIdx.x >> 5;
    const uint32_t below = (1u << (threadIdx.x & 31)) - 1;
    // eight expert slots at a time: all loads first, then the stores (see k_gm_fill)
    for (int k0 = 0; k0 < a.K; k0 += 8) {
        int e[8], r[8], slot[8];
        bool use[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) e[u] = k0 + u < a.K ? a.ids[(size_t)t * a.K + k0 + u] : -1;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const bool ok = e[u] >= 0 && e[u] < a.E;
            r[u] = ok ? a.e2r[e[u]] : -1;
            use[u] = ok;
            slot[u] = -1;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) use[u] = use[u] && r[u] >= 0 && r[u] < a.R;
        for (int j = 0; j < k0 + 7 && j < a.K; ++j) {          // an expert named twice by a token counts once (the first time)
            const int ej = a.ids[(size_t)t * a.K + j];
#pragma unroll
            for (int u = 0; u < 8; ++u) use[u] = use[u] && !(j < k0 + u && ej == e[u]);
        }
#pragma unroll 4
        for (int i = 0; i < a.Kd; ++i) {
            const int dr = a.d.dest_rank[(size_t)t * a.Kd + i], dp = a.d.dest_pos[(size_t)t * a.Kd + i];
#pragma unroll
            for (int u = 0; u < 8; ++u) slot[u] = (use[u] && dr == r[u]) ? dp : slot[u];
        }
        int pos[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            pos[u] = 0;
            if (!use[u]) continue;
            pos[u] = FUSED ? start[e[u]] : a.offsets[e[u]] + a.d.ex_tile_cnt[(size_t)blockIdx.x * a.E + e[u]];
            for (int w = 0; w < warp; ++w) pos[u] += __popc(sm32[(size_t)e[u] * 8 + w]);
            pos[u] += __popc(sm32[(size_t)e[u] * 8 + warp] & below);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (use[u]) { a.token[pos[u]] = t; a.slot[pos[u]] = slot[u]; }
    }
}

bool gm_stash(const mw_ctx *ctx) { return ctx->Kd <= 16; }
size_t gm_smem(const mw_ctx *ctx)
{
    return (size_t)kTile * ctx->W * 8 + (size_t)kTile * 4 + ((size_t)2 * ctx->cfg.R + 1) * 4 +
           (gm_stash(ctx) ? (size_t)2 * kTile * ctx->Kd * 4 : 0);
}
size_t ex_smem(const mw_ctx *ctx) { return (size_t)ctx->cfg.E * 36; }     // bit matrix (32 bytes per expert) + one list position

}  // namespace

int mw_order_smem_setup(mw_ctx *ctx)
{
    const size_t gm = gm_smem(ctx);
    if (gm > 48 * 1024) {
        if (gm > (size_t)ctx->max_smem_optin) return MW_ERR_INVALID_ARG;
        if (cudaFuncSetAttribute(k_gm_sum, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gm) != cudaSuccess ||
            cudaFuncSetAttribute(k_gm_fill<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gm) != cudaSuccess ||
            cudaFuncSetAttribute(k_gm_fill<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gm) != cudaSuccess)
            return MW_ERR_CUDA;
    }
    const size_t ex = ex_smem(ctx);
    if (ex > 48 * 1024 && ex + 1024 <= (size_t)ctx->max_smem_optin) {
        if (cudaFuncSetAttribute(k_ex_count, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ex) != cudaSuccess ||
            cudaFuncSetAttribute(k_ex_fill<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ex) != cudaSuccess ||
            cudaFuncSetAttribute(k_ex_fill<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ex) != cudaSuccess)
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
    a.stash = gm_stash(ctx) ? 1 : 0;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t smem = gm_smem(ctx);
    if (++ctx->gm_calls == 0) {                         // the records' 32-bit call number starts a new lap: wipe the old lap
        ctx->gm_calls = 1;
        if (cudaMemsetAsync(ctx->d.gm_tile_rec, 0, sizeof(unsigned long long) * (size_t)kFuseTiles * a.R, st) != cudaSuccess) return MW_ERR_CUDA;
    }
    a.call = ctx->gm_calls;
    a.wait_call = (ctx->test_skew & MW_TEST_SKEW_GROUP_MAJOR) ? a.call + 0x40000000u : a.call;    // records nobody writes
    ctx->test_skew &= ~(uint32_t)MW_TEST_SKEW_GROUP_MAJOR;
    a.spin_limit = ctx->spin_limit;
    if (a.tiles <= kFuseTiles) {
        mw_launch(k_gm_fill<false>, dim3(a.tiles), dim3(kFillThreads), smem, st, true, a);
        ctx->launches += 1;
    } else {
        k_gm_sum<<<a.tiles, kTile, smem, st>>>(a);
        k_gm_scan<<<(a.R + kTile - 1) / kTile, kTile, 0, st>>>(a);
        mw_launch(k_gm_fill<true>, dim3(a.tiles), dim3(kFillThreads), smem, st, true, a);
        ctx->launches += 3;
    }
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
    if (T > 0 && a.tiles <= kFuseTiles) {
        k_ex_count<<<a.tiles, kTile, ex_smem(ctx), st>>>(a);
        mw_launch(k_ex_fill<true>, dim3(a.tiles), dim3(kTile), ex_smem(ctx), st, true, a);
        ctx->launches += 2;
    } else {
        if (T > 0) k_ex_count<<<a.tiles, kTile, ex_smem(ctx), st>>>(a);
        k_ex_scan<<<1, 1024, 0, st>>>(a);
        if (T > 0) mw_launch(k_ex_fill<false>, dim3(a.tiles), dim3(kTile), ex_smem(ctx), st, true, a);
        ctx->launches += T > 0 ? 3 : 1;
    }
    return cudaGetLastError() == cudaSuccess ? MW_OK : MW_ERR_CUDA;
}
