// Single-launch plan + pack + deliver for small batches (T <= 1024 tokens: 256 threads per block for the
// decode-sized ones, 1024 threads beyond 128 tokens).
//
// With a few dozen tokens the three-launch chain (plan, pack, deliver) is dominated by launch gaps and
// by the plan's chain of global-memory round trips, the cost the paper reports for its small batches
// (Section 6.3: replication overhead outweighs the savings at batch 64).  Here every block of the grid
// recomputes the whole plan in its own shared memory (the inputs are 2 KB) -- same rules, same results
// as the plan kernels, no grid-wide synchronisation -- and then moves its share of the rows: each row
// chunk is read once from x into registers and written to its slot of the MultiWrite send buffer and to
// every destination region.  A few blocks move no rows and write the plan metadata instead, so the
// context is left exactly as after mw_plan + mw_dispatch.
//
// The kernel is latency-bound (a batch of 64 tokens occupies two warps), so the work of every phase is
// spread over all threads of the block: whatever exists once per (token, expert slot) -- rank lookup,
// bitmap bit, slot inside the destination region, descriptors -- is done by one thread per pair, and
// only the group table and the per-token scalars are done by one thread per token.  Two expert slots of
// a token that name the same rank compute and store identical values; nothing below counts them twice.
// The kernel keeps no state on the host or in global scratch, so a captured launch can be replayed.
#include "mw_internal.cuh"

#include <type_traits>

namespace {

constexpr int kSmallThreads = 256;     // threads = largest T of the narrow variant (decode-sized batches)
constexpr int kMidThreads = 1024;      // threads = largest T of the wide variant (batches of up to 1024 tokens)
constexpr int kSmallNarrowBest = 128;  // up to this many tokens the 256-thread variant is the faster one
constexpr int kSmallMaxKd = 16;
constexpr int kSmallMaxW = 4;          // R <= 256: the three prefix sums fit one packed block scan
constexpr int kSmallChunk = 2048;      // bytes of a row moved by one warp at a time (4 x 16 bytes per lane)
constexpr int kSmallWriters = 4;       // blocks that write plan metadata instead of moving rows
constexpr int kSmallMinGrid = 16;      // smaller grids: block 0 writes everything and also moves rows

struct SmallArgs {
    const int32_t *ids, *e2r;
    const uint8_t *x;
    uint8_t *send, *recv;
    int T, K, E, R, W, Kd, src_rank, Tm;
    int64_t row_bytes, send_capacity_rows, recv_stride, recv_capacity_rows;
    // plan arrays the metadata blocks fill
    uint64_t *token_mask, *group_mask;
    int32_t *token_ndest, *token_group, *token_mw_row, *mw_row_token, *group_offsets, *rank_offsets, *rank_tokens;
    int32_t *dest_rank, *dest_pos, *token_leader, *row_ndest, *row_dest_rank, *row_dest_pos, *row_dest_flat;
    mw_totals *totals;
};

// Exclusive prefix sum over the NT threads of the block; `total` is returned to every thread.  V is a packed word:
// 32 bits hold the three sums of a 256-token batch, the 1024-token batch needs 64.
template <int NT, class V>
__device__ __forceinline__ V block_scan(V v, V *warp_sums, V &total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    V incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const V n = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += n; }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    const V ws = lane < NT / 32 ? warp_sums[lane] : (V)0;
    V wincl = ws;
#pragma unroll
    for (int o = 1; o < NT / 32; o <<= 1) { const V n = __shfl_up_sync(0xffffffffu, wincl, o); if (lane >= o) wincl += n; }
    total = __shfl_sync(0xffffffffu, wincl, NT / 32 - 1);
    const V before = __shfl_sync(0xffffffffu, wincl - ws, warp);
    return before + incl - v;
}

__device__ __forceinline__ uint4 ld16(const uint8_t *p)
{
    uint4 v;
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// Rank named by expert slot p = t * K + k, or -1 (padding or invalid).  ids and the table are inputs of the
// launch and never written by it, so the second look at them (descriptor phase) is served by L1.
__device__ __forceinline__ int slot_rank(const SmallArgs &a, int p, int &id_out)
{
    const int id = __ldg(a.ids + p);
    id_out = id;
    if (id < 0 || id >= a.E) return -1;
    const int r = __ldg(a.e2r + id);
    return (r >= 0 && r < a.R) ? r : -1;
}

template <int NT>
__global__ void __launch_bounds__(NT) k_dispatch_small(const __grid_constant__ SmallArgs a)
{
    constexpr int kSlots = 2 * NT;            // bitmap table in shared memory (load <= 1/2)
    constexpr int kWords = NT / 32;           // 32-token words per rank row of the bit matrix
    constexpr int kRow = kWords + 1;          // padded row
    // packed scan word: leaders | members << kB1 | destinations << kB2 (NT = 256: 9 + 9 + 13 bits; 1024: 11 + 11 + 15)
    using Packed = typename std::conditional<NT == 256, uint32_t, uint64_t>::type;
    constexpr int kB1 = NT == 256 ? 9 : 11, kB2 = 2 * kB1;
    constexpr Packed kM1 = ((Packed)1 << kB1) - 1;
    extern __shared__ __align__(16) uint8_t ssm[];
    // shared-memory layout (sizes depend on R, W, Kd)
    uint64_t *mask64 = (uint64_t *)ssm;                                    // [NT, W] bitmap of token t
    uint32_t *mask32 = (uint32_t *)ssm;                                    //          the same words as 32-bit halves
    unsigned long long *hkey = (unsigned long long *)(mask64 + NT * a.W);   // [2 NT] (hash tag, first claimant)
    int *hlead = (int *)(hkey + kSlots);                              // [2 NT] smallest token with that bitmap
    int *hcnt = hlead + kSlots;                                       // [2 NT] tokens with that bitmap
    int *hrun = hcnt + kSlots;                                        // [2 NT] members counted so far (rank inside a group)
    uint32_t *bits = (uint32_t *)(hrun + kSlots);                     // [R, NT/32 + 1] bit t of row r: token t targets rank r (padded rows)
    int *pre = (int *)(bits + a.R * kRow);                                    // [R, NT/32 + 1] tokens before each 32-token word that target r
    int *ro = pre + a.R * kRow;                                               // [R + 1] region starts
    int *nd_s = ro + a.R + 1;                                              // [NT] destinations of token t
    int *gid_s = nd_s + NT;                                     // [NT] group id, at the leader's index
    int *goff_s = gid_s + NT;                                   // [NT] group offset, at the leader's index
    int *tok_row_s = goff_s + NT;                               // [NT] send row of token t, -1 if none
    int *row_token_s = tok_row_s + NT;                          // [NT] token of send row j
    int *row_nd_s = row_token_s + NT;                           // [NT] destinations of send row j
    int *row_flat_s = row_nd_s + NT;                            // [NT, Kd] destination rows (rank<<16|slot when strided)
    __shared__ Packed warp_sums[32];
    __shared__ int s_acc[3];

    const int tid = threadIdx.x, t = tid, lane = tid & 31, warp = tid >> 5;
    const bool active = t < a.T;
    const int pairs = a.T * a.K;
    // which part of the metadata this block writes (-1: none), and its place among the blocks that move rows
    const int writers = (int)gridDim.x >= kSmallMinGrid ? kSmallWriters : 1;
    const int my_part = (int)blockIdx.x < writers ? (int)blockIdx.x : -1;
    auto writes = [&](int part) { return my_part >= 0 && part % writers == my_part; };
    const int movers = writers == 1 ? (int)gridDim.x : (int)gridDim.x - writers;
    const int mover = writers == 1 ? (int)blockIdx.x : (int)blockIdx.x - writers;

    // ---- clear the tables (no global memory involved: overlaps the tail of the previous kernel) ----
    grid_launch_dependents();
    for (int i = tid; i < NT * a.W; i += NT) mask64[i] = 0;
    for (int i = tid; i < kSlots; i += NT) { hkey[i] = ~0ull; hlead[i] = 0x7fffffff; hcnt[i] = 0; hrun[i] = 0; }
    for (int i = tid; i < a.R * kRow; i += NT) bits[i] = 0;
    if (tid < 3) s_acc[tid] = 0;
    grid_dependency_wait();        // the previous dispatch may still read the plan arrays this launch rewrites
    __syncthreads();

    // ---- one thread per expert slot: rank lookup, bitmap bit (Section 4.1: bit r set <=> rank r is a target;
    //      OR = several experts on one rank count once), token bit in the rank's row ----
    {
        int valid = 0, bad = 0;
        for (int p = tid; p < pairs; p += NT) {
            int id;
            const int r = slot_rank(a, p, id);
            bad |= (id != -1 && r < 0);
            if (r < 0) continue;
            ++valid;
            const int tk = p / a.K;
            atomicOr(mask32 + tk * 2 * a.W + (r >> 5), 1u << (r & 31));
            atomicOr(bits + r * kRow + (tk >> 5), 1u << (tk & 31));
        }
        valid = __reduce_add_sync(0xffffffffu, valid);
        bad = __reduce_or_sync(0xffffffffu, (unsigned)bad);
        if (lane == 0) {
            if (valid) atomicAdd(s_acc + 0, valid);
            if (bad) s_acc[2] = 1;
        }
    }
    __syncthreads();

    // ---- one thread per token: groups (table keyed by bitmap, leader = smallest token index);
    //      one thread per rank: tokens of each 32-token word that target it ----
    int nd = 0, slot = -1;
    if (active) {
        uint64_t h = 0x2545f4914f6cdd1dull;
        for (int w = 0; w < a.W; ++w) { const uint64_t m = mask64[t * a.W + w]; nd += __popcll(m); h = mix64(h, m); }
        if (a.src_rank >= 0 && nd == 1 && ((mask64[t * a.W + (a.src_rank >> 6)] >> (a.src_rank & 63)) & 1)) atomicAdd(s_acc + 1, 1);
        if (nd > 0) {
            const uint32_t tag = (uint32_t)(h >> 32);
            const unsigned long long mine = ((unsigned long long)tag << 32) | (uint32_t)t;
            slot = (int)(h & (kSlots - 1));
            for (int probes = 0; probes < kSlots; ++probes) {
                const unsigned long long cur = atomicCAS(hkey + slot, ~0ull, mine);
                if (cur == ~0ull) break;
                if ((uint32_t)(cur >> 32) == tag) {
                    const uint64_t *om = mask64 + (size_t)(uint32_t)cur * a.W;
                    bool same = true;
                    for (int w = 0; w < a.W; ++w) same &= (om[w] == mask64[t * a.W + w]);
                    if (same) break;
                }
                slot = (slot + 1) & (kSlots - 1);
            }
            atomicMin(hlead + slot, t);
            atomicAdd(hcnt + slot, 1);
        }
    }
    nd_s[tid] = nd;
    int my_cnt = 0;                // tokens that target rank `tid`
    if (tid < a.R) {
#pragma unroll
        for (int w8 = 0; w8 < kWords; ++w8) { pre[tid * kRow + w8] = my_cnt; my_cnt += __popc(bits[tid * kRow + w8]); }
    }
    __syncthreads();

    // ---- group ids, group offsets and region starts: three exclusive prefix sums in one packed scan
    //      (leaders <= NT, members <= NT, destinations <= 16 NT) ----
    const int leader = nd > 0 ? hlead[slot] : -1;
    const int gcount = nd > 0 ? hcnt[slot] : 0;
    const bool is_leader = nd > 0 && leader == t;
    Packed total;
    const Packed excl = block_scan<NT, Packed>((is_leader ? (Packed)1 | ((Packed)gcount << kB1) : (Packed)0) | ((Packed)my_cnt << kB2),
                                               warp_sums, total);
    const int G = (int)(total & kM1), Tn = (int)((total >> kB1) & kM1), SD = (int)(total >> kB2);
    const int goff_mine = (int)((excl >> kB1) & kM1);
    if (is_leader) { gid_s[tid] = (int)(excl & kM1); goff_s[tid] = goff_mine; }
    if (tid < a.R) ro[tid] = (int)(excl >> kB2);
    if (tid == 0) ro[a.R] = SD;

    // ---- rank inside the group, in token order.  Only when some group has more than one member: the warps
    //      take turns, and in each the first member of a group claims places for all its members of that warp ----
    int within = 0;
    if (G != Tn) {
        const int key = (nd > 0 && gcount > 1) ? slot : -1 - lane;       // negative keys are unique: groups of one
        const unsigned same = __match_any_sync(0xffffffffu, key);
        const int first = __ffs(same) - 1;
        for (int turn = 0; turn < NT / 32; ++turn) {
            if (warp == turn) {
                int base = 0;
                if (key >= 0 && lane == first) base = atomicAdd(hrun + slot, __popc(same));
                within = __shfl_sync(0xffffffffu, base, first) + __popc(same & ((1u << lane) - 1u));
            }
            __syncthreads();
        }
    } else {
        __syncthreads();
    }

    // ---- one thread per token: send row ----
    int g = -1, row = -1, overflow = 0;
    if (nd > 0) {
        g = gid_s[leader];
        row = goff_s[leader] + within;
        row_token_s[row] = t;
        row_nd_s[row] = nd;
        overflow = row >= a.send_capacity_rows;
    }
    tok_row_s[tid] = row;
    __syncthreads();

    // ---- one thread per expert slot: place among the token's destinations (= set bits below r), slot inside
    //      the region (= earlier tokens that target r), descriptors ----
    for (int p = tid; p < pairs; p += NT) {
        int id;
        const int r = slot_rank(a, p, id);
        if (r < 0) continue;
        const int tk = p / a.K, wi = tk >> 5;
        const uint64_t *m = mask64 + tk * a.W;
        int i = __popcll(m[r >> 6] & ((1ull << (r & 63)) - 1ull));
        for (int w = 0; w < (r >> 6); ++w) i += __popcll(m[w]);
        const int pos = pre[r * kRow + wi] + __popc(bits[r * kRow + wi] & ((1u << (tk & 31)) - 1u));
        const int flat = ro[r] + pos, rowk = tok_row_s[tk];
        row_flat_s[rowk * a.Kd + i] = a.recv_stride ? ((r << 16) | pos) : flat;
        overflow |= (a.recv_stride ? pos : flat) >= a.recv_capacity_rows;
        if (writes(2)) {
            a.dest_rank[tk * a.Kd + i] = r;
            a.dest_pos[tk * a.Kd + i] = pos;
            a.rank_tokens[flat] = tk;
        }
        if (writes(3)) {
            a.row_dest_rank[(int64_t)i * a.Tm + rowk] = r;
            a.row_dest_pos[(int64_t)i * a.Tm + rowk] = pos;
            a.row_dest_flat[(int64_t)i * a.Tm + rowk] = flat;
        }
    }
    __syncthreads();

    // ---- the metadata blocks leave the plan arrays exactly as the plan kernels would ----
    if (writes(0)) {
        // rows that do not fit their buffer are skipped by whichever block meets them; the status is written here
        overflow = __syncthreads_or(overflow);
        for (int r = tid; r <= a.R; r += NT) a.rank_offsets[r] = ro[r];
        if (tid == 0) {
            const int64_t self_copies = a.src_rank >= 0 ? ro[a.src_rank + 1] - ro[a.src_rank] : 0;
            const int64_t sent_rows = (int64_t)Tn - s_acc[1];
            mw_totals tt;
            tt.T_nonempty = Tn; tt.G = G; tt.total_dest = SD;
            tt.mw_bytes = sent_rows * a.row_bytes;
            tt.unicast_bytes = ((int64_t)SD - self_copies) * a.row_bytes;
            tt.unicast_per_expert_bytes = (int64_t)s_acc[0] * a.row_bytes;
            // Section 6.4: beyond 64 ranks the bitmap travels in the payload, once per 4096-byte packet
            tt.meta_bytes = a.R <= 64 ? 0 : sent_rows * ((a.row_bytes + 4095) / 4096) * (int64_t)(8 * a.W);
            tt.status = s_acc[2] ? MW_ERR_BAD_INDEX : overflow ? MW_ERR_CAPACITY : MW_OK;
            tt.reserved = 0;
            *a.totals = tt;
        }
        // tails
        for (int u = tid; u <= a.T; u += NT) {
            if (u > G) a.group_offsets[u] = -1;
            if (u == G) a.group_offsets[u] = Tn;
            if (u < a.T) {
                if (u >= Tn) a.mw_row_token[u] = -1;
                if (u >= G)
                    for (int w = 0; w < a.W; ++w) a.group_mask[(int64_t)u * a.W + w] = 0;
            }
        }
        for (int q = SD + tid; q < a.T * a.Kd; q += NT) a.rank_tokens[q] = -1;
    }
    if (writes(1) && active) {
        for (int w = 0; w < a.W; ++w) a.token_mask[(int64_t)t * a.W + w] = mask64[t * a.W + w];
        a.token_ndest[t] = nd;
        a.token_group[t] = g;
        a.token_mw_row[t] = row;
        a.token_leader[t] = leader;
        if (nd > 0) {
            a.mw_row_token[row] = t;
            a.row_ndest[row] = nd;
            if (is_leader) {
                a.group_offsets[g] = goff_mine;
                for (int w = 0; w < a.W; ++w) a.group_mask[(int64_t)g * a.W + w] = mask64[t * a.W + w];
            }
        }
    }
    if (writes(2) || writes(3)) {
        // unused entries: -1
        const bool lists = writes(2), planes = writes(3);
        for (int q = tid; q < a.T * a.Kd; q += NT) {
            const int tk = q / a.Kd, i = q % a.Kd, n = nd_s[tk];
            if (i < n) continue;
            if (lists) { a.dest_rank[q] = -1; a.dest_pos[q] = -1; }
            if (planes && n > 0) {
                const int64_t at = (int64_t)i * a.Tm + tok_row_s[tk];
                a.row_dest_rank[at] = -1; a.row_dest_pos[at] = -1; a.row_dest_flat[at] = -1;
            }
        }
    }
    if (mover < 0) return;

    // ---- rows: every warp of the moving blocks takes (send row, chunk) items round robin ----
    const int chunks = (int)((a.row_bytes + kSmallChunk - 1) / kSmallChunk);
    const int items = Tn * chunks;
    const int warps = movers * (NT / 32);
    for (int item = warp * movers + mover; item < items; item += warps) {
        const int j = item / chunks;
        const int64_t off = (int64_t)(item % chunks) * kSmallChunk;
        const int nvec = (int)(min((int64_t)kSmallChunk, a.row_bytes - off) >> 4);
        const uint8_t *src = a.x + (int64_t)row_token_s[j] * a.row_bytes + off + lane * 16;
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (u * 32 + lane < nvec) v[u] = ld16(src + u * 512);
        // destination 0 is the row's slot in the send buffer, the others are its receive slots
        const int n = row_nd_s[j];
        uint8_t *my_dst = nullptr;
        if (lane == 0) {
            if (j < a.send_capacity_rows) my_dst = a.send + (int64_t)j * a.row_bytes;
        } else if (lane <= n) {
            const int f = row_flat_s[j * a.Kd + lane - 1];
            if (a.recv_stride) {
                const int r = f >> 16, pos = f & 0xffff;
                if (pos < a.recv_capacity_rows) my_dst = a.recv + (int64_t)r * a.recv_stride + (int64_t)pos * a.row_bytes;
            } else {
                if (f < a.recv_capacity_rows) my_dst = a.recv + (int64_t)f * a.row_bytes;
            }
        }
        for (int q = 0; q <= n; ++q) {
            uint8_t *d = (uint8_t *)__shfl_sync(0xffffffffu, (unsigned long long)my_dst, q);
            if (!d) continue;
            d += off + lane * 16;
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (u * 32 + lane < nvec) *(uint4 *)(d + u * 512) = v[u];
        }
    }
}

size_t small_smem_bytes(const mw_ctx *ctx, int NT)
{
    const size_t R = (size_t)ctx->cfg.R, W = (size_t)ctx->W, Kd = (size_t)ctx->Kd, N = (size_t)NT;
    return N * W * 8 + 2 * N * 20 + R * (N / 32 + 1) * 8 + (R + 1) * 4 + 6 * N * 4 + N * Kd * 4 + 64;
}

bool small_fits(const mw_ctx *ctx, int NT)
{
    return ctx->W <= kSmallMaxW && ctx->Kd <= kSmallMaxKd && small_smem_bytes(ctx, NT) + 1024 <= (size_t)ctx->max_smem_optin;
}

}  // namespace

// True if the single-launch path can serve this context and batch.
bool mw_small_applies(const mw_ctx *ctx, int32_t T, int layout)
{
    return layout == MW_LAYOUT_MULTIWRITE &&
           !(ctx->cfg.flags & MW_FLAG_PLAN_MULTIPASS) &&
           ((T <= kSmallThreads && small_fits(ctx, kSmallThreads)) || (T <= kMidThreads && small_fits(ctx, kMidThreads)));
}

int mw_small_setup(mw_ctx *ctx)
{
    if (small_fits(ctx, kSmallThreads) && small_smem_bytes(ctx, kSmallThreads) > 48 * 1024 &&
        cudaFuncSetAttribute(k_dispatch_small<kSmallThreads>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)small_smem_bytes(ctx, kSmallThreads)) != cudaSuccess)
        return MW_ERR_CUDA;
    if (small_fits(ctx, kMidThreads) && small_smem_bytes(ctx, kMidThreads) > 48 * 1024 &&
        cudaFuncSetAttribute(k_dispatch_small<kMidThreads>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)small_smem_bytes(ctx, kMidThreads)) != cudaSuccess)
        return MW_ERR_CUDA;
    return MW_OK;
}

int mw_small_launch(mw_ctx *ctx, const int32_t *topk_ids, const int32_t *expert_to_rank, int32_t T, const void *x,
                    void *send_buf, int64_t send_capacity_rows, void *recv_base, int64_t recv_stride_bytes,
                    int64_t recv_capacity_rows, cudaStream_t st)
{
    SmallArgs a;
    a.ids = topk_ids; a.e2r = expert_to_rank;
    a.x = (const uint8_t *)x; a.send = (uint8_t *)send_buf; a.recv = (uint8_t *)recv_base;
    a.T = T; a.K = ctx->cfg.K; a.E = ctx->cfg.E; a.R = ctx->cfg.R; a.W = ctx->W; a.Kd = ctx->Kd;
    a.src_rank = ctx->cfg.src_rank; a.Tm = ctx->cfg.max_tokens;
    a.row_bytes = ctx->cfg.row_bytes;
    a.send_capacity_rows = send_capacity_rows;
    a.recv_stride = recv_stride_bytes;
    a.recv_capacity_rows = recv_capacity_rows;
    const mw_dev &d = ctx->d;
    a.token_mask = d.token_mask; a.group_mask = d.group_mask;
    a.token_ndest = d.token_ndest; a.token_group = d.token_group; a.token_mw_row = d.token_mw_row;
    a.mw_row_token = d.mw_row_token; a.group_offsets = d.group_offsets; a.rank_offsets = d.rank_offsets;
    a.rank_tokens = d.rank_tokens; a.dest_rank = d.dest_rank; a.dest_pos = d.dest_pos; a.token_leader = d.token_leader;
    a.row_ndest = d.row_ndest; a.row_dest_rank = d.row_dest_rank; a.row_dest_pos = d.row_dest_pos;
    a.row_dest_flat = d.row_dest_flat; a.totals = d.totals;
    // Measured on B200 (plan part alone, 64 ranks, top-8; microseconds per call back to back, 256 / 1024 threads):
    // 64 tokens 4.9 / 5.3, 128 tokens 6.0 / 6.0, 192 tokens 8.4 / 6.9, 256 tokens 10.2 / 8.4.
    const bool narrow = T <= kSmallThreads && small_fits(ctx, kSmallThreads) && (T <= kSmallNarrowBest || !small_fits(ctx, kMidThreads));
    const cudaError_t e = !narrow
        ? mw_launch(k_dispatch_small<kMidThreads>, dim3(ctx->sm_count), dim3(kMidThreads), small_smem_bytes(ctx, kMidThreads), st,
                    !(ctx->cfg.flags & MW_FLAG_NO_OVERLAP), a)
        : mw_launch(k_dispatch_small<kSmallThreads>, dim3(ctx->sm_count), dim3(kSmallThreads), small_smem_bytes(ctx, kSmallThreads), st,
                    !(ctx->cfg.flags & MW_FLAG_NO_OVERLAP), a);
    ctx->launches += 1;
    ctx->planned_T = T;
    ctx->epoch += 1;          // a new plan (the tiled plan's own counts live on the device and are not touched here)
    ctx->plan_epoch = ctx->epoch;
    ctx->prefetched = nullptr;
    if (e != cudaSuccess) { cudaGetLastError(); return MW_ERR_CUDA; }
    return MW_OK;
}
