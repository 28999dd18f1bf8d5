// Single-launch plan + pack + deliver for small batches (decode-sized: T <= 256 tokens).
//
// With a few dozen tokens the three-launch chain (plan, pack, deliver) is dominated by launch gaps and
// by the plan's chain of global-memory round trips, the cost the paper reports for its small batches
// (Section 6.3: replication overhead outweighs the savings at batch 64).  Here every block of a
// persistent grid recomputes the whole plan in its own shared memory (the inputs are 2 KB) -- same
// rules, same results as the plan kernels, no grid-wide synchronisation -- and then moves its share of
// the rows: each row chunk is read once from x into registers and written to its slot of the MultiWrite
// send buffer and to every destination region.  Block 0 also writes the plan metadata, so the context
// is left exactly as after mw_plan + mw_dispatch.
#include "mw_internal.cuh"

namespace {

constexpr int kSmallThreads = 256;     // = largest T
constexpr int kSmallSlots = 512;       // bitmap table in shared memory (load <= 1/2)
constexpr int kSmallMaxKd = 16;
constexpr int kSmallMaxW = 4;
constexpr int kSmallChunk = 2048;      // bytes of a row moved by one warp at a time (4 x 16 bytes per lane)

struct SmallArgs {
    const int32_t *ids, *e2r;
    const uint8_t *x;
    uint8_t *send, *recv;
    int T, K, E, R, W, Kd, src_rank, Tm;
    int64_t row_bytes, send_capacity_rows, recv_stride, recv_capacity_rows;
    mw_dev d;
};

__device__ __forceinline__ uint64_t mix64s(uint64_t h, uint64_t v)
{
    h ^= v + 0x9e3779b97f4a7c15ull + (h << 6) + (h >> 2);
    h ^= h >> 33; h *= 0xff51afd7ed558ccdull; h ^= h >> 29;
    return h;
}

// Exclusive prefix sum over the 256 threads of the block; `total` is returned to every thread.
__device__ __forceinline__ int scan256(int v, int *warp_sums, int &total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { int n = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += n; }
    __syncthreads();
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    int before = 0, sum = 0;
#pragma unroll
    for (int w = 0; w < kSmallThreads / 32; ++w) { const int s = warp_sums[w]; if (w < warp) before += s; sum += s; }
    total = sum;
    return before + incl - v;
}

__device__ __forceinline__ uint4 ld16(const uint8_t *p)
{
    uint4 v;
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st16(uint8_t *p, const uint4 &v)
{
    asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

template <int WT>
__global__ void __launch_bounds__(kSmallThreads) k_dispatch_small(const __grid_constant__ SmallArgs a)
{
    extern __shared__ __align__(16) uint8_t ssm[];
    // shared-memory layout (sizes depend on R, W, Kd)
    uint64_t *masks_s = (uint64_t *)ssm;                                   // [256, W]
    unsigned long long *hkey = (unsigned long long *)(masks_s + kSmallThreads * a.W);   // [512]
    int *hlead = (int *)(hkey + kSmallSlots);                              // [512]
    int *hcnt = hlead + kSmallSlots;                                       // [512]
    uint32_t *bits = (uint32_t *)(hcnt + kSmallSlots);                     // [R, 9] (padded rows)
    int *pre = (int *)(bits + a.R * 9);                                    // [R, 9]
    int *cnt = pre + a.R * 9;                                              // [R]
    int *ro = cnt + a.R;                                                   // [R + 1]
    int *leader_s = ro + a.R + 1;                                          // [256]
    int *gid_s = leader_s + kSmallThreads;                                 // [256] group id, at the leader's index
    int *goff_s = gid_s + kSmallThreads;                                   // [256] group offset, at the leader's index
    int *row_token_s = goff_s + kSmallThreads;                             // [256] token of send row j
    int *row_nd_s = row_token_s + kSmallThreads;                           // [256] destinations of send row j
    int *row_flat_s = row_nd_s + kSmallThreads;                            // [256, Kd] destination rows (or rank<<16|slot when strided)
    __shared__ int warp_sums[kSmallThreads / 32];
    __shared__ int s_acc[3];

    const int tid = threadIdx.x, t = tid;
    const bool active = t < a.T;
    grid_launch_dependents();
    grid_dependency_wait();        // the previous dispatch may still read the plan arrays block 0 rewrites

    // ---- bitmaps ----
    uint64_t m[WT];
#pragma unroll
    for (int w = 0; w < WT; ++w) m[w] = 0;
    int nd = 0, valid = 0, bad = 0, self_only = 0;
    uint64_t h = 0x2545f4914f6cdd1dull;
    if (active) {
        const int32_t *my = a.ids + (int64_t)t * a.K;
        for (int k0 = 0; k0 < a.K; k0 += 8) {
            int id[8], r[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) id[j] = (k0 + j < a.K) ? my[k0 + j] : -1;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const bool ok = id[j] >= 0 && id[j] < a.E;
                bad |= (id[j] != -1 && !ok);
                r[j] = ok ? a.e2r[id[j]] : -1;
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const bool ok = r[j] >= 0 && r[j] < a.R;
                bad |= (id[j] >= 0 && id[j] < a.E && !ok);
                valid += ok;
                if (ok) {
#pragma unroll
                    for (int w = 0; w < WT; ++w)
                        if ((r[j] >> 6) == w) m[w] |= 1ull << (r[j] & 63);          // OR = per-rank dedup
                }
            }
        }
#pragma unroll
        for (int w = 0; w < WT; ++w)
            if (w < a.W) { masks_s[tid * a.W + w] = m[w]; nd += __popcll(m[w]); h = mix64s(h, m[w]); }
        if (a.src_rank >= 0 && nd == 1) {
#pragma unroll
            for (int w = 0; w < WT; ++w)
                if ((a.src_rank >> 6) == w) self_only = (m[w] >> (a.src_rank & 63)) & 1;
        }
    }
    for (int i = tid; i < kSmallSlots; i += kSmallThreads) { hkey[i] = ~0ull; hlead[i] = 0x7fffffff; hcnt[i] = 0; }
    for (int i = tid; i < a.R * 9; i += kSmallThreads) bits[i] = 0;
    if (tid < 3) s_acc[tid] = 0;
    __syncthreads();
    valid = __reduce_add_sync(0xffffffffu, valid);
    self_only = __reduce_add_sync(0xffffffffu, self_only);
    bad = __reduce_or_sync(0xffffffffu, (unsigned)bad);
    if ((tid & 31) == 0) {
        if (valid) atomicAdd(s_acc + 0, valid);
        if (self_only) atomicAdd(s_acc + 1, self_only);
        if (bad) s_acc[2] = 1;
    }

    // ---- groups: table keyed by bitmap, leader = smallest token index ----
    int slot = -1;
    const int wi = tid >> 5;
    const uint32_t bit = 1u << (tid & 31);
    if (nd > 0) {
        const uint32_t tag = (uint32_t)(h >> 32);
        const unsigned long long mine = ((unsigned long long)tag << 32) | (uint32_t)t;
        slot = (int)(h & (kSmallSlots - 1));
        for (int probes = 0; probes < kSmallSlots; ++probes) {
            const unsigned long long cur = atomicCAS(hkey + slot, ~0ull, mine);
            if (cur == ~0ull) break;
            if ((uint32_t)(cur >> 32) == tag) {
                const uint64_t *om = masks_s + (size_t)(uint32_t)cur * a.W;
                bool same = true;
#pragma unroll
                for (int w = 0; w < WT; ++w)
                    if (w < a.W) same &= (om[w] == m[w]);
                if (same) break;
            }
            slot = (slot + 1) & (kSmallSlots - 1);
        }
        atomicMin(hlead + slot, t);
        atomicAdd(hcnt + slot, 1);
#pragma unroll
        for (int w = 0; w < WT; ++w)
            for (uint64_t word = m[w]; word; word &= word - 1)
                atomicOr(bits + (size_t)(w * 64 + __ffsll((long long)word) - 1) * 9 + wi, bit);
    }
    __syncthreads();
    const int leader = nd > 0 ? hlead[slot] : -1;
    const int gcount = nd > 0 ? hcnt[slot] : 0;
    leader_s[tid] = leader;
    const bool is_leader = nd > 0 && leader == t;
    for (int r = tid; r < a.R; r += kSmallThreads) {
        int run = 0;
#pragma unroll
        for (int w8 = 0; w8 < 8; ++w8) { pre[r * 9 + w8] = run; run += __popc(bits[r * 9 + w8]); }
        cnt[r] = run;
    }
    int G, Tn, SD;
    const int gid = scan256(is_leader ? 1 : 0, warp_sums, G);
    const int goff_mine = scan256(is_leader ? gcount : 0, warp_sums, Tn);
    if (is_leader) { gid_s[tid] = gid; goff_s[tid] = goff_mine; }
    {
        int carry = 0;
        for (int r0 = 0; r0 < a.R; r0 += kSmallThreads) {
            const int r = r0 + tid;
            int total;
            const int excl = scan256(r < a.R ? cnt[r] : 0, warp_sums, total);
            if (r < a.R) ro[r] = carry + excl;
            carry += total;
        }
        SD = carry;
        if (tid == 0) ro[a.R] = carry;
    }
    __syncthreads();

    // ---- send rows and destination slots ----
    int row = -1, g = -1;
    if (nd > 0) {
        int within = 0;
        if (gcount > 1)
            for (int u = leader; u < t; ++u) within += (leader_s[u] == leader);
        g = gid_s[leader];
        row = goff_s[leader] + within;
        row_token_s[row] = t;
        row_nd_s[row] = nd;
        int i = 0;
#pragma unroll
        for (int w = 0; w < WT; ++w)
            for (uint64_t word = m[w]; word; word &= word - 1) {
                const int r = w * 64 + __ffsll((long long)word) - 1;
                const int pos = pre[r * 9 + wi] + __popc(bits[r * 9 + wi] & (bit - 1));
                row_flat_s[row * a.Kd + i] = a.recv_stride ? ((r << 16) | pos) : ro[r] + pos;
                ++i;
            }
    }
    __syncthreads();

    // ---- block 0 leaves the plan metadata exactly as the plan kernels would ----
    if (blockIdx.x == 0) {
        // rows that do not fit their buffer are skipped by whichever block meets them; the status is block 0's to write
        int overflow = 0;
        if (nd > 0) {
            overflow |= row >= a.send_capacity_rows;
            for (int i = 0; i < nd; ++i) {
                const int f = row_flat_s[row * a.Kd + i];
                overflow |= (a.recv_stride ? (f & 0xffff) : f) >= a.recv_capacity_rows;
            }
        }
        overflow = __syncthreads_or(overflow);
        for (int r = tid; r <= a.R; r += kSmallThreads) a.d.rank_offsets[r] = ro[r];
        if (tid == 0) {
            const int64_t self_copies = a.src_rank >= 0 ? cnt[a.src_rank] : 0;
            const int64_t sent_rows = (int64_t)Tn - s_acc[1];
            a.d.group_offsets[G] = Tn;
            mw_totals tt;
            tt.T_nonempty = Tn; tt.G = G; tt.total_dest = SD;
            tt.mw_bytes = sent_rows * a.row_bytes;
            tt.unicast_bytes = ((int64_t)SD - self_copies) * a.row_bytes;
            tt.unicast_per_expert_bytes = (int64_t)s_acc[0] * a.row_bytes;
            // Section 6.4: beyond 64 ranks the bitmap travels in the payload, once per 4096-byte packet
            tt.meta_bytes = a.R <= 64 ? 0 : sent_rows * ((a.row_bytes + 4095) / 4096) * (int64_t)(8 * a.W);
            tt.status = s_acc[2] ? MW_ERR_BAD_INDEX : overflow ? MW_ERR_CAPACITY : MW_OK;
            tt.reserved = 0;
            *a.d.totals = tt;
        }
        for (int u = tid; u <= a.T; u += kSmallThreads) {
            if (u > G) a.d.group_offsets[u] = -1;
            if (u < a.T) {
                if (u >= Tn) a.d.mw_row_token[u] = -1;
                for (int i = 0; i < a.Kd; ++i)
                    if (u * a.Kd + i >= SD) a.d.rank_tokens[u * a.Kd + i] = -1;
                if (u >= G)
                    for (int w = 0; w < a.W; ++w) a.d.group_mask[(int64_t)u * a.W + w] = 0;
            }
        }
        if (active) {
            for (int w = 0; w < a.W; ++w) a.d.token_mask[(int64_t)t * a.W + w] = masks_s[tid * a.W + w];
            a.d.token_ndest[t] = nd;
            a.d.token_group[t] = g;
            a.d.token_mw_row[t] = row;
            int32_t *dr = a.d.dest_rank + (int64_t)t * a.Kd, *dp = a.d.dest_pos + (int64_t)t * a.Kd;
            int i = 0;
            if (nd > 0) {
                a.d.mw_row_token[row] = t;
                a.d.row_ndest[row] = nd;
                a.d.token_leader[t] = leader;
                if (is_leader) {
                    a.d.group_offsets[g] = goff_s[tid];
                    for (int w = 0; w < a.W; ++w) a.d.group_mask[(int64_t)g * a.W + w] = masks_s[tid * a.W + w];
                }
#pragma unroll
                for (int w = 0; w < WT; ++w)
                    for (uint64_t word = m[w]; word; word &= word - 1) {
                        const int r = w * 64 + __ffsll((long long)word) - 1;
                        const int pos = pre[r * 9 + wi] + __popc(bits[r * 9 + wi] & (bit - 1));
                        dr[i] = r;
                        dp[i] = pos;
                        a.d.rank_tokens[ro[r] + pos] = t;
                        a.d.row_dest_rank[(int64_t)i * a.Tm + row] = r;
                        a.d.row_dest_pos[(int64_t)i * a.Tm + row] = pos;
                        a.d.row_dest_flat[(int64_t)i * a.Tm + row] = ro[r] + pos;
                        ++i;
                    }
                for (int q = i; q < a.Kd; ++q) {
                    a.d.row_dest_rank[(int64_t)q * a.Tm + row] = -1;
                    a.d.row_dest_pos[(int64_t)q * a.Tm + row] = -1;
                    a.d.row_dest_flat[(int64_t)q * a.Tm + row] = -1;
                }
            } else {
                a.d.token_leader[t] = -1;
            }
            for (; i < a.Kd; ++i) { dr[i] = -1; dp[i] = -1; }
        }
    }

    // ---- rows: every warp of the grid takes (send row, chunk) items round robin ----
    const int lane = tid & 31;
    const int chunks = (int)((a.row_bytes + kSmallChunk - 1) / kSmallChunk);
    const int items = Tn * chunks;
    const int warps = gridDim.x * (kSmallThreads / 32);
    for (int item = (tid >> 5) * gridDim.x + blockIdx.x; item < items; item += warps) {
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
                if (u * 32 + lane < nvec) st16(d + u * 512, v[u]);
        }
    }
}

size_t small_smem_bytes(const mw_ctx *ctx)
{
    const size_t R = (size_t)ctx->cfg.R, W = (size_t)ctx->W, Kd = (size_t)ctx->Kd;
    return kSmallThreads * W * 8 + kSmallSlots * 16 + R * 9 * 8 + (2 * R + 1) * 4 + 5 * kSmallThreads * 4 + kSmallThreads * Kd * 4 + 64;
}

}  // namespace

// True if the single-launch path can serve this context and batch.
bool mw_small_applies(const mw_ctx *ctx, int32_t T, int layout)
{
    return T <= kSmallThreads && layout == MW_LAYOUT_MULTIWRITE && ctx->W <= kSmallMaxW && ctx->Kd <= kSmallMaxKd &&
           !(ctx->cfg.flags & (MW_FLAG_PLAN_MULTIPASS | MW_FLAG_PLAN_COOPERATIVE | MW_FLAG_COPY_LDST | MW_FLAG_COPY_REG_STORE)) &&
           small_smem_bytes(ctx) + 1024 <= (size_t)ctx->max_smem_optin;
}

int mw_small_setup(mw_ctx *ctx)
{
    const size_t need = small_smem_bytes(ctx);
    if (ctx->W > kSmallMaxW || ctx->Kd > kSmallMaxKd || need + 1024 > (size_t)ctx->max_smem_optin) return MW_OK;   // path not available
    void (*fn)(SmallArgs) = ctx->W <= 1 ? k_dispatch_small<1> : ctx->W <= 2 ? k_dispatch_small<2> : k_dispatch_small<4>;
    if (need > 48 * 1024 && cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need) != cudaSuccess)
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
    a.d = ctx->d;
    void (*fn)(SmallArgs) = ctx->W <= 1 ? k_dispatch_small<1> : ctx->W <= 2 ? k_dispatch_small<2> : k_dispatch_small<4>;
    const cudaError_t e = mw_launch(fn, dim3(ctx->sm_count), dim3(kSmallThreads), small_smem_bytes(ctx), st,
                                    !(ctx->cfg.flags & MW_FLAG_NO_OVERLAP), a);
    ctx->launches += 1;
    ctx->planned_T = T;
    if (e != cudaSuccess) { cudaGetLastError(); return MW_ERR_CUDA; }
    return MW_OK;
}
