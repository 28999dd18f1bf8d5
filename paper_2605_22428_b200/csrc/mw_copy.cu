// Row-copy engine: every data-movement step of the path (pack in either layout, deliver in either
// layout, the AllGather forms) is "read a row once, write it to n destinations", with n and the
// destination addresses given by the plan.  (Paper: Section 5.2 step 1, loading the send buffer;
// Section 4.1 steps 3-5 and Section 4.3.3, the relay replicating a payload to every destination
// named by its bitmap.)
//
// Two implementations of the same work list:
//   k_copy_bulk  each warp runs its own pipeline of bulk asynchronous copies: global -> shared
//                (completion counted on an mbarrier), then one shared -> global bulk store per
//                destination, issued by different lanes.  A handful of instructions per row,
//                the copy engines move the bytes, and a row is read from memory exactly once.
//   k_copy_ldst  each warp moves a row chunk through registers with 16-byte loads and stores.
// A work item is (row, chunk); items are dealt round-robin to all warps of a persistent grid.
#include "mw_internal.cuh"

namespace {

constexpr int kBulkWarps = 4;          // pipelines per block
constexpr int kMaxStages = 8;
constexpr int kLdstThreads = 512;
constexpr int kWaitLimit = 1 << 20;    // mbarrier polls (about 1 us each) before giving up

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, int count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Polls with a suspend-time hint; false after kWaitLimit polls.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity)
{
    const uint32_t addr = smem_u32(bar);
    for (int i = 0; i < kWaitLimit; ++i) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done) : "r"(addr), "r"(parity), "r"(1000u) : "memory");
        if (done) return true;
    }
    return false;
}
__device__ __forceinline__ void bulk_load(void *smem_dst, const void *gsrc, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void bulk_store(void *gdst, const void *smem_src, uint32_t bytes, uint64_t policy)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;"
                 ::"l"(gdst), "r"(smem_u32(smem_src)), "r"(bytes), "l"(policy) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ uint64_t policy_evict_first()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t policy_evict_normal()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
    return p;
}

__device__ __forceinline__ void flag_error(const mw_copy_args &a, int err) { atomicCAS(&a.totals->status, 0, err); }

// ---- the work list -------------------------------------------------------------------------
__device__ __forceinline__ int64_t n_rows(const mw_copy_args &a)
{
    if (a.rows_from == 1) return a.totals->T_nonempty;
    if (a.rows_from == 2) return a.totals->total_dest;
    return a.host_rows;
}

__device__ __forceinline__ const uint8_t *src_row(const mw_copy_args &a, int64_t row)
{
    switch (a.mode) {
    case MW_CP_PACK_MW: return a.src + (int64_t)a.src_index[row] * a.row_bytes;
    case MW_CP_AG_DELIVER_UC: {
        const int64_t i = row / a.dst_count, d = row % a.dst_count;
        return (a.dst_begin + d == i) ? a.src2 + i * a.row_bytes : a.src + row * a.row_bytes;
    }
    default: return a.src + row * a.row_bytes;
    }
}

__device__ __forceinline__ int n_dst(const mw_copy_args &a, int64_t row)
{
    switch (a.mode) {
    case MW_CP_SCATTER: return a.ndst[row];
    case MW_CP_AG_DELIVER_MW:
    case MW_CP_AG_PACK_UC: return a.dst_count;
    default: return 1;
    }
}

// Destination q of a row; nullptr when the copy must not happen (capacity exceeded -> status, or the
// AllGather copy addressed to the shard's own rank, which is never transmitted).
__device__ __forceinline__ uint8_t *dst_row(const mw_copy_args &a, int64_t row, int q)
{
    switch (a.mode) {
    case MW_CP_PACK_MW:
    case MW_CP_AG_PACK_MW:
        if (row >= a.capacity_rows) { flag_error(a, MW_ERR_CAPACITY); return nullptr; }
        return a.dst + row * a.row_bytes;
    case MW_CP_SCATTER: {
        const int r = a.d_rank[row * a.Kd + q], p = a.d_pos[row * a.Kd + q];
        if (r < 0) return nullptr;
        if (a.dst_stride) {
            if (p >= a.capacity_rows) { flag_error(a, MW_ERR_CAPACITY); return nullptr; }
            return a.dst + (int64_t)r * a.dst_stride + (int64_t)p * a.row_bytes;
        }
        const int64_t at = (int64_t)a.rank_offsets[r] + p;
        if (at >= a.capacity_rows) { flag_error(a, MW_ERR_CAPACITY); return nullptr; }
        return a.dst + at * a.row_bytes;
    }
    case MW_CP_DELIVER_UC: {
        if (!a.dst_stride) {
            if (row >= a.capacity_rows) { flag_error(a, MW_ERR_CAPACITY); return nullptr; }
            return a.dst + row * a.row_bytes;
        }
        const int r = a.uc_row_rank[row];
        const int64_t p = row - a.rank_offsets[r];
        if (p >= a.capacity_rows) { flag_error(a, MW_ERR_CAPACITY); return nullptr; }
        return a.dst + (int64_t)r * a.dst_stride + p * a.row_bytes;
    }
    case MW_CP_AG_DELIVER_MW: return a.dst + (int64_t)q * a.dst_stride + row * a.row_bytes;
    case MW_CP_AG_PACK_UC:
        if (a.dst_begin + q == row) return nullptr;
        return a.dst + (row * a.dst_count + q) * a.row_bytes;
    case MW_CP_AG_DELIVER_UC: {
        const int64_t i = row / a.dst_count, d = row % a.dst_count;
        return a.dst + d * a.dst_stride + i * a.row_bytes;
    }
    }
    return nullptr;
}

__device__ __forceinline__ bool plan_unusable(const mw_copy_args &a)
{
    return a.totals && a.rows_from != 0 && a.totals->status == MW_ERR_TIMEOUT;
}

// ---- bulk-copy pipelines -------------------------------------------------------------------
__global__ void __launch_bounds__(kBulkWarps * 32, 1) k_copy_bulk(const __grid_constant__ mw_copy_args a)
{
    extern __shared__ __align__(128) uint8_t stage_mem[];
    __shared__ __align__(8) uint64_t bars[kBulkWarps * kMaxStages];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nst = a.stages;
    const uint32_t stage_stride = ((uint32_t)a.chunk_bytes + 127u) & ~127u;
    uint8_t *stages = stage_mem + (size_t)warp * nst * stage_stride;
    uint64_t *bar = bars + warp * kMaxStages;
    if (lane == 0)
        for (int s = 0; s < nst; ++s) mbar_init(bar + s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncwarp();
    if (plan_unusable(a)) return;

    const int64_t items = n_rows(a) * a.chunks_per_row;
    const int64_t step = (int64_t)gridDim.x * kBulkWarps;
    const int64_t first = (int64_t)warp * gridDim.x + blockIdx.x;
    // send rows are read again by the deliver step: keep them in L2; receive rows are not
    const uint64_t policy = (a.mode == MW_CP_PACK_MW || a.mode == MW_CP_AG_PACK_MW) ? policy_evict_normal() : policy_evict_first();

    auto issue_load = [&](int64_t item, int s) {
        const int64_t row = item / a.chunks_per_row;
        const int64_t off = (item % a.chunks_per_row) * (int64_t)a.chunk_bytes;
        const uint32_t bytes = (uint32_t)min((int64_t)a.chunk_bytes, a.row_bytes - off);
        mbar_expect_tx(bar + s, bytes);
        bulk_load(stages + (size_t)s * stage_stride, src_row(a, row) + off, bytes, bar + s);
    };

    int64_t next_load = first;
    int loads_issued = 0;
    if (lane == 0)
        for (int s = 0; s < nst - 1 && next_load < items; ++s, next_load += step, ++loads_issued) issue_load(next_load, s);
    loads_issued = __shfl_sync(0xffffffffu, loads_issued, 0);
    next_load = first + (int64_t)loads_issued * step;

    int n = 0;
    bool ok = true;
    for (int64_t item = first; item < items; item += step, ++n) {
        const int s = n % nst;
        const int64_t row = item / a.chunks_per_row;
        const int64_t off = (item % a.chunks_per_row) * (int64_t)a.chunk_bytes;
        const uint32_t bytes = (uint32_t)min((int64_t)a.chunk_bytes, a.row_bytes - off);
        const int nd = n_dst(a, row);
        uint8_t *my_dst = lane < nd ? dst_row(a, row, lane) : nullptr;      // overlaps the wait below
        if (!mbar_wait(bar + s, (uint32_t)(n / nst) & 1u)) { ok = false; break; }
        const uint8_t *stage = stages + (size_t)s * stage_stride;
        if (my_dst) bulk_store(my_dst + off, stage, bytes, policy);
        for (int q = lane + 32; q < nd; q += 32) {
            uint8_t *d = dst_row(a, row, q);
            if (d) bulk_store(d + off, stage, bytes, policy);
        }
        bulk_commit();
        if (next_load < items) {
            // the stage that item n-1 used is free once every lane's stores of that item have read it
            bulk_wait_read<1>();
            __syncwarp();
            if (lane == 0) issue_load(next_load, (n + nst - 1) % nst);
            next_load += step;
            ++loads_issued;
        }
    }
    if (!ok) {
        // a load never arrived: report it, then give the loads still in flight a bounded chance to land
        if (lane == 0) flag_error(a, MW_ERR_TIMEOUT);
        for (int m = n + 1; m < loads_issued; ++m) mbar_wait(bar + (m % nst), (uint32_t)(m / nst) & 1u);
    }
    bulk_wait_all();
}

// ---- register copies -----------------------------------------------------------------------
__device__ __forceinline__ uint4 ld_stream(const uint8_t *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(uint8_t *p, const uint4 &v)
{
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

__global__ void __launch_bounds__(kLdstThreads) k_copy_ldst(const __grid_constant__ mw_copy_args a)
{
    if (plan_unusable(a)) return;
    constexpr int U = 4;
    const int lane = threadIdx.x & 31;
    const int warps_per_block = kLdstThreads / 32;
    const int64_t items = n_rows(a) * a.chunks_per_row;
    const int64_t step = (int64_t)gridDim.x * warps_per_block;
    for (int64_t item = (int64_t)(threadIdx.x >> 5) * gridDim.x + blockIdx.x; item < items; item += step) {
        const int64_t row = item / a.chunks_per_row;
        const int64_t off = (item % a.chunks_per_row) * (int64_t)a.chunk_bytes;
        const int nvec = (int)(min((int64_t)a.chunk_bytes, a.row_bytes - off) >> 4);
        const int nd = n_dst(a, row);
        const uint8_t *src = src_row(a, row) + off;
        for (int qb = 0; qb < nd; qb += 32) {
            uint8_t *my_dst = qb + lane < nd ? dst_row(a, row, qb + lane) : nullptr;
            const int nq = min(32, nd - qb);
            for (int v0 = 0; v0 < nvec; v0 += 32 * U) {
                uint4 v[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int vi = v0 + u * 32 + lane;
                    if (vi < nvec) v[u] = ld_stream(src + (int64_t)vi * 16);
                }
                for (int q = 0; q < nq; ++q) {
                    uint8_t *d = (uint8_t *)__shfl_sync(0xffffffffu, (unsigned long long)my_dst, q);
                    if (!d) continue;
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        const int vi = v0 + u * 32 + lane;
                        if (vi < nvec) st_stream(d + off + (int64_t)vi * 16, v[u]);
                    }
                }
            }
        }
    }
}

}  // namespace

int mw_copy_smem_setup(mw_ctx *ctx)
{
    if (cudaFuncSetAttribute(k_copy_bulk, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             ctx->max_smem_optin - 1024) != cudaSuccess)
        return MW_ERR_CUDA;
    return MW_OK;
}

// Chooses the work-item size and the pipeline depth, then launches a persistent grid.
int mw_copy_launch(mw_ctx *ctx, mw_copy_args a, cudaStream_t st)
{
    const bool ldst = (ctx->cfg.flags & MW_FLAG_COPY_LDST) != 0;
    const int64_t est_rows = a.host_rows >= 0 ? a.host_rows : 0;
    const int64_t warps = (int64_t)ctx->sm_count * (ldst ? 2 * (kLdstThreads / 32) : kBulkWarps);
    int64_t chunk = a.row_bytes < 16384 ? a.row_bytes : 16384;
    // few, long rows (AllGather shards): cut smaller pieces so that every warp has work
    while (chunk > 2048 && chunk % 32 == 0 && est_rows * ((a.row_bytes + chunk - 1) / chunk) < 2 * warps) chunk /= 2;
    a.chunk_bytes = (int32_t)chunk;
    a.chunks_per_row = (int32_t)((a.row_bytes + chunk - 1) / chunk);
    if (ldst) {
        k_copy_ldst<<<ctx->sm_count * 2, kLdstThreads, 0, st>>>(a);
    } else {
        const int64_t stage_stride = (chunk + 127) & ~(int64_t)127;
        const int64_t budget = ctx->max_smem_optin - 1024;
        int stages = (int)(budget / (kBulkWarps * stage_stride));
        if (stages > kMaxStages) stages = kMaxStages;
        if (stages < 2) return MW_ERR_INVALID_ARG;
        a.stages = stages;
        k_copy_bulk<<<ctx->sm_count, kBulkWarps * 32, (size_t)(kBulkWarps * stages * stage_stride), st>>>(a);
    }
    ctx->launches += 1;
    return cudaGetLastError() == cudaSuccess ? MW_OK : MW_ERR_CUDA;
}
