// Row-copy engine: every data-movement step of the path (pack in either layout, deliver in either
// layout, the AllGather forms) is "read a row once, write it to n destinations", with n and the
// destination addresses given by the plan.  (Paper: Section 5.2 step 1, loading the send buffer;
// Section 4.1 steps 3-5 and Section 4.3.3, the relay replicating a payload to every destination
// named by its bitmap.)
//
// k_copy_rows (the default): an ordinary grid with one block per (row, piece of at most 512 16-byte vectors);
//                 a thread loads its vectors once and stores them to every destination of the row.  The deliver
//                 from a MultiWrite send buffer walks the rows from the last to the first and streams its stores,
//                 so that the send rows the pack launch just wrote are read from L2.
// Behind MW_FLAG_COPY_BULK: a persistent grid of one block per SM, one pipeline per warp, work item = (row, chunk
// of at most 7168 bytes), claimed through a ticket counter.
//   k_copy_bulk   bulk asynchronous copies global -> shared (completion counted on an mbarrier),
//                 several stages deep, then one shared -> global bulk copy per destination, issued
//                 by different lanes.
// Measured on B200 (4096 rows of 14336 bytes, 7.7 copies each): deliver 75 us with k_copy_rows after a pack
// launch (6.8 TB/s), 88 us with k_copy_bulk.
#include "mw_internal.cuh"

namespace {

constexpr int kMaxBulkWarps = 8;       // pipelines per block (one per warp)
constexpr int kMaxStages = 8;
constexpr int64_t kMaxChunk = 7168;    // bytes per work item: 4 warps x 8 stages x 7 KB fill the 224 KB a block may use

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, int count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Polls with a suspend-time hint of 1 us; false after `limit` polls.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, int limit)
{
    const uint32_t addr = smem_u32(bar);
    for (int i = 0; i < limit; ++i) {
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
__device__ __forceinline__ uint4 ld_stream(const uint8_t *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void flag_error(const mw_copy_args &a, int err) { atomicCAS(&a.totals->status, 0, err); }

// ---- the work list -------------------------------------------------------------------------
__device__ __forceinline__ int64_t n_rows(const mw_copy_args &a)
{
    if (a.rows_from == 1) return a.totals->T_nonempty;
    if (a.rows_from == 2) return a.totals->total_dest;
    return a.host_rows;
}

__device__ __forceinline__ const uint8_t *src_row(const mw_copy_args &a, int64_t row, int mode)
{
    switch (mode) {
    case MW_CP_PACK_MW:
    case MW_CP_DISPATCH_MW:
    case MW_CP_DISPATCH_UC: return a.src + (int64_t)a.src_index[row] * a.row_bytes;
    case MW_CP_SCATTER: return a.src + (a.src_index ? (int64_t)a.src_index[row] : row) * a.row_bytes;
    case MW_CP_AG_DELIVER_UC: {
        const int64_t i = row / a.dst_count, d = row % a.dst_count;
        return (a.dst_begin + d == i) ? a.src2 + i * a.row_bytes : a.src + row * a.row_bytes;
    }
    case MW_CP_PAIR_DIRECT:
    case MW_CP_PAIR_SEND: return a.src + row * a.shard_bytes + a.seg_off;
    case MW_CP_PAIR_FORWARD: {
        const int64_t r = row / (a.pair_n - 1), k = row % (a.pair_n - 1);
        const int64_t partner = (r + a.pair_n) % a.R;
        return a.src + (partner * a.pair_copies + (a.pair_copies == 1 ? 0 : k)) * a.row_bytes;
    }
    default: return a.src + row * a.row_bytes;
    }
}

// Rows whose source is found through an index array: the index is loaded one item ahead of its use.
__device__ __forceinline__ bool src_is_indexed(const mw_copy_args &a, int mode)
{
    return mode == MW_CP_PACK_MW || mode == MW_CP_DISPATCH_MW || mode == MW_CP_DISPATCH_UC || (mode == MW_CP_SCATTER && a.src_index);
}
__device__ __forceinline__ bool src_is_indexed(const mw_copy_args &a) { return src_is_indexed(a, a.mode); }
__device__ __forceinline__ const uint8_t *src_row_with(const mw_copy_args &a, int64_t row, int index, int mode)
{
    return src_is_indexed(a, mode) ? a.src + (int64_t)index * a.row_bytes : src_row(a, row, mode);
}
__device__ __forceinline__ const uint8_t *src_row_with(const mw_copy_args &a, int64_t row, int index)
{
    return src_row_with(a, row, index, a.mode);
}

__device__ __forceinline__ int n_dst(const mw_copy_args &a, int64_t row, int mode)
{
    switch (mode) {
    case MW_CP_SCATTER: return a.ndst[row];
    case MW_CP_DISPATCH_MW: return a.ndst[row] + 1;
    case MW_CP_DISPATCH_UC: return 2 * a.ndst[row];
    case MW_CP_AG_DELIVER_MW:
    case MW_CP_AG_PACK_UC: return a.dst_count;
    case MW_CP_AG_FUSED_MW: return a.dst_count + 1;
    case MW_CP_AG_FUSED_UC: return 2 * a.dst_count;
    case MW_CP_PAIR_DIRECT: return a.pair_n;
    case MW_CP_PAIR_SEND: return a.pair_copies + 1;
    default: return 1;
    }
}

__device__ __forceinline__ int n_dst(const mw_copy_args &a, int64_t row) { return n_dst(a, row, a.mode); }

// Receive slot of destination q of send row `row` (plan descriptors in plane layout).
// Region r given by its own base address (Section 4.3.2: a write that takes an array of remote buffer addresses).
// The addresses live in device memory, so they are checked here: a null or misaligned one is reported, nothing is written.
__device__ __forceinline__ uint8_t *region_base(const mw_copy_args &a, int r)
{
    uint8_t *base = a.dst_ptrs[r];
    if (!base) { flag_error(a, MW_ERR_INVALID_ARG); return nullptr; }
    if ((uintptr_t)base & 15u) { flag_error(a, MW_ERR_ALIGNMENT); return nullptr; }
    return base;
}

__device__ __forceinline__ uint8_t *scatter_dst(const mw_copy_args &a, int64_t row, int q)
{
    if (a.dst_ptrs) {
        const int r = a.d_rank[q * a.d_stride + row], p = a.d_pos[q * a.d_stride + row];
        if (r < 0) return nullptr;
        if (p >= a.capacity_rows) { flag_error(a, MW_ERR_CAPACITY); return nullptr; }
        uint8_t *base = region_base(a, r);
        return base ? base + (int64_t)p * a.row_bytes : nullptr;
    }
    if (a.dst_stride) {
        const int r = a.d_rank[q * a.d_stride + row], p = a.d_pos[q * a.d_stride + row];
        if (r < 0) return nullptr;
        if (p >= a.capacity_rows) { flag_error(a, MW_ERR_CAPACITY); return nullptr; }
        return a.dst + (int64_t)r * a.dst_stride + (int64_t)p * a.row_bytes;
    }
    const int64_t at = a.d_flat[q * a.d_stride + row];
    if (at < 0) return nullptr;
    if (at >= a.capacity_rows) { flag_error(a, MW_ERR_CAPACITY); return nullptr; }
    return a.dst + at * a.row_bytes;
}

// Destination q of a row; nullptr when the copy must not happen (capacity exceeded -> status, or the
// AllGather copy addressed to the shard's own rank, which is never transmitted).
__device__ __forceinline__ uint8_t *dst_row(const mw_copy_args &a, int64_t row, int q, int mode)
{
    switch (mode) {
    case MW_CP_PACK_MW:
    case MW_CP_AG_PACK_MW:
        if (row >= a.capacity_rows) { flag_error(a, MW_ERR_CAPACITY); return nullptr; }
        return a.dst + row * a.row_bytes;
    case MW_CP_SCATTER: return scatter_dst(a, row, q);
    case MW_CP_DISPATCH_MW:
        if (q > 0) return scatter_dst(a, row, q - 1);
        if (row >= a.capacity2_rows) { flag_error(a, MW_ERR_CAPACITY); return nullptr; }
        return a.dst2 + row * a.row_bytes;
    case MW_CP_DISPATCH_UC: {
        // the unicast send buffer is laid out like the compact receive area: slot = d_flat
        const int n0 = a.ndst[row];
        if (q >= n0) return scatter_dst(a, row, q - n0);
        const int64_t at = a.d_flat[q * a.d_stride + row];
        if (at < 0) return nullptr;
        if (at >= a.capacity2_rows) { flag_error(a, MW_ERR_CAPACITY); return nullptr; }
        return a.dst2 + at * a.row_bytes;
    }
    case MW_CP_DELIVER_UC: {
        if (!a.dst_stride && !a.dst_ptrs) {
            if (row >= a.capacity_rows) { flag_error(a, MW_ERR_CAPACITY); return nullptr; }
            return a.dst + row * a.row_bytes;
        }
        // rank of unicast row `row`: the last r with rank_offsets[r] <= row (binary search, R + 1 entries)
        int lo = 0, hi = a.R;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (a.rank_offsets[mid] <= row) lo = mid; else hi = mid;
        }
        const int64_t p = row - a.rank_offsets[lo];
        if (p >= a.capacity_rows) { flag_error(a, MW_ERR_CAPACITY); return nullptr; }
        if (a.dst_ptrs) {
            uint8_t *base = region_base(a, lo);
            return base ? base + p * a.row_bytes : nullptr;
        }
        return a.dst + (int64_t)lo * a.dst_stride + p * a.row_bytes;
    }
    case MW_CP_AG_DELIVER_MW: return a.dst + (int64_t)q * a.dst_stride + row * a.row_bytes;
    case MW_CP_AG_FUSED_MW:
        if (q == a.dst_count) return a.dst2 + row * a.row_bytes;
        return a.dst + (int64_t)q * a.dst_stride + row * a.row_bytes;
    case MW_CP_AG_FUSED_UC:
        if (q >= a.dst_count) return a.dst + (int64_t)(q - a.dst_count) * a.dst_stride + row * a.row_bytes;
        if (a.dst_begin + q == row) return nullptr;                      // the copy to the shard's own rank is never sent
        return a.dst2 + (row * a.dst_count + q) * a.row_bytes;
    case MW_CP_AG_PACK_UC:
        if (a.dst_begin + q == row) return nullptr;
        return a.dst + (row * a.dst_count + q) * a.row_bytes;
    case MW_CP_AG_DELIVER_UC: {
        const int64_t i = row / a.dst_count, d = row % a.dst_count;
        return a.dst + d * a.dst_stride + i * a.row_bytes;
    }
    // paired AllGather: receive region of rank d holds the n shards of d's domain, shard of rank r at slot r % n
    case MW_CP_PAIR_DIRECT: {
        const int64_t d = (row / a.pair_n) * a.pair_n + q;
        return a.dst + (d * a.pair_n + row % a.pair_n) * a.shard_bytes + a.seg_off;
    }
    case MW_CP_PAIR_SEND: {
        if (q == a.pair_copies) return a.dst2 + (row * a.pair_n + row % a.pair_n) * a.shard_bytes + a.seg_off;   // own copy, local
        const int64_t partner = (row + a.pair_n) % a.R;
        return a.dst + (partner * a.pair_copies + q) * a.row_bytes;
    }
    case MW_CP_PAIR_FORWARD: {
        const int64_t r = row / (a.pair_n - 1), k = row % (a.pair_n - 1);
        const int64_t qd = k < r % a.pair_n ? k : k + 1;                 // k-th member of r's domain other than r
        const int64_t d = (r / a.pair_n) * a.pair_n + qd;
        return a.dst + (d * a.pair_n + r % a.pair_n) * a.shard_bytes + a.seg_off;
    }
    }
    return nullptr;
}

__device__ __forceinline__ uint8_t *dst_row(const mw_copy_args &a, int64_t row, int q) { return dst_row(a, row, q, a.mode); }

__device__ __forceinline__ bool plan_unusable(const mw_copy_args &a)
{
    return a.totals && a.rows_from != 0 && a.totals->status == MW_ERR_TIMEOUT;
}

__device__ __forceinline__ bool writes_send_buffer(const mw_copy_args &a)
{
    return a.mode == MW_CP_PACK_MW || a.mode == MW_CP_AG_PACK_MW || a.keep_in_l2;
}

// The plan's descriptors of a row, as loaded (no arithmetic, no dependent load): the staged kernels
// fetch them one iteration before they are needed, so their latency overlaps the previous item's stores.
struct RawDesc { int x, y, n; };

__device__ __forceinline__ RawDesc fetch_raw(const mw_copy_args &a, int64_t row, int lane)
{
    RawDesc d;
    d.x = -1; d.y = -1; d.n = 1;
    if (a.mode == MW_CP_SCATTER) {
        d.n = a.ndst[row];
        if (lane < a.Kd) {
            if (a.dst_stride || a.dst_ptrs) { d.x = a.d_rank[lane * a.d_stride + row]; d.y = a.d_pos[lane * a.d_stride + row]; }
            else d.x = a.d_flat[lane * a.d_stride + row];
        }
    }
    return d;
}

// Destination `lane` of the row from its raw descriptors (nullptr if none or suppressed); *nd = destinations of the row.
__device__ __forceinline__ uint8_t *resolve_dst(const mw_copy_args &a, int64_t row, int lane, const RawDesc &d, int *nd)
{
    switch (a.mode) {
    case MW_CP_SCATTER: {
        *nd = d.n;
        if (lane >= d.n || d.x < 0) return nullptr;
        if (a.dst_ptrs) {
            if (d.y >= a.capacity_rows) { flag_error(a, MW_ERR_CAPACITY); return nullptr; }
            uint8_t *base = region_base(a, d.x);
            return base ? base + (int64_t)d.y * a.row_bytes : nullptr;
        }
        if (a.dst_stride) {
            if (d.y >= a.capacity_rows) { flag_error(a, MW_ERR_CAPACITY); return nullptr; }
            return a.dst + (int64_t)d.x * a.dst_stride + (int64_t)d.y * a.row_bytes;
        }
        if (d.x >= a.capacity_rows) { flag_error(a, MW_ERR_CAPACITY); return nullptr; }
        return a.dst + (int64_t)d.x * a.row_bytes;
    }
    case MW_CP_DELIVER_UC:
        *nd = 1;
        return lane == 0 ? dst_row(a, row, 0) : nullptr;
    default:
        *nd = n_dst(a, row);          // no load involved in the remaining modes
        return lane < *nd ? dst_row(a, row, lane) : nullptr;
    }
}

// ---- work tickets ----------------------------------------------------------------------------
// A warp takes the next `batch` consecutive items with one atomicAdd and asks for its next ticket
// while it still works on the current one, so the atomic's latency is never waited for.  Measured on
// B200: the same stores reach about 7 TB/s when work is handed out on demand and about 6 TB/s with a
// static round-robin split of a persistent grid (SMs do not all see the same memory throughput).
// The first items of every pipeline are assigned statically, one per lane, so that a warp's first
// loads go out in parallel without waiting for a ticket.  The last warp to finish sets both counters
// back to zero for the next launch.
struct TicketSource {
    unsigned int *ticket;
    int64_t items, base;
    int batch;
    int64_t cur, cur_end;
    unsigned int pending;
    // Items below `first_item` were handed out statically (the pipelines' first loads); tickets cover the rest.
    __device__ __forceinline__ void start(unsigned int *t, int64_t n, int b, int64_t first_item)
    {
        ticket = t; items = n; batch = b; base = first_item; cur = cur_end = 0;
        pending = 0;
        if (n > first_item) pending = atomicAdd(ticket, 1u);   // small launches are fully covered by the static part
        else items = 0;
    }
    // Next item of this warp, or -1 when the work list is exhausted (stays -1 afterwards).
    __device__ __forceinline__ int64_t next()
    {
        if (cur == cur_end) {
            const int64_t b0 = base + (int64_t)pending * batch;
            if (b0 >= items) return -1;
            cur = b0;
            cur_end = min(b0 + (int64_t)batch, items);
            pending = atomicAdd(ticket, 1u);      // result is needed only when this batch is used up
        }
        return cur++;
    }
};

__device__ __forceinline__ void tickets_finish(const mw_copy_args &a, int lane, unsigned total_warps, bool used)
{
    if (lane == 0 && used) {
        __threadfence();
        if (atomicAdd(a.work_ctr + 1, 1u) == total_warps - 1u) {
            a.work_ctr[0] = 0;
            a.work_ctr[1] = 0;
            __threadfence();
        }
    }
}

struct ItemGeom { int64_t row, off; uint32_t bytes; };
__device__ __forceinline__ ItemGeom geom(const mw_copy_args &a, int64_t item)
{
    ItemGeom g;
    g.row = item / a.chunks_per_row;
    g.off = (item % a.chunks_per_row) * (int64_t)a.chunk_bytes;
    g.bytes = (uint32_t)min((int64_t)a.chunk_bytes, a.row_bytes - g.off);
    return g;
}

// ---- bulk-copy loads, bulk-copy stores ------------------------------------------------------
__global__ void __launch_bounds__(kMaxBulkWarps * 32, 1) k_copy_bulk(const __grid_constant__ mw_copy_args a)
{
    extern __shared__ __align__(128) uint8_t stage_mem[];
    __shared__ __align__(8) uint64_t bars[kMaxBulkWarps * kMaxStages];
    __shared__ int64_t ring[kMaxBulkWarps * kMaxStages];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nwarps = blockDim.x >> 5;
    const int nst = a.stages;
    const uint32_t stage_stride = ((uint32_t)a.chunk_bytes + 127u) & ~127u;
    uint8_t *stages = stage_mem + (size_t)warp * nst * stage_stride;
    uint64_t *bar = bars + warp * kMaxStages;
    int64_t *held = ring + warp * kMaxStages;
    if (lane == 0)
        for (int s = 0; s < nst; ++s) mbar_init(bar + s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncwarp();
    grid_launch_dependents();
    grid_dependency_wait();
    if (plan_unusable(a)) return;

    const int64_t items = n_rows(a) * a.chunks_per_row;
    const uint64_t policy = writes_send_buffer(a) ? policy_evict_normal() : policy_evict_first();
    auto issue_load = [&](int64_t item, int index, int s) {
        const ItemGeom g = geom(a, item);
        mbar_expect_tx(bar + s, g.bytes + (uint32_t)a.expect_extra);
        bulk_load(stages + (size_t)s * stage_stride, src_row_with(a, g.row, index) + g.off, g.bytes, bar + s);
    };

    // first loads: item (lane * warps of the grid + this warp) goes to stage `lane`, issued by that lane, so a
    // small launch spreads over all warps and a large one starts with every pipeline full
    const int npro = nst - 1;
    const int64_t gw = (int64_t)warp * gridDim.x + blockIdx.x;
    if (lane < nst) {
        const int64_t it = lane < npro ? (int64_t)lane * gridDim.x * nwarps + gw : -1;
        const bool has = it >= 0 && it < items;
        held[lane] = has ? it : -1;
        if (has) issue_load(it, src_is_indexed(a) ? a.src_index[it / a.chunks_per_row] : 0, lane);
    }
    TicketSource src;                 // used by lane 0 only
    int64_t pend_item = -1;           // next item to load (lane 0), chosen one iteration before its load is issued
    int pend_index = 0;
    if (lane == 0) {
        src.start(a.work_ctr, items, a.batch, (int64_t)gridDim.x * nwarps * npro);
        pend_item = src.next();
        if (pend_item >= 0 && src_is_indexed(a)) pend_index = a.src_index[pend_item / a.chunks_per_row];
    }
    __syncwarp();

    RawDesc raw_next = {-1, -1, 0};
    if (held[0] >= 0) raw_next = fetch_raw(a, held[0] / a.chunks_per_row, lane);

    bool ok = true;
    int n = 0;
    for (;; ++n) {
        const int s = n % nst;
        const int64_t item = held[s];
        if (item < 0) break;
        const ItemGeom g = geom(a, item);
        int nd;
        uint8_t *my_dst = resolve_dst(a, g.row, lane, raw_next, &nd);
        {
            const int64_t nitem = held[(n + 1) % nst];
            if (nitem >= 0) raw_next = fetch_raw(a, nitem / a.chunks_per_row, lane);
        }
        if (!mbar_wait(bar + s, (uint32_t)(n / nst) & 1u, a.wait_limit)) { ok = false; break; }
        const uint8_t *stage = stages + (size_t)s * stage_stride;
        if (my_dst) bulk_store(my_dst + g.off, stage, g.bytes, policy);
        for (int q = lane + 32; q < nd; q += 32) {
            uint8_t *d = dst_row(a, g.row, q);
            if (d) bulk_store(d + g.off, stage, g.bytes, policy);
        }
        bulk_commit();
        // the stage that item n-1 used is free once every lane's stores of that item have read it
        bulk_wait_read<1>();
        __syncwarp();
        if (lane == 0) {
            const int sr = (n + nst - 1) % nst;
            held[sr] = pend_item;
            if (pend_item >= 0) {
                issue_load(pend_item, pend_index, sr);
                pend_item = src.next();
                if (pend_item >= 0 && src_is_indexed(a)) pend_index = a.src_index[pend_item / a.chunks_per_row];
            }
        }
        __syncwarp();
    }
    if (!ok) {
        if (lane == 0) flag_error(a, MW_ERR_TIMEOUT);
        for (int m = n + 1; m < n + nst - 1; ++m)      // stages n+1 .. n+nst-2 hold loads issued ahead
            if (held[m % nst] >= 0) mbar_wait(bar + (m % nst), (uint32_t)(m / nst) & 1u, a.wait_limit);
    }
    bulk_wait_all();
    tickets_finish(a, lane, (unsigned)(gridDim.x * nwarps), items > (int64_t)gridDim.x * nwarps * npro);
}

// ---- one block per (row, piece): plain loads and stores, ordinary grid ---------------------------
// The default.  A piece is blockDim.x * V 16-byte vectors (at most kRowsMaxVecs); a thread loads V vectors of
// the piece once and stores them to every destination of the row.  With many more blocks than SMs the hardware
// scheduler balances the load and hides each block's start-up behind its neighbours.  Blocks live for a few
// microseconds, so every dependent step before the first store counts: measured on B200 (4096 rows of 14336
// bytes, 7.7 copies each) a 64-bit division, inline-asm stores the compiler cannot schedule around, or one more
// dependent round trip to L2 each cost 2 to 12 % of the run time.
constexpr int kRowsMaxVecs = 512;
constexpr int kRowsDstBatch = 64;

__host__ __device__ constexpr bool mode_is_one_to_one(int mode)
{
    return mode == MW_CP_PACK_MW || mode == MW_CP_DELIVER_UC || mode == MW_CP_AG_PACK_MW || mode == MW_CP_AG_DELIVER_UC ||
           mode == MW_CP_PAIR_FORWARD;
}

template <int V, int MODE, bool kAfterPack = false>
__global__ void __launch_bounds__(kRowsMaxVecs) k_copy_rows(const __grid_constant__ mw_copy_args a)
{
    __shared__ uint8_t *dst_s[kRowsDstBatch];
    grid_launch_dependents();
    grid_dependency_wait();
    const int tid = threadIdx.x;
    // Deliver walks the send rows from the last to the first and writes with streaming (evict-first) stores.
    // The rows come out of the pack launch in ascending order, so the most recently packed ones are still in
    // L2; taking them first, with stores that do not displace them, turns most send-row reads into L2 hits and
    // leaves DRAM an almost pure write stream.  Measured on B200, deliver right after pack: 4096 rows of
    // 14336 bytes (59 MB of send rows) 85 -> 74 us; 8192 rows (117 MB, about the size of L2) 164 -> 154 us.
    // With send rows that are not in L2 the streaming stores cost 3 to 4 % instead, so only the deliver from a
    // MultiWrite send buffer is launched with kAfterPack (the unicast pack scatters rows of x, which come from DRAM).
    const unsigned blk = (kAfterPack && MODE == MW_CP_SCATTER) ? gridDim.x - 1 - blockIdx.x : blockIdx.x;
    // 32-bit on purpose: the division is on the way to the first load
    const int row = blk / a.chunks_per_row, piece = blk % a.chunks_per_row;
    // what decides whether the block has work is loaded together and looked at afterwards: one round trip
    // (all of it lies inside the plan's arrays for any row below the launch bound)
    const int status = (a.totals && a.rows_from != 0) ? a.totals->status : MW_OK;
    const int64_t rows = n_rows(a);
    const int nd = n_dst(a, row, MODE);
    const int index = src_is_indexed(a, MODE) ? a.src_index[row] : 0;
    if (status == MW_ERR_TIMEOUT || row >= rows) return;
    const uint8_t *src = src_row_with(a, row, index, MODE);
    const int64_t off = (int64_t)piece * a.chunk_bytes + tid * 16;      // vector k of this thread: off + k * blockDim.x * 16
    const int64_t step = (int64_t)blockDim.x * 16;
    uint4 v[V];
#pragma unroll
    for (int k = 0; k < V; ++k)
        if (off + k * step < a.row_bytes) v[k] = ld_stream(src + off + k * step);
    if constexpr (mode_is_one_to_one(MODE)) {
        uint8_t *d = dst_row(a, row, 0, MODE);
        if (!d) return;
#pragma unroll
        for (int k = 0; k < V; ++k)
            if (off + k * step < a.row_bytes) *(uint4 *)(d + off + k * step) = v[k];
    } else {
        for (int qb = 0; qb < nd; qb += kRowsDstBatch) {
            const int nq = min(kRowsDstBatch, nd - qb);
            if (qb) __syncthreads();
            if (tid < nq) dst_s[tid] = dst_row(a, row, qb + tid, MODE);
            __syncthreads();
            for (int q = 0; q < nq; ++q) {
                uint8_t *d = dst_s[q];
                if (!d) continue;
#pragma unroll
                for (int k = 0; k < V; ++k)
                    if (off + k * step < a.row_bytes) {
                        // one pass from prefetched rows: the send slot (destination 0) is kept, the receive slots stream
                        if (kAfterPack && (MODE != MW_CP_DISPATCH_MW || qb + q > 0)) __stcs((uint4 *)(d + off + k * step), v[k]);
                        else *(uint4 *)(d + off + k * step) = v[k];
                    }
            }
        }
    }
}

// One instantiation per mode, so that the mode switches of the work list fold away.
template <int V, int MODE, bool AFTER_PACK = false>
cudaError_t rows_launch(dim3 grid, dim3 block, cudaStream_t st, bool overlap, const mw_copy_args &a)
{
    return mw_launch(k_copy_rows<V, MODE, AFTER_PACK>, grid, block, 0, st, overlap, a);
}

struct CopyShape { int warps; int stages; int64_t chunk; int batch; };

// Rows longer than kMaxChunk are cut into equal pieces (multiples of 16 bytes); when that still leaves
// fewer items than about two per warp (AllGather shards, decode batches) the pieces are halved further.
int64_t choose_chunk(int64_t row_bytes, int64_t est_rows, int64_t all_warps)
{
    const int64_t pieces = (row_bytes + kMaxChunk - 1) / kMaxChunk;
    int64_t chunk = ((row_bytes + pieces - 1) / pieces + 15) & ~(int64_t)15;
    while (chunk > 2048 && est_rows * ((row_bytes + chunk - 1) / chunk) < 2 * all_warps) chunk = ((chunk / 2) + 15) & ~(int64_t)15;
    return chunk;
}

// Work-item size, pipelines per block, pipeline depth and ticket size for the staged kernels.  Measured
// on B200 (4096 rows of 14336 bytes, 7.7 copies each): depth matters more than item size; 4 warps x 8
// stages of half rows beat 4 warps x 4 stages of whole rows by 4.5 %.
CopyShape choose_shape(const mw_ctx *ctx, const mw_copy_args &a, int64_t est_rows)
{
    CopyShape s;
    // one-to-one copies (pack, unicast deliver) are bound by how many loads are in flight: more, shallower
    // pipelines; fan-out copies are bound by the stores: fewer, deeper pipelines
    const bool one_to_one = a.mode == MW_CP_PACK_MW || a.mode == MW_CP_DELIVER_UC || a.mode == MW_CP_AG_PACK_MW ||
                            a.mode == MW_CP_AG_DELIVER_UC;
    s.warps = one_to_one ? 8 : 4;
    s.chunk = choose_chunk(a.row_bytes, est_rows, (int64_t)ctx->sm_count * s.warps);
    const int64_t stage_stride = (s.chunk + 127) & ~(int64_t)127;
    const int64_t budget = ctx->max_smem_optin - 2048;
    s.stages = (int)(budget / (s.warps * stage_stride));
    if (s.stages > kMaxStages) s.stages = kMaxStages;
    // items per ticket: about seven tickets per warp, at least two items (keeps the single-address
    // atomic far from saturation), at most 32
    const int64_t est_items = est_rows * ((a.row_bytes + s.chunk - 1) / s.chunk);
    const int64_t batch = est_items / ((int64_t)ctx->sm_count * s.warps * 7);
    s.batch = (int)(batch < 2 ? 2 : batch > 32 ? 32 : batch);
    return s;
}

}  // namespace

int mw_copy_smem_setup(mw_ctx *ctx)
{
    const int limit = ctx->max_smem_optin - 2048;
    if (cudaFuncSetAttribute(k_copy_bulk, cudaFuncAttributeMaxDynamicSharedMemorySize, limit) != cudaSuccess) return MW_ERR_CUDA;
    return MW_OK;
}

// Default: one block per (row, piece) on an ordinary grid.  With MW_FLAG_COPY_BULK (or a launch whose row bound is
// loose, or a grid too large for 32-bit block indices): chooses the work-item size and the pipeline shape and launches
// the persistent bulk-copy grid.
int mw_copy_launch(mw_ctx *ctx, mw_copy_args a, cudaStream_t st)
{
    const bool overlap = !(ctx->cfg.flags & MW_FLAG_NO_OVERLAP);
    const int64_t est_rows = a.host_rows >= 0 ? a.host_rows : 0;
    cudaError_t err;
    int64_t pieces = 0;
    int threads = 0;
    // one-to-one copies need more loads in flight per thread; fan-out copies are bound by their stores
    const int V = mode_is_one_to_one(a.mode) ? 2 : 1;
    if (!(ctx->cfg.flags & MW_FLAG_COPY_BULK) && a.host_rows >= 0 && !a.loose_bound) {
        // near-equal pieces of at most kRowsMaxVecs vectors; smaller ones while the grid would leave SMs idle
        const int64_t vecs = a.row_bytes / 16;
        pieces = (vecs + kRowsMaxVecs - 1) / kRowsMaxVecs;
        while (a.host_rows * pieces < 4 * (int64_t)ctx->sm_count && (vecs + pieces - 1) / pieces > 128) pieces *= 2;
        const int64_t piece_vecs = (vecs + pieces - 1) / pieces;
        threads = (int)(((piece_vecs + V - 1) / V + 31) / 32 * 32);
        if (threads < kRowsDstBatch) threads = kRowsDstBatch;
        a.chunk_bytes = threads * V * 16;
        pieces = (a.row_bytes + a.chunk_bytes - 1) / a.chunk_bytes;
        a.chunks_per_row = (int32_t)pieces;
    }
    if (pieces > 0 && a.host_rows * pieces <= 0x7fffffff) {
        if (a.host_rows == 0) return MW_OK;
        const dim3 grid((unsigned)(a.host_rows * pieces));
        const dim3 block(threads);
        switch (a.mode) {
        case MW_CP_PACK_MW: err = rows_launch<2, MW_CP_PACK_MW>(grid, block, st, overlap, a); break;
        case MW_CP_SCATTER:
            // no source index: the rows are a send buffer, packed just before
            err = (a.src_index || a.src_not_recent) ? rows_launch<1, MW_CP_SCATTER>(grid, block, st, overlap, a)
                                                    : rows_launch<1, MW_CP_SCATTER, true>(grid, block, st, overlap, a);
            break;
        case MW_CP_DELIVER_UC: err = rows_launch<2, MW_CP_DELIVER_UC>(grid, block, st, overlap, a); break;
        case MW_CP_PAIR_DIRECT: err = rows_launch<1, MW_CP_PAIR_DIRECT>(grid, block, st, overlap, a); break;
        case MW_CP_PAIR_SEND: err = rows_launch<1, MW_CP_PAIR_SEND>(grid, block, st, overlap, a); break;
        case MW_CP_PAIR_FORWARD: err = rows_launch<2, MW_CP_PAIR_FORWARD>(grid, block, st, overlap, a); break;
        case MW_CP_DISPATCH_MW:
            err = a.src_in_l2 ? rows_launch<1, MW_CP_DISPATCH_MW, true>(grid, block, st, overlap, a)
                              : rows_launch<1, MW_CP_DISPATCH_MW>(grid, block, st, overlap, a);
            break;
        case MW_CP_DISPATCH_UC: err = rows_launch<1, MW_CP_DISPATCH_UC>(grid, block, st, overlap, a); break;
        case MW_CP_AG_FUSED_MW: err = rows_launch<1, MW_CP_AG_FUSED_MW>(grid, block, st, overlap, a); break;
        case MW_CP_AG_FUSED_UC: err = rows_launch<1, MW_CP_AG_FUSED_UC>(grid, block, st, overlap, a); break;
        default: return MW_ERR_INVALID_ARG;     // the two-launch AllGather modes only run with MW_FLAG_COPY_BULK
        }
    } else {
        const CopyShape s = choose_shape(ctx, a, est_rows);
        if (s.stages < 2 || s.warps < 1 || s.warps > kMaxBulkWarps || s.chunk > kMaxChunk) return MW_ERR_INVALID_ARG;
        const int64_t stage_stride = (s.chunk + 127) & ~(int64_t)127;
        a.chunk_bytes = (int32_t)s.chunk;
        a.chunks_per_row = (int32_t)((a.row_bytes + s.chunk - 1) / s.chunk);
        a.stages = s.stages;
        a.batch = s.batch;
        a.work_ctr = ctx->d.copy_ctr;
        a.wait_limit = ctx->copy_wait_limit;
        // test hook: every load is announced 16 bytes larger than it is, so no stage ever completes and the
        // bounded wait runs out (the loads themselves are untouched and land as usual)
        a.expect_extra = (ctx->test_skew & MW_TEST_SKEW_BULK_LOAD) ? 16 : 0;
        ctx->test_skew &= ~(uint32_t)MW_TEST_SKEW_BULK_LOAD;
        const size_t smem = (size_t)(s.warps * s.stages * stage_stride);
        err = mw_launch(k_copy_bulk, dim3(ctx->sm_count), dim3(s.warps * 32), smem, st, overlap, a);
    }
    ctx->launches += 1;
    if (err != cudaSuccess) { cudaGetLastError(); return MW_ERR_CUDA; }
    return MW_OK;
}
