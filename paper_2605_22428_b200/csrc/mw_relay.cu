// Two-level (relayed) MultiWrite dispatch (paper: Section 3.2, Section 4.1 "Local forwarding table",
// Section 4.3.3).  Declared and documented in include/mw.h.
//
// First level = the ordinary plan / pack / deliver machinery run on next-hop sets: the expert->rank
// table is replaced by expert->next-hop, so "one copy per distinct next hop" is just the per-rank
// dedup of the flat path.  Second level = one more launch of the row-copy engine: its source rows are
// the rows of the hop area, its descriptors (built by k_relay_desc) list, for each hop row, the final
// destinations whose next hop that is, with the slots of the flat plan.
#include <new>
#include <string.h>

#include "mw_internal.cuh"

struct mw_relay {
    mw_ctx *hop, *flat;
    int P;                       // ranks per server
    int64_t rows_max;            // max_tokens * Kd: most rows the hop area can hold
    int32_t *e2hop;              // [E] next hop of every expert's rank
    int32_t *s2_ndst;            // [rows_max] final destinations of hop row q
    int32_t *s2_rank, *s2_pos, *s2_flat;   // [Kd, rows_max] their ranks, slots, rows of the compact receive area
    mw_relay_totals *totals;     // device
    void *slab;
    int planned;
};

namespace {

__host__ __device__ inline int next_hop(int r, int src, int P)
{
    return (r / P == src / P) ? r : (r / P) * P + src % P;      // own server: direct; else the same-index rank there
}

__global__ void k_relay_table(const int32_t *e2r, int E, int R, int src, int P, int32_t *e2hop)
{
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= E) return;
    const int r = e2r[e];
    e2hop[e] = (r < 0 || r >= R) ? r : next_hop(r, src, P);     // out-of-range entries stay so: the plan reports them
}

struct DescArgs {
    int T, Kd, R, src, P;
    int64_t rows_max, row_bytes;
    const int32_t *hop_rank_tokens, *hop_rank_offsets;
    const int32_t *flat_dest_rank, *flat_dest_pos, *flat_rank_offsets;
    const mw_totals *hop_totals, *flat_totals;
    int32_t *s2_ndst, *s2_rank, *s2_pos, *s2_flat;
    mw_relay_totals *totals;
};

// One thread per row of the hop area (rows of one hop are consecutive, so the plane stores of a warp are
// coalesced): the row's token comes from the first-level plan's rank_tokens, its hop from a binary search in the
// hop offsets, and the final destinations behind that hop from the flat plan's (rank, slot) pairs of the token.
__global__ void __launch_bounds__(256) k_relay_desc(DescArgs a)
{
    const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    long long direct = 0, inter_mw = 0, inter_uc = 0, forward = 0, hop_rows = 0, delivered = 0;
    if (q < a.hop_totals->total_dest) {
        int lo = 0, hi = a.R;                                  // hop h: the last rank with hop_rank_offsets[h] <= q
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (a.hop_rank_offsets[mid] <= q) lo = mid; else hi = mid;
        }
        const int h = lo;
        const int tok = a.hop_rank_tokens[q];
        const int32_t *fr = a.flat_dest_rank + (int64_t)tok * a.Kd, *fp = a.flat_dest_pos + (int64_t)tok * a.Kd;
        const bool remote = h / a.P != a.src / a.P;
        hop_rows = 1;
        inter_mw = remote;
        int n = 0;
        for (int i = 0; i < a.Kd; ++i) {
            const int r = fr[i];
            if (r < 0) break;
            if (next_hop(r, a.src, a.P) != h) continue;
            a.s2_rank[(int64_t)n * a.rows_max + q] = r;
            a.s2_pos[(int64_t)n * a.rows_max + q] = fp[i];
            a.s2_flat[(int64_t)n * a.rows_max + q] = a.flat_rank_offsets[r] + fp[i];
            ++n;
            ++delivered;
            if (remote) { ++inter_uc; forward += (r != h); }
            else direct += (r != a.src);
        }
        a.s2_ndst[q] = n;
        for (int i = n; i < a.Kd; ++i) {
            a.s2_rank[(int64_t)i * a.rows_max + q] = -1;
            a.s2_pos[(int64_t)i * a.rows_max + q] = -1;
            a.s2_flat[(int64_t)i * a.rows_max + q] = -1;
        }
    }
    // block totals -> device totals (integer sums: independent of the order of the atomics)
    long long v[6] = {hop_rows, delivered, direct, inter_mw, inter_uc, forward};
#pragma unroll
    for (int k = 0; k < 6; ++k)
        for (int o = 16; o > 0; o >>= 1) v[k] += __shfl_down_sync(0xffffffffu, v[k], o);
    if ((threadIdx.x & 31) == 0) {
        unsigned long long *out = (unsigned long long *)a.totals;
        if (v[0]) atomicAdd(out + 0, (unsigned long long)v[0]);
        if (v[1]) atomicAdd(out + 1, (unsigned long long)v[1]);
        if (v[2]) atomicAdd(out + 2, (unsigned long long)(v[2] * a.row_bytes));
        if (v[3]) atomicAdd(out + 3, (unsigned long long)(v[3] * a.row_bytes));
        if (v[4]) atomicAdd(out + 4, (unsigned long long)(v[4] * a.row_bytes));
        if (v[5]) atomicAdd(out + 5, (unsigned long long)(v[5] * a.row_bytes));
    }
    if (q == 0) {                                              // thread 0 forwards the plans' status
        const int s = a.flat_totals->status ? a.flat_totals->status : a.hop_totals->status;
        if (s) atomicCAS(&a.totals->status, 0, s);
    }
}

inline bool aligned16(const void *p) { return ((uintptr_t)p & 15u) == 0; }
inline size_t round256(size_t n) { return (n + 255) & ~(size_t)255; }

}  // namespace

extern "C" {

int mw_relay_create(mw_relay **out, const mw_config *cfg, int32_t ranks_per_server)
{
    if (!out) return MW_ERR_INVALID_ARG;
    *out = nullptr;
    if (!cfg || ranks_per_server < 1 || cfg->R < 1 || cfg->R % ranks_per_server || cfg->src_rank < 0 || cfg->src_rank >= cfg->R)
        return MW_ERR_INVALID_ARG;
    mw_relay *r = new (std::nothrow) mw_relay();
    if (!r) return MW_ERR_INVALID_ARG;
    memset(r, 0, sizeof(*r));
    r->P = ranks_per_server;
    mw_config inner = *cfg;
    inner.flags &= ~MW_FLAG_HOST_STAGING;
    int rc = mw_create(&r->hop, &inner);
    if (rc == MW_OK) rc = mw_create(&r->flat, &inner);
    if (rc == MW_OK) {
        const size_t Kd = (size_t)r->hop->Kd, rows = (size_t)cfg->max_tokens * Kd;
        r->rows_max = (int64_t)rows;
        const size_t b_tab = round256((size_t)cfg->E * 4), b_n = round256(rows * 4), b_plane = round256(rows * Kd * 4);
        const size_t bytes = b_tab + b_n + 3 * b_plane + 256;
        if (cudaMalloc(&r->slab, bytes) != cudaSuccess) { cudaGetLastError(); rc = MW_ERR_CUDA; }
        else {
            uint8_t *p = (uint8_t *)r->slab;
            r->e2hop = (int32_t *)p; p += b_tab;
            r->s2_ndst = (int32_t *)p; p += b_n;
            r->s2_rank = (int32_t *)p; p += b_plane;
            r->s2_pos = (int32_t *)p; p += b_plane;
            r->s2_flat = (int32_t *)p; p += b_plane;
            r->totals = (mw_relay_totals *)p;
            if (cudaMemset(r->slab, 0, bytes) != cudaSuccess) rc = MW_ERR_CUDA;
        }
    }
    if (rc != MW_OK) { mw_relay_destroy(r); return rc; }
    *out = r;
    return MW_OK;
}

int mw_relay_destroy(mw_relay *relay)
{
    if (!relay) return MW_OK;
    int rc = MW_OK;
    if (relay->hop) { cudaSetDevice(relay->hop->cfg.device); cudaDeviceSynchronize(); }
    if (relay->slab && cudaFree(relay->slab) != cudaSuccess) rc = MW_ERR_CUDA;
    if (relay->hop && mw_destroy(relay->hop) != MW_OK) rc = MW_ERR_CUDA;
    if (relay->flat && mw_destroy(relay->flat) != MW_OK) rc = MW_ERR_CUDA;
    delete relay;
    return rc;
}

int mw_relay_contexts(mw_relay *relay, mw_ctx **hop_ctx, mw_ctx **flat_ctx)
{
    if (!relay) return MW_ERR_INVALID_ARG;
    if (hop_ctx) *hop_ctx = relay->hop;
    if (flat_ctx) *flat_ctx = relay->flat;
    return MW_OK;
}

int mw_relay_plan(mw_relay *relay, const int32_t *topk_ids, const int32_t *expert_to_rank, int32_t T, void *stream)
{
    if (!relay || !expert_to_rank || T < 0 || T > relay->hop->cfg.max_tokens || (T > 0 && !topk_ids)) return MW_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const mw_config &c = relay->hop->cfg;
    k_relay_table<<<(c.E + 255) / 256, 256, 0, st>>>(expert_to_rank, c.E, c.R, c.src_rank, relay->P, relay->e2hop);
    int rc = mw_plan(relay->hop, topk_ids, relay->e2hop, T, nullptr, stream);
    if (rc == MW_OK) rc = mw_plan(relay->flat, topk_ids, expert_to_rank, T, nullptr, stream);
    if (rc != MW_OK) return rc;
    if (cudaMemsetAsync(relay->totals, 0, sizeof(mw_relay_totals), st) != cudaSuccess) return MW_ERR_CUDA;
    DescArgs a;
    a.T = T; a.Kd = relay->hop->Kd; a.R = c.R; a.src = c.src_rank; a.P = relay->P;
    a.rows_max = relay->rows_max; a.row_bytes = c.row_bytes;
    a.hop_rank_tokens = relay->hop->d.rank_tokens;
    a.hop_rank_offsets = relay->hop->d.rank_offsets;
    a.flat_dest_rank = relay->flat->d.dest_rank; a.flat_dest_pos = relay->flat->d.dest_pos;
    a.flat_rank_offsets = relay->flat->d.rank_offsets;
    a.hop_totals = relay->hop->d.totals; a.flat_totals = relay->flat->d.totals;
    a.s2_ndst = relay->s2_ndst; a.s2_rank = relay->s2_rank; a.s2_pos = relay->s2_pos; a.s2_flat = relay->s2_flat;
    a.totals = relay->totals;
    // one thread per possible hop row (T * Kd bounds their number); at least one block forwards the plans' status
    const int64_t rows_bound = (int64_t)T * a.Kd;
    k_relay_desc<<<(unsigned)(rows_bound > 0 ? (rows_bound + 255) / 256 : 1), 256, 0, st>>>(a);
    relay->hop->launches += 2;
    relay->planned = 1;
    return cudaGetLastError() == cudaSuccess ? MW_OK : MW_ERR_CUDA;
}

int mw_relay_get_totals(mw_relay *relay, mw_relay_totals *host_out, void *stream)
{
    if (!relay || !host_out) return MW_ERR_INVALID_ARG;
    if (!relay->planned) return MW_ERR_NO_PLAN;
    cudaStream_t st = (cudaStream_t)stream;
    mw_totals hop;
    if (cudaMemcpyAsync(host_out, relay->totals, sizeof(*host_out), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaMemcpyAsync(&hop, relay->hop->d.totals, sizeof(hop), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return MW_ERR_CUDA;
    if (host_out->status == MW_OK) host_out->status = hop.status;     // capacity errors of the dispatch land in the hop plan's status
    return MW_OK;
}

int mw_relay_dispatch(mw_relay *relay, const void *x, void *send_buf, int64_t send_capacity_rows, void *hop_buf,
                      int64_t hop_capacity_rows, void *recv_base, int64_t recv_stride_bytes, int64_t recv_capacity_rows,
                      void *stream)
{
    if (!relay || !x || !send_buf || !hop_buf || !recv_base || send_capacity_rows < 0 || hop_capacity_rows < 0 ||
        recv_stride_bytes < 0 || recv_capacity_rows < 0)
        return MW_ERR_INVALID_ARG;
    if (!relay->planned) return MW_ERR_NO_PLAN;
    if (!aligned16(x) || !aligned16(send_buf) || !aligned16(hop_buf) || !aligned16(recv_base) || recv_stride_bytes % 16)
        return MW_ERR_ALIGNMENT;
    mw_ctx *hop = relay->hop;
    if (recv_stride_bytes && recv_capacity_rows * hop->cfg.row_bytes > recv_stride_bytes) return MW_ERR_CAPACITY;
    // first level: each row once per group of identical next-hop set, one copy per next hop
    int rc = mw_dispatch(hop, x, MW_LAYOUT_MULTIWRITE, send_buf, send_capacity_rows, hop_buf, 0, hop_capacity_rows, stream);
    if (rc != MW_OK) return rc;
    // second level: every hop row to the final destinations behind that hop
    mw_copy_args a;
    memset(&a, 0, sizeof(a));
    a.mode = MW_CP_SCATTER;
    a.src = (const uint8_t *)hop_buf;
    a.dst = (uint8_t *)recv_base;
    a.row_bytes = hop->cfg.row_bytes;
    a.dst_stride = recv_stride_bytes;
    a.capacity_rows = recv_capacity_rows;
    a.rows_from = 2;                                      // rows of the hop area = total_dest of the first-level plan
    a.loose_bound = 1;                                    // T * Kd is far above the hop rows (70 % on the prefill shape)
    a.host_rows = (int64_t)hop->planned_T * hop->Kd;      // estimate for the chunking heuristic
    a.Kd = hop->Kd; a.R = hop->cfg.R;
    a.ndst = relay->s2_ndst;
    a.d_rank = relay->s2_rank; a.d_pos = relay->s2_pos; a.d_flat = relay->s2_flat;
    a.d_stride = relay->rows_max;
    a.rank_offsets = relay->flat->d.rank_offsets;
    a.totals = hop->d.totals;
    return mw_copy_launch(hop, a, (cudaStream_t)stream);
}

}  // extern "C"
