// C ABI entry points (declared and documented in include/mw.h): argument checks, workspace
// carving, and the launch sequences.  No step of the path runs on the host.
#include <math.h>
#include <new>
#include <stdlib.h>
#include <string.h>

#include "mw_internal.cuh"

namespace {

inline bool aligned16(const void *p) { return ((uintptr_t)p & 15u) == 0; }
inline size_t round256(size_t n) { return (n + 255) & ~(size_t)255; }

struct Carver {
    uint8_t *base;
    size_t used;
    template <class T> T *take(size_t count)
    {
        T *p = base ? (T *)(base + used) : nullptr;
        used += round256(count * sizeof(T));
        return p;
    }
};

// The arrays of one plan slot: what a plan writes for the data path to read (and its own per-token values).
void carve_slot(mw_ctx *c, Carver &k, mw_dev &d)
{
    const size_t Tm = (size_t)c->cfg.max_tokens, W = (size_t)c->W, Kd = (size_t)c->Kd, R = (size_t)c->cfg.R;
    d.token_mask = k.take<uint64_t>(Tm * W);
    d.token_ndest = k.take<int32_t>(Tm);
    d.token_group = k.take<int32_t>(Tm);
    d.token_mw_row = k.take<int32_t>(Tm);
    d.mw_row_token = k.take<int32_t>(Tm);
    d.group_offsets = k.take<int32_t>(Tm + 1);
    d.group_mask = k.take<uint64_t>(Tm * W);
    d.rank_offsets = k.take<int32_t>(R + 1);
    d.rank_tokens = k.take<int32_t>(Tm * Kd);
    d.dest_rank = k.take<int32_t>(Tm * Kd);
    d.dest_pos = k.take<int32_t>(Tm * Kd);
    d.totals = k.take<mw_totals>(1);
    d.token_slot = k.take<int32_t>(Tm);
    d.token_leader = k.take<int32_t>(Tm);
    d.token_gcount = k.take<int32_t>(Tm);
    d.gid_at = k.take<int32_t>(Tm);
    d.goff_at = k.take<int32_t>(Tm);
    d.row_ndest = k.take<int32_t>(Tm);
    d.row_dest_rank = k.take<int32_t>(Tm * Kd);
    d.row_dest_pos = k.take<int32_t>(Tm * Kd);
    d.row_dest_flat = k.take<int32_t>(Tm * Kd);
}

// Lays the workspace out inside one slab; with base == nullptr it only measures.  Two plan slots, then the arrays
// derived from the current plan on the caller's stream, then the scratch all plans share (plans are ordered
// among themselves, so one copy is enough); mw_reset re-initialises the scratch part only.
size_t carve(mw_ctx *c, uint8_t *base)
{
    Carver k{base, 0};
    const size_t Tm = (size_t)c->cfg.max_tokens, Kd = (size_t)c->Kd, R = (size_t)c->cfg.R;
    mw_dev &d = c->d;
    carve_slot(c, k, d);
    carve_slot(c, k, c->other.d);
    d.gm_rank = k.take<int32_t>(Tm * Kd);
    d.gm_offset = k.take<int32_t>(Tm * Kd);
    d.dest_pos_gm = k.take<int32_t>(Tm * Kd);
    d.row_dest_pos_gm = k.take<int32_t>(Tm * Kd);
    d.row_dest_flat_gm = k.take<int32_t>(Tm * Kd);
    d.gm_tile_sum = k.take<int32_t>((size_t)c->max_tiles * R);
    {
        const size_t n = (size_t)c->max_tiles * (size_t)c->cfg.E;     // beyond 256 MB the expert index is not offered
        d.ex_tile_cnt = n * sizeof(int32_t) <= ((size_t)256 << 20) ? k.take<int32_t>(n) : nullptr;
    }
    c->scratch_begin = base ? base + k.used : nullptr;
    const size_t scratch_from = k.used;
    d.slot_key = k.take<unsigned long long>((size_t)c->HS);
    d.slot_leader = k.take<int32_t>((size_t)c->HS);
    d.slot_count = k.take<int32_t>((size_t)c->HS);
    d.tile_state = k.take<unsigned long long>((size_t)c->max_tiles * (size_t)c->NC);
    d.tile_agg = k.take<unsigned long long>((size_t)c->max_tiles);
    d.ticket = k.take<unsigned int>(1);
    d.gbar = k.take<unsigned int>(1);
    d.copy_ctr = k.take<unsigned int>(2);
    d.acc = k.take<mw_acc>(2);
    d.gave_up = k.take<unsigned int>(1);
    d.gm_tile_rec = k.take<unsigned long long>((size_t)32 * R);
    d.plan_state = k.take<mw_plan_state>(1);
    c->scratch_bytes = k.used - scratch_from;
    {   // the second slot shares everything that is not a plan array
        mw_dev &o = c->other.d;
        o.gm_rank = d.gm_rank; o.gm_offset = d.gm_offset; o.dest_pos_gm = d.dest_pos_gm;
        o.row_dest_pos_gm = d.row_dest_pos_gm; o.row_dest_flat_gm = d.row_dest_flat_gm;
        o.gm_tile_sum = d.gm_tile_sum; o.ex_tile_cnt = d.ex_tile_cnt;
        o.slot_key = d.slot_key; o.slot_leader = d.slot_leader; o.slot_count = d.slot_count;
        o.tile_state = d.tile_state; o.tile_agg = d.tile_agg; o.ticket = d.ticket; o.gbar = d.gbar;
        o.copy_ctr = d.copy_ctr; o.acc = d.acc; o.gave_up = d.gave_up; o.gm_tile_rec = d.gm_tile_rec; o.plan_state = d.plan_state;
    }
    if (c->cfg.flags & MW_FLAG_HOST_STAGING) {
        const size_t B = (size_t)c->cfg.row_bytes;
        c->st_ids = k.take<int32_t>(Tm * (size_t)c->cfg.K);
        c->st_e2r = k.take<int32_t>((size_t)c->cfg.E);
        c->st_x = k.take<uint8_t>(Tm * B);
        c->st_send = k.take<uint8_t>(Tm * Kd * B);  // large enough for the unicast layout
        c->st_recv = k.take<uint8_t>(Tm * Kd * B);
        c->st_recv_rows = (int64_t)(Tm * Kd);
    }
    return k.used;
}

__global__ void k_fill_i32(int32_t *p, int64_t n, int32_t v)
{
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) p[i] = v;
}

inline cudaStream_t as_stream(void *s) { return (cudaStream_t)s; }

int check_layout(int layout) { return (layout == MW_LAYOUT_MULTIWRITE || layout == MW_LAYOUT_UNICAST) ? MW_OK : MW_ERR_INVALID_ARG; }

mw_copy_args base_args(mw_ctx *ctx)
{
    mw_copy_args a;
    memset(&a, 0, sizeof(a));
    a.row_bytes = ctx->cfg.row_bytes;
    a.host_rows = -1;
    a.Kd = ctx->Kd;
    a.R = ctx->cfg.R;
    a.rank_offsets = ctx->d.rank_offsets;
    a.d_stride = ctx->cfg.max_tokens;
    a.totals = ctx->d.totals;
    return a;
}

void fill_view(const mw_ctx *ctx, int32_t T, mw_plan_view *view)
{
    const mw_dev &d = ctx->d;
    view->token_mask = d.token_mask; view->token_ndest = d.token_ndest; view->token_group = d.token_group;
    view->token_mw_row = d.token_mw_row; view->mw_row_token = d.mw_row_token; view->group_offsets = d.group_offsets;
    view->group_mask = d.group_mask; view->rank_offsets = d.rank_offsets; view->rank_tokens = d.rank_tokens;
    view->dest_rank = d.dest_rank; view->dest_pos = d.dest_pos; view->totals = d.totals;
    view->T = T; view->W = ctx->W; view->Kd = ctx->Kd; view->reserved = 0;
}

// Exchanges the current plan slot with the other one (host-side bookkeeping only).
void swap_slots(mw_ctx *ctx)
{
    const mw_slot cur = {ctx->d, ctx->planned_T, ctx->prefetched, ctx->plan_epoch};
    ctx->d = ctx->other.d; ctx->planned_T = ctx->other.planned_T; ctx->prefetched = ctx->other.prefetched;
    ctx->plan_epoch = ctx->other.plan_epoch;
    ctx->other = cur;
}

// Brings the scratch that all plans share (bitmap table, look-back records, counters and running counts, accumulators)
// and the host-side bookkeeping back to their initial state.  The device must be idle as far as this context goes.
int init_scratch(mw_ctx *c)
{
    if (cudaMemset(c->scratch_begin, 0, c->scratch_bytes) != cudaSuccess) return MW_ERR_CUDA;
    k_fill_i32<<<64, 256>>>((int32_t *)c->d.slot_key, 2 * (int64_t)c->HS, -1);   // all ones = empty slot
    k_fill_i32<<<64, 256>>>(c->d.slot_leader, c->HS, 0x7fffffff);                 // no leader
    if (cudaDeviceSynchronize() != cudaSuccess) return MW_ERR_CUDA;
    c->epoch = 0;
    c->planned_T = -1; c->prefetched = nullptr; c->plan_epoch = 0;
    c->other.planned_T = -1; c->other.prefetched = nullptr; c->other.plan_epoch = 0;
    c->next_pending = 0; c->plans_on_side_stream = 0; c->gm_epoch = 0; c->gm_calls = 0;
    c->test_skew = 0; c->poisoned = 0;
    return MW_OK;
}

void release(mw_ctx *c)
{
    if (c->ev_submitted) cudaEventDestroy(c->ev_submitted);
    if (c->ev_planned) cudaEventDestroy(c->ev_planned);
    if (c->plan_stream) cudaStreamDestroy(c->plan_stream);
    if (c->slab) cudaFree(c->slab);
    cudaGetLastError();
    delete c;
}

// A plan launch touches the shared scratch, so it must not overtake the previous plan.  Plans issued through
// mw_plan_next run on the library's own stream; the first plan launched on another stream afterwards waits for them.
int order_after_side_plans(mw_ctx *ctx, cudaStream_t st)
{
    if (ctx->plans_on_side_stream && st != ctx->plan_stream) {
        if (cudaStreamWaitEvent(st, ctx->ev_planned, 0) != cudaSuccess) return MW_ERR_CUDA;
        ctx->plans_on_side_stream = 0;
    }
    return MW_OK;
}

}  // namespace

int mw_plan_on_side_stream(mw_ctx *ctx, const int32_t *topk_ids, const int32_t *expert_to_rank, int32_t T, cudaStream_t user)
{
    if (cudaEventRecord(ctx->ev_submitted, user) != cudaSuccess ||
        cudaStreamWaitEvent(ctx->plan_stream, ctx->ev_submitted, 0) != cudaSuccess)
        return MW_ERR_CUDA;
    const int rc = mw_plan_launch(ctx, topk_ids, expert_to_rank, T, nullptr, ctx->plan_stream);
    if (rc != MW_OK) return rc;
    if (cudaEventRecord(ctx->ev_planned, ctx->plan_stream) != cudaSuccess) return MW_ERR_CUDA;
    ctx->plans_on_side_stream = 1;
    return MW_OK;
}

extern "C" {

int mw_create(mw_ctx **out, const mw_config *cfg)
{
    if (!out) return MW_ERR_INVALID_ARG;
    *out = nullptr;
    if (!cfg) return MW_ERR_INVALID_ARG;
    if (cfg->R < 1 || cfg->R > MW_MAX_RANKS || cfg->E < 1 || cfg->K < 1 || cfg->K > MW_MAX_TOPK ||
        cfg->max_tokens < 1 || cfg->max_tokens > (1 << 24) || cfg->row_bytes < 16 || cfg->src_rank < -1 ||
        cfg->src_rank >= cfg->R || cfg->device < 0)
        return MW_ERR_INVALID_ARG;
    if (cfg->row_bytes % 16) return MW_ERR_ALIGNMENT;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || cfg->device >= ndev) return MW_ERR_CUDA;
    if (cudaSetDevice(cfg->device) != cudaSuccess) return MW_ERR_CUDA;

    mw_ctx *c = new (std::nothrow) mw_ctx();
    if (!c) return MW_ERR_INVALID_ARG;
    memset(c, 0, sizeof(*c));
    c->cfg = *cfg;
    c->W = (cfg->R + 63) / 64;
    c->Kd = cfg->K < cfg->R ? cfg->K : cfg->R;
    c->NC = cfg->R + 2;
    c->max_tiles = (cfg->max_tokens + MW_TILE - 1) / MW_TILE;
    int hs = 1024;                                    // load factor <= 1/8 keeps probe chains short
    while (hs < 8 * cfg->max_tokens) hs <<= 1;
    c->HS = hs;
    c->spin_limit = (cfg->flags & MW_FLAG_SHORT_WAITS) ? (1 << 10) : (1 << 20);       // about a millisecond / a second
    c->bar_spin_limit = (cfg->flags & MW_FLAG_SHORT_WAITS) ? (1 << 11) : (1 << 21);
    c->copy_wait_limit = (cfg->flags & MW_FLAG_SHORT_WAITS) ? (1 << 10) : (1 << 20);
    cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, cfg->device);
    cudaDeviceGetAttribute(&c->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, cfg->device);
    cudaDeviceGetAttribute(&c->l2_bytes, cudaDevAttrL2CacheSize, cfg->device);

    const size_t bytes = carve(c, nullptr);
    if (cudaMalloc(&c->slab, bytes) != cudaSuccess) { cudaGetLastError(); delete c; return MW_ERR_CUDA; }
    carve(c, (uint8_t *)c->slab);
    int rc = MW_OK;
    if (cudaMemset(c->slab, 0, bytes) != cudaSuccess) rc = MW_ERR_CUDA;
    if (rc == MW_OK) rc = init_scratch(c);
    if (rc == MW_OK) {
        // planning stream of mw_plan_next: its few blocks should be placed as soon as an SM has room, ahead of the
        // copy kernels' backlog, hence the highest priority
        int lo = 0, hi = 0;
        if (cudaDeviceGetStreamPriorityRange(&lo, &hi) != cudaSuccess ||
            cudaStreamCreateWithPriority(&c->plan_stream, cudaStreamNonBlocking, hi) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_submitted, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_planned, cudaEventDisableTiming) != cudaSuccess)
            rc = MW_ERR_CUDA;
    }
    if (rc == MW_OK) rc = mw_plan_smem_setup(c);
    if (rc == MW_OK) rc = mw_copy_smem_setup(c);
    if (rc == MW_OK) rc = mw_small_setup(c);
    if (rc == MW_OK) rc = mw_order_smem_setup(c);
    if (rc != MW_OK) { release(c); return rc; }
    *out = c;
    return MW_OK;
}

int mw_destroy(mw_ctx *ctx)
{
    if (!ctx) return MW_OK;
    cudaSetDevice(ctx->cfg.device);
    const cudaError_t e = cudaDeviceSynchronize();
    release(ctx);
    return e == cudaSuccess ? MW_OK : MW_ERR_CUDA;
}

int mw_reset(mw_ctx *ctx)
{
    if (!ctx) return MW_ERR_INVALID_ARG;
    if (cudaSetDevice(ctx->cfg.device) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) return MW_ERR_CUDA;
    return init_scratch(ctx);
}

int mw_test_skew_waits(mw_ctx *ctx, uint32_t what)
{
    if (!ctx || (what & ~(MW_TEST_SKEW_LOOKBACK | MW_TEST_SKEW_BARRIER | MW_TEST_SKEW_BULK_LOAD | MW_TEST_SKEW_GROUP_MAJOR))) return MW_ERR_INVALID_ARG;
    ctx->test_skew = what;
    return MW_OK;
}

namespace {
int plan_with_rows(mw_ctx *ctx, const int32_t *topk_ids, const int32_t *expert_to_rank, int32_t T, const void *rows,
                   mw_plan_view *view, void *stream)
{
    if (!ctx || !expert_to_rank || T < 0 || T > ctx->cfg.max_tokens || (T > 0 && !topk_ids)) return MW_ERR_INVALID_ARG;
    MW_REFUSE_IF_POISONED(ctx);
    if (rows && !aligned16(rows)) return MW_ERR_ALIGNMENT;
    if (view) fill_view(ctx, T, view);
    const int rc = order_after_side_plans(ctx, as_stream(stream));
    if (rc != MW_OK) return rc;
    return mw_plan_launch(ctx, topk_ids, expert_to_rank, T, rows, as_stream(stream));
}
}  // namespace

int mw_plan(mw_ctx *ctx, const int32_t *topk_ids, const int32_t *expert_to_rank, int32_t T, mw_plan_view *view, void *stream)
{
    return plan_with_rows(ctx, topk_ids, expert_to_rank, T, nullptr, view, stream);
}

int mw_plan_prefetch(mw_ctx *ctx, const int32_t *topk_ids, const int32_t *expert_to_rank, int32_t T, const void *x,
                     mw_plan_view *view, void *stream)
{
    if (!x && T > 0) return MW_ERR_INVALID_ARG;
    return plan_with_rows(ctx, topk_ids, expert_to_rank, T, x, view, stream);
}

int mw_plan_next(mw_ctx *ctx, const int32_t *topk_ids, const int32_t *expert_to_rank, int32_t T, const void *x, void *stream)
{
    if (!ctx || !expert_to_rank || T < 0 || T > ctx->cfg.max_tokens || (T > 0 && !topk_ids)) return MW_ERR_INVALID_ARG;
    MW_REFUSE_IF_POISONED(ctx);
    if (x && !aligned16(x)) return MW_ERR_ALIGNMENT;
    // everything the caller has submitted so far comes first: the inputs of this plan, and the copy kernels that
    // still read the slot about to be overwritten (it held the batch before the current one)
    if (cudaEventRecord(ctx->ev_submitted, as_stream(stream)) != cudaSuccess ||
        cudaStreamWaitEvent(ctx->plan_stream, ctx->ev_submitted, 0) != cudaSuccess)
        return MW_ERR_CUDA;
    swap_slots(ctx);                                   // plan into the slot the data path is not using
    const int rc = mw_plan_launch(ctx, topk_ids, expert_to_rank, T, x, ctx->plan_stream);
    swap_slots(ctx);
    if (rc != MW_OK) return rc;
    if (cudaEventRecord(ctx->ev_planned, ctx->plan_stream) != cudaSuccess) return MW_ERR_CUDA;
    ctx->plans_on_side_stream = 1;
    ctx->next_pending = 1;
    return MW_OK;
}

int mw_plan_swap(mw_ctx *ctx, mw_plan_view *view, void *stream)
{
    if (!ctx) return MW_ERR_INVALID_ARG;
    MW_REFUSE_IF_POISONED(ctx);
    if (!ctx->next_pending) return MW_ERR_NO_PLAN;
    if (cudaStreamWaitEvent(as_stream(stream), ctx->ev_planned, 0) != cudaSuccess) return MW_ERR_CUDA;
    swap_slots(ctx);
    ctx->next_pending = 0;
    if (view) fill_view(ctx, ctx->planned_T, view);
    return MW_OK;
}

int mw_get_plan_view(mw_ctx *ctx, mw_plan_view *view)
{
    if (!ctx || !view) return MW_ERR_INVALID_ARG;
    if (ctx->planned_T < 0) return MW_ERR_NO_PLAN;
    fill_view(ctx, ctx->planned_T, view);
    return MW_OK;
}

int mw_get_totals(mw_ctx *ctx, mw_totals *host_out, void *stream)
{
    if (!ctx || !host_out) return MW_ERR_INVALID_ARG;
    if (ctx->planned_T < 0) return MW_ERR_NO_PLAN;
    if (cudaMemcpyAsync(host_out, ctx->d.totals, sizeof(mw_totals), cudaMemcpyDeviceToHost, as_stream(stream)) != cudaSuccess)
        return MW_ERR_CUDA;
    if (cudaStreamSynchronize(as_stream(stream)) != cudaSuccess) return MW_ERR_CUDA;
    // a wait that gave up leaves the shared scratch and the host's running counts out of step: no further
    // device work on this context until mw_reset
    if (host_out->status == MW_ERR_TIMEOUT) ctx->poisoned = 1;
    return MW_OK;
}

int mw_pack(mw_ctx *ctx, const void *x, int layout, void *send_buf, int64_t send_capacity_rows, void *stream)
{
    if (!ctx || !x || !send_buf || send_capacity_rows < 0 || check_layout(layout)) return MW_ERR_INVALID_ARG;
    MW_REFUSE_IF_POISONED(ctx);
    if (ctx->planned_T < 0) return MW_ERR_NO_PLAN;
    if (!aligned16(x) || !aligned16(send_buf)) return MW_ERR_ALIGNMENT;
    mw_copy_args a = base_args(ctx);
    a.src = (const uint8_t *)x;
    a.dst = (uint8_t *)send_buf;
    a.capacity_rows = send_capacity_rows;
    if (layout == MW_LAYOUT_MULTIWRITE) {
        a.mode = MW_CP_PACK_MW;
        a.rows_from = 1;                       // T' send rows, known on the device
        a.src_index = ctx->d.mw_row_token;
        a.host_rows = ctx->planned_T;          // estimate for the chunking heuristic
    } else {
        // one pass over the non-empty tokens: each hidden row is read once and written to its |D_t| unicast slots
        a.mode = MW_CP_SCATTER;
        a.rows_from = 1;
        a.host_rows = ctx->planned_T;          // estimate for the chunking heuristic
        a.src_index = ctx->d.mw_row_token;
        a.ndst = ctx->d.row_ndest;
        a.d_rank = ctx->d.row_dest_rank;
        a.d_pos = ctx->d.row_dest_pos;
        a.d_flat = ctx->d.row_dest_flat;
        a.dst_stride = 0;
    }
    return mw_copy_launch(ctx, a, as_stream(stream));
}

int mw_deliver(mw_ctx *ctx, int layout, const void *send_buf, void *recv_base, int64_t recv_stride_bytes,
               int64_t recv_capacity_rows, void *stream)
{
    if (!ctx || !send_buf || !recv_base || recv_stride_bytes < 0 || recv_capacity_rows < 0 || check_layout(layout))
        return MW_ERR_INVALID_ARG;
    MW_REFUSE_IF_POISONED(ctx);
    if (ctx->planned_T < 0) return MW_ERR_NO_PLAN;
    if (!aligned16(send_buf) || !aligned16(recv_base) || recv_stride_bytes % 16) return MW_ERR_ALIGNMENT;
    if (recv_stride_bytes && recv_capacity_rows * ctx->cfg.row_bytes > recv_stride_bytes) return MW_ERR_CAPACITY;
    mw_copy_args a = base_args(ctx);
    a.src = (const uint8_t *)send_buf;
    a.dst = (uint8_t *)recv_base;
    a.dst_stride = recv_stride_bytes;
    a.capacity_rows = recv_capacity_rows;
    if (layout == MW_LAYOUT_MULTIWRITE) {
        a.mode = MW_CP_SCATTER;
        a.rows_from = 1;
        a.ndst = ctx->d.row_ndest;
        a.d_rank = ctx->d.row_dest_rank;
        a.d_pos = ctx->d.row_dest_pos;
        a.d_flat = ctx->d.row_dest_flat;
        a.host_rows = ctx->planned_T;          // estimate for the chunking heuristic
    } else {
        a.mode = MW_CP_DELIVER_UC;
        a.rows_from = 2;
        a.host_rows = (int64_t)ctx->planned_T * ctx->Kd;
    }
    return mw_copy_launch(ctx, a, as_stream(stream));
}

int mw_deliver_ptrs(mw_ctx *ctx, int layout, const void *send_buf, void *const *recv_ptrs, int64_t recv_capacity_rows,
                    void *stream)
{
    if (!ctx || !send_buf || !recv_ptrs || recv_capacity_rows < 0 || check_layout(layout)) return MW_ERR_INVALID_ARG;
    MW_REFUSE_IF_POISONED(ctx);
    if (ctx->planned_T < 0) return MW_ERR_NO_PLAN;
    if (!aligned16(send_buf) || ((uintptr_t)recv_ptrs & 7u)) return MW_ERR_ALIGNMENT;
    mw_copy_args a = base_args(ctx);
    a.src = (const uint8_t *)send_buf;
    a.dst_ptrs = (uint8_t *const *)recv_ptrs;
    a.capacity_rows = recv_capacity_rows;
    if (layout == MW_LAYOUT_MULTIWRITE) {
        a.mode = MW_CP_SCATTER;
        a.rows_from = 1;
        a.ndst = ctx->d.row_ndest;
        a.d_rank = ctx->d.row_dest_rank;
        a.d_pos = ctx->d.row_dest_pos;
        a.d_flat = ctx->d.row_dest_flat;
        a.host_rows = ctx->planned_T;
    } else {
        a.mode = MW_CP_DELIVER_UC;
        a.rows_from = 2;
        a.host_rows = (int64_t)ctx->planned_T * ctx->Kd;
    }
    return mw_copy_launch(ctx, a, as_stream(stream));
}

int mw_dispatch(mw_ctx *ctx, const void *x, int layout, void *send_buf, int64_t send_capacity_rows,
                void *recv_base, int64_t recv_stride_bytes, int64_t recv_capacity_rows, void *stream)
{
    if (!ctx || !x || !send_buf || !recv_base) return MW_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(send_buf) || !aligned16(recv_base) || recv_stride_bytes % 16) return MW_ERR_ALIGNMENT;
    if (ctx->cfg.flags & MW_FLAG_COPY_BULK) {
        int rc = mw_pack(ctx, x, layout, send_buf, send_capacity_rows, stream);
        if (rc != MW_OK) return rc;
        return mw_deliver(ctx, layout, send_buf, recv_base, recv_stride_bytes, recv_capacity_rows, stream);
    }
    // one pass: every hidden row is read once and written to its send slot(s) and to all its receive slots
    if (recv_stride_bytes < 0 || recv_capacity_rows < 0 || send_capacity_rows < 0 || check_layout(layout)) return MW_ERR_INVALID_ARG;
    MW_REFUSE_IF_POISONED(ctx);
    if (ctx->planned_T < 0) return MW_ERR_NO_PLAN;
    if (recv_stride_bytes && recv_capacity_rows * ctx->cfg.row_bytes > recv_stride_bytes) return MW_ERR_CAPACITY;
    mw_copy_args a = base_args(ctx);
    a.mode = layout == MW_LAYOUT_MULTIWRITE ? MW_CP_DISPATCH_MW : MW_CP_DISPATCH_UC;
    a.src = (const uint8_t *)x;
    a.src_in_l2 = ctx->prefetched == x && layout == MW_LAYOUT_MULTIWRITE;
    a.src_index = ctx->d.mw_row_token;
    a.dst = (uint8_t *)recv_base;
    a.dst_stride = recv_stride_bytes;
    a.capacity_rows = recv_capacity_rows;
    a.dst2 = (uint8_t *)send_buf;
    a.capacity2_rows = send_capacity_rows;
    a.rows_from = 1;
    a.host_rows = ctx->planned_T;
    a.ndst = ctx->d.row_ndest;
    a.d_rank = ctx->d.row_dest_rank;
    a.d_pos = ctx->d.row_dest_pos;
    a.d_flat = ctx->d.row_dest_flat;
    return mw_copy_launch(ctx, a, as_stream(stream));
}

int mw_plan_dispatch(mw_ctx *ctx, const int32_t *topk_ids, const int32_t *expert_to_rank, int32_t T, const void *x,
                     int layout, void *send_buf, int64_t send_capacity_rows, void *recv_base, int64_t recv_stride_bytes,
                     int64_t recv_capacity_rows, mw_plan_view *view, void *stream)
{
    if (!ctx || !expert_to_rank || T < 0 || T > ctx->cfg.max_tokens || (T > 0 && !topk_ids) || !x || !send_buf || !recv_base ||
        send_capacity_rows < 0 || recv_stride_bytes < 0 || recv_capacity_rows < 0 || check_layout(layout))
        return MW_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(send_buf) || !aligned16(recv_base) || recv_stride_bytes % 16) return MW_ERR_ALIGNMENT;
    if (recv_stride_bytes && recv_capacity_rows * ctx->cfg.row_bytes > recv_stride_bytes) return MW_ERR_CAPACITY;
    if (!mw_small_applies(ctx, T, layout)) {
        const int rc = mw_plan_prefetch(ctx, topk_ids, expert_to_rank, T, x, view, stream);
        if (rc != MW_OK) return rc;
        return mw_dispatch(ctx, x, layout, send_buf, send_capacity_rows, recv_base, recv_stride_bytes, recv_capacity_rows, stream);
    }
    MW_REFUSE_IF_POISONED(ctx);
    if (view) fill_view(ctx, T, view);
    {
        const int rc = order_after_side_plans(ctx, as_stream(stream));    // the launch writes the accumulators plans share
        if (rc != MW_OK) return rc;
    }
    return mw_small_launch(ctx, topk_ids, expert_to_rank, T, x, send_buf, send_capacity_rows, recv_base, recv_stride_bytes,
                           recv_capacity_rows, as_stream(stream));
}

int mw_allgather_pack(mw_ctx *ctx, const void *shards, int64_t shard_bytes, int layout, void *send_buf,
                      void *recv_base, int64_t recv_stride_bytes, int32_t dst_rank_begin, int32_t dst_rank_count,
                      mw_totals *host_totals, void *stream)
{
    if (!ctx || !shards || !send_buf || !recv_base || shard_bytes < 16 || recv_stride_bytes < 0 || check_layout(layout))
        return MW_ERR_INVALID_ARG;
    const int R = ctx->cfg.R;
    if (dst_rank_begin < 0 || dst_rank_count < 0 || dst_rank_begin + dst_rank_count > R) return MW_ERR_INVALID_ARG;
    if (shard_bytes % 16 || recv_stride_bytes % 16 || !aligned16(shards) || !aligned16(send_buf) || !aligned16(recv_base))
        return MW_ERR_ALIGNMENT;
    const int64_t stride = recv_stride_bytes ? recv_stride_bytes : (int64_t)R * shard_bytes;
    if (stride < (int64_t)R * shard_bytes) return MW_ERR_CAPACITY;
    if (host_totals) {
        memset(host_totals, 0, sizeof(*host_totals));
        host_totals->T_nonempty = R;
        host_totals->G = R;
        host_totals->total_dest = (int64_t)R * R;
        host_totals->mw_bytes = R > 1 ? (int64_t)R * shard_bytes : 0;
        host_totals->unicast_bytes = (int64_t)R * (R - 1) * shard_bytes;     // Section 2.3.1: R - 1 copies per source
        host_totals->unicast_per_expert_bytes = host_totals->unicast_bytes;
        host_totals->meta_bytes = (R <= 64) ? 0 : (int64_t)R * ((shard_bytes + 4095) / 4096) * (8 * ctx->W);
    }
    if (dst_rank_count == 0 && layout == MW_LAYOUT_UNICAST) return MW_OK;   // empty window: no unicast slot exists
    mw_copy_args a = base_args(ctx);
    a.row_bytes = shard_bytes;
    a.rows_from = 0;
    a.dst_begin = dst_rank_begin;
    a.dst_count = dst_rank_count;
    a.capacity_rows = INT64_MAX;
    int rc;
    if (!(ctx->cfg.flags & MW_FLAG_COPY_BULK)) {
        // one pass: every shard is read once and written to its send slot(s) and to its slot in every region of the window
        a.mode = layout == MW_LAYOUT_MULTIWRITE ? MW_CP_AG_FUSED_MW : MW_CP_AG_FUSED_UC;
        a.src = (const uint8_t *)shards; a.dst = (uint8_t *)recv_base; a.dst2 = (uint8_t *)send_buf;
        a.dst_stride = stride; a.host_rows = R;
        return mw_copy_launch(ctx, a, as_stream(stream));
    }
    if (layout == MW_LAYOUT_MULTIWRITE) {
        a.mode = MW_CP_AG_PACK_MW;
        a.src = (const uint8_t *)shards; a.dst = (uint8_t *)send_buf; a.host_rows = R;
        if ((rc = mw_copy_launch(ctx, a, as_stream(stream))) != MW_OK || dst_rank_count == 0) return rc;
        a.mode = MW_CP_AG_DELIVER_MW;
        a.src = (const uint8_t *)send_buf; a.dst = (uint8_t *)recv_base; a.dst_stride = stride;
        return mw_copy_launch(ctx, a, as_stream(stream));
    }
    a.mode = MW_CP_AG_PACK_UC;
    a.src = (const uint8_t *)shards; a.dst = (uint8_t *)send_buf; a.host_rows = R;
    if ((rc = mw_copy_launch(ctx, a, as_stream(stream))) != MW_OK) return rc;
    a.mode = MW_CP_AG_DELIVER_UC;
    a.src = (const uint8_t *)send_buf; a.src2 = (const uint8_t *)shards; a.dst = (uint8_t *)recv_base;
    a.dst_stride = stride; a.host_rows = (int64_t)R * dst_rank_count;
    return mw_copy_launch(ctx, a, as_stream(stream));
}

int64_t mw_pair_balanced_direct_bytes(int64_t shard_bytes, int32_t ranks_per_domain, int layout)
{
    if (ranks_per_domain <= 1) return shard_bytes;
    const int64_t c = layout == MW_LAYOUT_MULTIWRITE ? 1 : ranks_per_domain - 1;
    return (shard_bytes * c / (1 + c)) / 16 * 16;
}

int64_t mw_pair_split_direct_bytes(int64_t shard_bytes, int32_t ranks_per_domain, int layout, double w_direct, double w_pair)
{
    if (ranks_per_domain <= 1 || !(w_direct > 0.0) || !(w_pair > 0.0)) return shard_bytes;
    const double copies = layout == MW_LAYOUT_MULTIWRITE ? 1.0 : (double)(ranks_per_domain - 1);
    // a direct link carries d bytes, the pair link `copies` times the rest: d / w_direct = copies (s - d) / w_pair
    const double together = floor((double)shard_bytes * copies * w_direct / (w_pair + copies * w_direct));
    int64_t d = (int64_t)together / 16 * 16;
    if (d > shard_bytes) d = shard_bytes / 16 * 16;
    return d;
}

int mw_paired_allgather(mw_ctx *ctx, const void *shards, int64_t shard_bytes, int64_t direct_bytes, int layout,
                        void *relay_buf, void *recv_base, mw_pair_totals *host_totals, void *stream)
{
    if (!ctx || !shards || !recv_base || shard_bytes < 16 || direct_bytes < 0 || direct_bytes > shard_bytes || check_layout(layout))
        return MW_ERR_INVALID_ARG;
    const int R = ctx->cfg.R;
    if (R < 2 || R % 2) return MW_ERR_INVALID_ARG;
    const int n = R / 2;
    const int64_t relay_bytes = shard_bytes - direct_bytes;
    const int copies = layout == MW_LAYOUT_MULTIWRITE ? 1 : n - 1;
    if (relay_bytes > 0 && copies > 0 && !relay_buf) return MW_ERR_INVALID_ARG;
    if (shard_bytes % 16 || direct_bytes % 16 || !aligned16(shards) || !aligned16(recv_base) || (relay_buf && !aligned16(relay_buf)))
        return MW_ERR_ALIGNMENT;
    if (host_totals) {
        host_totals->direct_link_bytes = n > 1 ? direct_bytes : 0;
        host_totals->pair_link_bytes = n > 1 ? copies * relay_bytes : 0;
        host_totals->forward_link_bytes = n > 1 ? relay_bytes : 0;
        int64_t m = host_totals->direct_link_bytes;
        if (host_totals->pair_link_bytes > m) m = host_totals->pair_link_bytes;
        if (host_totals->forward_link_bytes > m) m = host_totals->forward_link_bytes;
        host_totals->max_link_bytes = m;
        host_totals->total_bytes = (int64_t)R * ((n - 1) * direct_bytes + host_totals->pair_link_bytes +
                                                 (n - 1) * host_totals->forward_link_bytes);
    }
    mw_copy_args a = base_args(ctx);
    a.rows_from = 0;
    a.capacity_rows = INT64_MAX;
    a.shard_bytes = shard_bytes;
    a.pair_n = n;
    a.pair_copies = copies;
    int rc = MW_OK;
    if (direct_bytes > 0) {                    // direct segment to every member of the domain (own copy included, local)
        a.mode = MW_CP_PAIR_DIRECT;
        a.src = (const uint8_t *)shards; a.dst = (uint8_t *)recv_base;
        a.row_bytes = direct_bytes; a.seg_off = 0; a.host_rows = R;
        if ((rc = mw_copy_launch(ctx, a, as_stream(stream))) != MW_OK) return rc;
    }
    if (relay_bytes > 0) {
        a.mode = MW_CP_PAIR_SEND;              // relayed segment to the partner's relay area (and own copy)
        a.src = (const uint8_t *)shards; a.dst = (uint8_t *)relay_buf; a.dst2 = (uint8_t *)recv_base;
        a.row_bytes = relay_bytes; a.seg_off = direct_bytes; a.host_rows = R;
        a.keep_in_l2 = 1;                      // the forward launch reads the relay area next
        if ((rc = mw_copy_launch(ctx, a, as_stream(stream))) != MW_OK) return rc;
        if (n > 1) {
            a.keep_in_l2 = 0;
            a.mode = MW_CP_PAIR_FORWARD;       // the partner forwards it to the other members of the source's domain
            a.src = (const uint8_t *)relay_buf; a.dst = (uint8_t *)recv_base;
            a.host_rows = (int64_t)R * (n - 1);
            rc = mw_copy_launch(ctx, a, as_stream(stream));
        }
    }
    return rc;
}

int mw_dispatch_host(mw_ctx *ctx, const int32_t *topk_ids_host, const int32_t *expert_to_rank_host,
                     const void *x_host, int32_t T, int layout, void *recv_host, int64_t recv_capacity_rows,
                     int32_t *rank_offsets_host, mw_totals *totals_host, void *stream)
{
    if (!ctx || !expert_to_rank_host || !recv_host || !rank_offsets_host || !totals_host || T < 0 ||
        T > ctx->cfg.max_tokens || (T > 0 && (!topk_ids_host || !x_host)) || check_layout(layout))
        return MW_ERR_INVALID_ARG;
    if (!(ctx->cfg.flags & MW_FLAG_HOST_STAGING)) return MW_ERR_INVALID_ARG;
    cudaStream_t st = as_stream(stream);
    const int64_t B = ctx->cfg.row_bytes;
    if (cudaMemcpyAsync(ctx->st_e2r, expert_to_rank_host, sizeof(int32_t) * (size_t)ctx->cfg.E, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return MW_ERR_CUDA;
    if (T > 0) {
        if (cudaMemcpyAsync(ctx->st_ids, topk_ids_host, sizeof(int32_t) * (size_t)T * ctx->cfg.K, cudaMemcpyHostToDevice, st) != cudaSuccess)
            return MW_ERR_CUDA;
        if (cudaMemcpyAsync(ctx->st_x, x_host, (size_t)T * B, cudaMemcpyHostToDevice, st) != cudaSuccess) return MW_ERR_CUDA;
    }
    int rc = mw_plan(ctx, ctx->st_ids, ctx->st_e2r, T, nullptr, stream);
    if (rc != MW_OK) return rc;
    rc = mw_dispatch(ctx, ctx->st_x, layout, ctx->st_send, ctx->st_recv_rows, ctx->st_recv, 0, ctx->st_recv_rows, stream);
    if (rc != MW_OK) return rc;
    if (cudaMemcpyAsync(rank_offsets_host, ctx->d.rank_offsets, sizeof(int32_t) * (size_t)(ctx->cfg.R + 1), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return MW_ERR_CUDA;
    rc = mw_get_totals(ctx, totals_host, stream);       // synchronises: the row count is needed for the copy back
    if (rc != MW_OK) return rc;
    if (totals_host->total_dest > recv_capacity_rows) return MW_ERR_CAPACITY;
    if (totals_host->total_dest > 0) {
        if (cudaMemcpyAsync(recv_host, ctx->st_recv, (size_t)totals_host->total_dest * B, cudaMemcpyDeviceToHost, st) != cudaSuccess)
            return MW_ERR_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return MW_ERR_CUDA;
    }
    return MW_OK;
}

int mw_read_device(mw_ctx *ctx, void *host_dst, const void *device_src, int64_t bytes, void *stream)
{
    if (!ctx || bytes < 0 || (bytes > 0 && (!host_dst || !device_src))) return MW_ERR_INVALID_ARG;
    if (cudaStreamSynchronize(as_stream(stream)) != cudaSuccess) return MW_ERR_CUDA;
    if (bytes == 0) return MW_OK;
    return cudaMemcpy(host_dst, device_src, (size_t)bytes, cudaMemcpyDeviceToHost) == cudaSuccess ? MW_OK : MW_ERR_CUDA;
}

int64_t mw_kernel_launches(const mw_ctx *ctx) { return ctx ? ctx->launches : 0; }

const char *mw_strerror(int code)
{
    switch (code) {
    case MW_OK: return "ok";
    case MW_ERR_INVALID_ARG: return "invalid argument";
    case MW_ERR_ALIGNMENT: return "pointer, stride or row size is not a multiple of 16 bytes";
    case MW_ERR_CAPACITY: return "a buffer is too small for the rows assigned to it";
    case MW_ERR_CUDA: return "a CUDA runtime call failed";
    case MW_ERR_BAD_INDEX: return "expert id or expert-to-rank entry out of range";
    case MW_ERR_TIMEOUT: return "a bounded device-side wait gave up";
    case MW_ERR_NO_PLAN: return "no plan has been made on this context";
    default: return "unknown error code";
    }
}

}  // extern "C"
