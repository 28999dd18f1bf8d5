// Two-level (relayed) MultiWrite dispatch (paper: Section 3.2, Section 4.1 "Local forwarding table",
// Section 4.3.3; Section 6.4 for the relay buffer).  Declared and documented in include/mw.h.
//
// The first-level plan is the ordinary plan machinery run on next-hop sets (the plan maps every rank to its next
// hop, so "one copy per distinct next hop" is just the per-rank dedup of the flat path); the flat plan gives the
// final slots.  The two plans are independent and run concurrently (one on the caller's stream, one on the
// library's planning stream); k_relay_desc then derives both levels' descriptors and the accounting.
// Data movement is one launch, k_relay_rows, one block per (first-level send row, piece of the row):
//   first level   the piece of the hidden row is read once and written to its send slot and to every next hop.  The
//                 receive buffer is the relay buffer: a copy whose next hop is itself a destination of the token goes
//                 straight to its final slot; only a copy held by a pure relay is staged in the hop area;
//   second level  for every relay that has something to forward, the same threads read the copy back from where the
//                 relay holds it (it was written a moment ago, so it comes out of L2, not DRAM) and store it to the
//                 token's other destinations inside that relay's server, at the slots of the flat plan.
// The final receive regions are byte-identical to those of the flat dispatch.
#include <new>
#include <string.h>

#include "mw_internal.cuh"

struct mw_relay {
    mw_ctx *hop, *flat;
    int P;                       // ranks per server
    int64_t Tm;                  // max_tokens: rows per descriptor plane (planes are indexed by first-level send row)
    int32_t *f1_rank, *f1_pos, *f1_flat;   // [Kd, Tm] where the copy for hop i of send row j goes: final slot, or hop-area row
    int32_t *s2_n;                         // [Tm]     copies the relays forward for send row j
    int32_t *s2_cnt;                       // [Kd, Tm] of which hop i forwards this many (consecutive in the lists below)
    int32_t *s2_rank, *s2_pos, *s2_flat;   // [Kd, Tm] final destination of forwarded copy k of send row j
    long long *block_part;                 // [max_tiles, 7] per-block sums of the accounting
    unsigned int *blocks_done;             // ticket of the descriptor kernel's blocks (zero between launches)
    mw_relay_totals *totals;     // device
    void *slab;
    int planned;
};

namespace {

constexpr int kDescThreads = 256; // rows per block of the descriptor kernels (64-thread blocks on more SMs were slower: 42 against 39 us per plan)
constexpr int kAccounts = 7;     // hop rows, delivered rows, direct, inter-server MultiWrite, inter-server unicast, forwarded, staged

struct DescArgs {
    int T, Kd, R, src, P;
    int64_t Tm, row_bytes;
    mw_dev hop, flat;            // the two plans
    int32_t *f1_rank, *f1_pos, *f1_flat, *s2_n, *s2_cnt, *s2_rank, *s2_pos, *s2_flat;
    long long *block_part;
    unsigned int *blocks_done;
    mw_relay_totals *totals;
};

// Block sums of the accounting, then the last block to finish adds the blocks up and writes the totals (integer sums:
// the order does not matter).  All threads of the block must call it.
__device__ void desc_finish(const DescArgs &a, long long (&v)[kAccounts], long long *part_s, unsigned int *last_s)
{
#pragma unroll
    for (int k = 0; k < kAccounts; ++k) {
        for (int o = 16; o > 0; o >>= 1) v[k] += __shfl_down_sync(0xffffffffu, v[k], o);
        if ((threadIdx.x & 31) == 0 && v[k]) atomicAdd((unsigned long long *)&part_s[k], (unsigned long long)v[k]);
    }
    __syncthreads();
    if (threadIdx.x < kAccounts) a.block_part[(int64_t)blockIdx.x * kAccounts + threadIdx.x] = part_s[threadIdx.x];
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) *last_s = atomicAdd(a.blocks_done, 1u) == gridDim.x - 1 ? 1u : 0u;
    __syncthreads();
    if (!*last_s) return;
    __threadfence();
    if (threadIdx.x < kAccounts) part_s[threadIdx.x] = 0;
    __syncthreads();
    for (unsigned i = threadIdx.x; i < gridDim.x * kAccounts; i += blockDim.x)          // independent loads, one round trip
        atomicAdd((unsigned long long *)&part_s[i % kAccounts], (unsigned long long)__ldcg(a.block_part + i));
    __syncthreads();
    if (threadIdx.x == 0) {
        mw_relay_totals tt;
        tt.hop_rows = part_s[0]; tt.delivered_rows = part_s[1];
        tt.direct_bytes = part_s[2] * a.row_bytes; tt.inter_multiwrite_bytes = part_s[3] * a.row_bytes;
        tt.inter_unicast_bytes = part_s[4] * a.row_bytes; tt.forward_bytes = part_s[5] * a.row_bytes;
        tt.staged_rows = part_s[6];
        tt.status = a.flat.totals->status ? a.flat.totals->status : a.hop.totals->status;
        tt.reserved = 0;
        *a.totals = tt;
        *a.blocks_done = 0;
    }
}

// One thread per first-level send row j (token t = hop.mw_row_token[j]): where each next hop's copy goes, which
// copies each relay forwards, and the bytes per link class.  Destinations of a token are ascending in rank and a
// server is a contiguous range of ranks, so the forwarded copies come out grouped by hop, in hop order.
// KD = compile-time bound on Kd: everything a thread needs is loaded up front into registers (the output planes may
// alias the inputs as far as the compiler knows, so loads inside the loops would be repeated after every store).
template <int KD>
__global__ void __launch_bounds__(kDescThreads) k_relay_desc(const __grid_constant__ DescArgs a)
{
    __shared__ long long part_s[kAccounts];
    __shared__ unsigned int last_s;
    extern __shared__ int32_t flat_off_s[];            // [R + 1] region starts of the flat plan
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (threadIdx.x < kAccounts) part_s[threadIdx.x] = 0;
    const bool plans_ok = a.hop.totals->status != MW_ERR_TIMEOUT && a.flat.totals->status != MW_ERR_TIMEOUT;
    const bool active = plans_ok && j < a.hop.totals->T_nonempty;
    // independent loads first: the row's token, its hops (planes, coalesced), the region starts
    const int t = active ? a.hop.mw_row_token[j] : 0;
    const int nh = active ? a.hop.row_ndest[j] : 0;
    int hop_rank[KD], hop_row[KD];
#pragma unroll
    for (int i = 0; i < KD; ++i) {
        hop_rank[i] = (active && i < a.Kd) ? a.hop.row_dest_rank[(int64_t)i * a.Tm + j] : -1;
        hop_row[i] = (active && i < a.Kd) ? a.hop.row_dest_flat[(int64_t)i * a.Tm + j] : -1;    // row of the hop area this copy would take
    }
    for (int r = threadIdx.x; r <= a.R; r += blockDim.x) flat_off_s[r] = a.flat.rank_offsets[r];
    int fr[KD], fp[KD];
#pragma unroll
    for (int k = 0; k < KD; ++k) {
        fr[k] = (active && k < a.Kd) ? a.flat.dest_rank[(int64_t)t * a.Kd + k] : -1;
        fp[k] = (active && k < a.Kd) ? a.flat.dest_pos[(int64_t)t * a.Kd + k] : -1;
    }
    __syncthreads();
    long long v[kAccounts] = {0, 0, 0, 0, 0, 0, 0};
    if (active) {
        // Kept small on purpose: compares and selects in the KD x KD part, stores only in the two KD-long loops
        // (with the stores inside the double loop the unrolled code outgrew the instruction cache: 31 us for 4096 rows).
        const int src_server = a.src / a.P, src_index = a.src % a.P;
        int via[KD], own[KD], cnt[KD];                 // per destination: index of its next hop; per hop: own slot, copies to forward
#pragma unroll
        for (int i = 0; i < KD; ++i) { own[i] = -1; cnt[i] = 0; }
        int n2 = 0;
#pragma unroll
        for (int k = 0; k < KD; ++k) {
            const int r = fr[k];
            const int server = r >= 0 ? r / a.P : -1;
            const bool remote = server != src_server;
            const int h = remote ? server * a.P + src_index : r;               // mw_next_hop, with the source's part hoisted
            via[k] = -1;
#pragma unroll
            for (int i = 0; i < KD; ++i) {
                const bool m = r >= 0 && i < nh && hop_rank[i] == h;
                via[k] = m ? i : via[k];
                own[i] = (m && r == h) ? fp[k] : own[i];
                cnt[i] += (m && r != h);
            }
            if (via[k] >= 0) {
                ++v[1];
                if (remote) { ++v[4]; v[5] += (r != h); }
                else v[2] += (r != a.src);
                if (r != h) {                                                 // the relay forwards this one
                    a.s2_rank[(int64_t)n2 * a.Tm + j] = r;
                    a.s2_pos[(int64_t)n2 * a.Tm + j] = fp[k];
                    a.s2_flat[(int64_t)n2 * a.Tm + j] = flat_off_s[r] + fp[k];
                    ++n2;
                }
            }
        }
#pragma unroll
        for (int i = 0; i < KD; ++i) {
            if (i >= a.Kd) break;
            const int h = hop_rank[i];
            const bool in_place = i < nh && own[i] >= 0, staged = i < nh && own[i] < 0;
            if (i < nh) { ++v[0]; v[3] += (h / a.P != src_server); v[6] += staged; }
            a.s2_cnt[(int64_t)i * a.Tm + j] = cnt[i];
            // the relay buffer is the receive buffer (Section 6.4): a next hop that is a destination holds its copy in its final slot
            a.f1_rank[(int64_t)i * a.Tm + j] = in_place ? h : staged ? -2 : -1;
            a.f1_pos[(int64_t)i * a.Tm + j] = in_place ? own[i] : staged ? hop_row[i] : -1;
            a.f1_flat[(int64_t)i * a.Tm + j] = in_place ? flat_off_s[h] + own[i] : staged ? -2 - hop_row[i] : -1;
        }
        for (int k = n2; k < a.Kd; ++k) {
            a.s2_rank[(int64_t)k * a.Tm + j] = -1; a.s2_pos[(int64_t)k * a.Tm + j] = -1; a.s2_flat[(int64_t)k * a.Tm + j] = -1;
        }
        a.s2_n[j] = n2;
    }
    desc_finish(a, v, part_s, &last_s);
}

// The same for any Kd (beyond 16 the unrolled kernel would not fit in registers): plain loops over global memory.
__global__ void __launch_bounds__(kDescThreads) k_relay_desc_any(const __grid_constant__ DescArgs a)
{
    __shared__ long long part_s[kAccounts];
    __shared__ unsigned int last_s;
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (threadIdx.x < kAccounts) part_s[threadIdx.x] = 0;
    __syncthreads();
    long long v[kAccounts] = {0, 0, 0, 0, 0, 0, 0};
    const bool plans_ok = a.hop.totals->status != MW_ERR_TIMEOUT && a.flat.totals->status != MW_ERR_TIMEOUT;
    if (plans_ok && j < a.hop.totals->T_nonempty) {
        const int t = a.hop.mw_row_token[j];
        const int32_t *fr = a.flat.dest_rank + (int64_t)t * a.Kd, *fp = a.flat.dest_pos + (int64_t)t * a.Kd;
        const int nh = a.hop.row_ndest[j];
        int n2 = 0;
        for (int i = 0; i < a.Kd; ++i) {
            const int h = i < nh ? a.hop.row_dest_rank[(int64_t)i * a.Tm + j] : -1;
            const int q = i < nh ? a.hop.row_dest_flat[(int64_t)i * a.Tm + j] : -1;
            const bool remote = i < nh && h / a.P != a.src / a.P;
            int own_pos = -1, forwards = 0;
            for (int k = 0; i < nh && k < a.Kd; ++k) {
                const int r = fr[k];
                if (r < 0) break;
                if (mw_next_hop(r, a.src, a.P) != h) continue;
                ++v[1];
                if (r == h) own_pos = fp[k];
                if (remote) { ++v[4]; v[5] += (r != h); }
                else v[2] += (r != a.src);
                if (r != h) {
                    a.s2_rank[(int64_t)n2 * a.Tm + j] = r;
                    a.s2_pos[(int64_t)n2 * a.Tm + j] = fp[k];
                    a.s2_flat[(int64_t)n2 * a.Tm + j] = a.flat.rank_offsets[r] + fp[k];
                    ++n2; ++forwards;
                }
            }
            const bool in_place = i < nh && own_pos >= 0, staged = i < nh && own_pos < 0;
            if (i < nh) { ++v[0]; v[3] += remote; v[6] += staged; }
            a.s2_cnt[(int64_t)i * a.Tm + j] = forwards;
            a.f1_rank[(int64_t)i * a.Tm + j] = in_place ? h : staged ? -2 : -1;
            a.f1_pos[(int64_t)i * a.Tm + j] = in_place ? own_pos : staged ? q : -1;
            a.f1_flat[(int64_t)i * a.Tm + j] = in_place ? a.flat.rank_offsets[h] + own_pos : staged ? -2 - q : -1;
        }
        for (int k = n2; k < a.Kd; ++k) {
            a.s2_rank[(int64_t)k * a.Tm + j] = -1; a.s2_pos[(int64_t)k * a.Tm + j] = -1; a.s2_flat[(int64_t)k * a.Tm + j] = -1;
        }
        a.s2_n[j] = n2;
    }
    desc_finish(a, v, part_s, &last_s);
}

// ---- data movement: both levels in one launch ---------------------------------------------------------------
struct RowsArgs {
    const uint8_t *x;            // hidden rows
    uint8_t *send;               // first-level send buffer (each row once per group of identical next-hop set)
    uint8_t *hop_buf;            // hop area: copies held by pure relays
    uint8_t *recv;               // final receive regions (also the relay buffer of relays that are destinations)
    int64_t row_bytes, recv_stride, recv_capacity_rows, hop_capacity_rows, send_capacity_rows, Tm;
    int Kd, pieces;
    int32_t piece_bytes;
    const int32_t *src_index;    // token of first-level send row j
    const int32_t *row_ndest;    // next hops of send row j
    const int32_t *f1_rank, *f1_pos, *f1_flat, *s2_n, *s2_cnt, *s2_rank, *s2_pos, *s2_flat;
    mw_totals *totals;           // first-level accounting: row count, status
};

constexpr int kRelayMaxThreads = 256;
constexpr int kRelayBatch = 4;   // relay copies a thread reads back before it starts storing

__device__ __forceinline__ uint4 ld_row(const uint8_t *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
// Reads back what this same thread stored a moment ago: an ordinary (coherent) load at L2, ordered after the store by
// the memory clobber and by same-address program order.
__device__ __forceinline__ uint4 ld_held(const uint8_t *p)
{
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}

// One block per (first-level send row, piece of the row).  See the head of this file.  (Section 4.1 steps 3 to 5: the
// relay has the payload in its buffer, parses the metadata, replicates.)  No slot that is read back here is written
// by another block: a relay is never a forwarding target, and every (token, rank) pair has its own slot.
__global__ void __launch_bounds__(kRelayMaxThreads) k_relay_rows(const __grid_constant__ RowsArgs a)
{
    __shared__ uint8_t *held_s[MW_MAX_TOPK];     // where next hop i holds its copy (null: the copy could not be stored)
    __shared__ int cnt_s[MW_MAX_TOPK];           // copies next hop i forwards
    __shared__ uint8_t *dst_s[MW_MAX_TOPK];      // final slot of forwarded copy k
    grid_launch_dependents();
    grid_dependency_wait();
    const int tid = threadIdx.x;
    const int row = blockIdx.x / a.pieces, piece = blockIdx.x % a.pieces;
    const int status = a.totals->status;
    const int64_t rows = a.totals->T_nonempty;
    const int nh = a.row_ndest[row], n2 = a.s2_n[row];
    const int index = a.src_index[row];
    if (status == MW_ERR_TIMEOUT || row >= rows) return;
    const int64_t off = (int64_t)piece * a.piece_bytes + tid * 16;
    const bool mine = off < a.row_bytes;
    uint4 v;
    if (mine) v = ld_row(a.x + (int64_t)index * a.row_bytes + off);
    if (tid < nh) {
        uint8_t *p = nullptr;
        if (a.recv_stride) {
            const int r = a.f1_rank[(int64_t)tid * a.Tm + row], q = a.f1_pos[(int64_t)tid * a.Tm + row];
            if (r >= 0) {
                if (q >= a.recv_capacity_rows) atomicCAS(&a.totals->status, 0, MW_ERR_CAPACITY);
                else p = a.recv + (int64_t)r * a.recv_stride + (int64_t)q * a.row_bytes;
            } else if (r == -2) {
                if (q >= a.hop_capacity_rows) atomicCAS(&a.totals->status, 0, MW_ERR_CAPACITY);
                else p = a.hop_buf + (int64_t)q * a.row_bytes;
            }
        } else {
            const int64_t at = a.f1_flat[(int64_t)tid * a.Tm + row];
            if (at >= 0) {
                if (at >= a.recv_capacity_rows) atomicCAS(&a.totals->status, 0, MW_ERR_CAPACITY);
                else p = a.recv + at * a.row_bytes;
            } else if (at <= -2) {
                if (-2 - at >= a.hop_capacity_rows) atomicCAS(&a.totals->status, 0, MW_ERR_CAPACITY);
                else p = a.hop_buf + (-2 - at) * a.row_bytes;
            }
        }
        held_s[tid] = p;
        cnt_s[tid] = a.s2_cnt[(int64_t)tid * a.Tm + row];
    }
    if (tid < n2) {
        uint8_t *d = nullptr;
        if (a.recv_stride) {
            const int r = a.s2_rank[(int64_t)tid * a.Tm + row], q = a.s2_pos[(int64_t)tid * a.Tm + row];
            if (r >= 0) {
                if (q >= a.recv_capacity_rows) atomicCAS(&a.totals->status, 0, MW_ERR_CAPACITY);
                else d = a.recv + (int64_t)r * a.recv_stride + (int64_t)q * a.row_bytes;
            }
        } else {
            const int64_t at = a.s2_flat[(int64_t)tid * a.Tm + row];
            if (at >= 0) {
                if (at >= a.recv_capacity_rows) atomicCAS(&a.totals->status, 0, MW_ERR_CAPACITY);
                else d = a.recv + at * a.row_bytes;
            }
        }
        dst_s[tid] = d;
    }
    if (tid == 0 && row >= a.send_capacity_rows) atomicCAS(&a.totals->status, 0, MW_ERR_CAPACITY);
    __syncthreads();
    if (!mine) return;
    // first level: the send slot and one copy per next hop
    // (a copy that is read back below is stored normally and stays in L2; everything else is written once and streams)
    if (row < a.send_capacity_rows) __stcs((uint4 *)(a.send + (int64_t)row * a.row_bytes + off), v);
    for (int i = 0; i < nh; ++i) {
        if (!held_s[i]) continue;
        if (cnt_s[i] > 0) *(uint4 *)(held_s[i] + off) = v;
        else __stcs((uint4 *)(held_s[i] + off), v);
    }
    if (n2 == 0) return;
    // second level: every relay's copy is read back from where it is held and forwarded
    int k0 = 0;                                         // first forwarded copy of the hops of this batch
    for (int i0 = 0; i0 < nh; i0 += kRelayBatch) {
        uint4 w[kRelayBatch];
#pragma unroll
        for (int u = 0; u < kRelayBatch; ++u)
            if (i0 + u < nh && cnt_s[i0 + u] > 0 && held_s[i0 + u]) w[u] = ld_held(held_s[i0 + u] + off);
#pragma unroll
        for (int u = 0; u < kRelayBatch; ++u) {
            if (i0 + u >= nh) break;
            const int c = cnt_s[i0 + u];
            if (c > 0 && held_s[i0 + u])
                for (int k = k0; k < k0 + c; ++k)
                    if (dst_s[k]) __stcs((uint4 *)(dst_s[k] + off), w[u]);        // written once, not read again by this path
            k0 += c;
        }
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
    inner.flags &= ~(uint32_t)(MW_FLAG_HOST_STAGING | MW_FLAG_COPY_BULK);    // the relayed dispatch has one copy path
    int rc = mw_create(&r->hop, &inner);
    if (rc == MW_OK) rc = mw_create(&r->flat, &inner);
    if (rc == MW_OK) {
        r->hop->relay_src = cfg->src_rank;              // the first-level plan sees every rank as its next hop
        r->hop->relay_P = ranks_per_server;
        const size_t Kd = (size_t)r->hop->Kd, Tm = (size_t)cfg->max_tokens;
        r->Tm = (int64_t)Tm;
        const size_t b_n = round256(Tm * 4), b_plane = round256(Tm * Kd * 4);
        const size_t b_part = round256(((Tm + kDescThreads - 1) / kDescThreads) * kAccounts * sizeof(long long));
        const size_t bytes = b_n + 7 * b_plane + b_part + 256 + 256;
        if (cudaMalloc(&r->slab, bytes) != cudaSuccess) { cudaGetLastError(); rc = MW_ERR_CUDA; }
        else {
            uint8_t *p = (uint8_t *)r->slab;
            r->s2_n = (int32_t *)p; p += b_n;
            r->f1_rank = (int32_t *)p; p += b_plane;
            r->f1_pos = (int32_t *)p; p += b_plane;
            r->f1_flat = (int32_t *)p; p += b_plane;
            r->s2_cnt = (int32_t *)p; p += b_plane;
            r->s2_rank = (int32_t *)p; p += b_plane;
            r->s2_pos = (int32_t *)p; p += b_plane;
            r->s2_flat = (int32_t *)p; p += b_plane;
            r->block_part = (long long *)p; p += b_part;
            r->blocks_done = (unsigned int *)p; p += 256;
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
    MW_REFUSE_IF_POISONED(relay->hop);
    MW_REFUSE_IF_POISONED(relay->flat);
    cudaStream_t st = (cudaStream_t)stream;
    const mw_config &c = relay->hop->cfg;
    // the two plans do not depend on each other: next hops on the library's planning stream, final destinations here
    int rc = mw_plan_on_side_stream(relay->hop, topk_ids, expert_to_rank, T, st);
    if (rc == MW_OK) rc = mw_plan(relay->flat, topk_ids, expert_to_rank, T, nullptr, stream);
    if (rc != MW_OK) return rc;
    if (cudaStreamWaitEvent(st, relay->hop->ev_planned, 0) != cudaSuccess) return MW_ERR_CUDA;
    DescArgs a;
    a.T = T; a.Kd = relay->hop->Kd; a.R = c.R; a.src = c.src_rank; a.P = relay->P;
    a.Tm = relay->Tm; a.row_bytes = c.row_bytes;
    a.hop = relay->hop->d; a.flat = relay->flat->d;
    a.f1_rank = relay->f1_rank; a.f1_pos = relay->f1_pos; a.f1_flat = relay->f1_flat;
    a.s2_n = relay->s2_n; a.s2_cnt = relay->s2_cnt; a.s2_rank = relay->s2_rank; a.s2_pos = relay->s2_pos; a.s2_flat = relay->s2_flat;
    a.block_part = relay->block_part; a.blocks_done = relay->blocks_done;
    a.totals = relay->totals;
    // one thread per possible first-level send row; at least one block, which writes the totals
    const unsigned blocks = (unsigned)(T > 0 ? (T + kDescThreads - 1) / kDescThreads : 1);
    const size_t smem = sizeof(int32_t) * (size_t)(c.R + 1);
    if (a.Kd <= 8) k_relay_desc<8><<<blocks, kDescThreads, smem, st>>>(a);
    else if (a.Kd <= 16) k_relay_desc<16><<<blocks, kDescThreads, smem, st>>>(a);
    else k_relay_desc_any<<<blocks, kDescThreads, 0, st>>>(a);
    relay->hop->launches += 1;
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
    if (host_out->status == MW_ERR_TIMEOUT) { relay->hop->poisoned = 1; relay->flat->poisoned = 1; }
    return MW_OK;
}

int mw_relay_reset(mw_relay *relay)
{
    if (!relay) return MW_ERR_INVALID_ARG;
    int rc = mw_reset(relay->hop);
    if (rc == MW_OK) rc = mw_reset(relay->flat);
    if (rc == MW_OK && cudaMemset(relay->blocks_done, 0, sizeof(unsigned int)) != cudaSuccess) rc = MW_ERR_CUDA;
    relay->planned = 0;
    return rc;
}

int mw_relay_dispatch(mw_relay *relay, const void *x, void *send_buf, int64_t send_capacity_rows, void *hop_buf,
                      int64_t hop_capacity_rows, void *recv_base, int64_t recv_stride_bytes, int64_t recv_capacity_rows,
                      void *stream)
{
    if (!relay || !x || !send_buf || !hop_buf || !recv_base || send_capacity_rows < 0 || hop_capacity_rows < 0 ||
        recv_stride_bytes < 0 || recv_capacity_rows < 0)
        return MW_ERR_INVALID_ARG;
    MW_REFUSE_IF_POISONED(relay->hop);
    if (!relay->planned) return MW_ERR_NO_PLAN;
    if (!aligned16(x) || !aligned16(send_buf) || !aligned16(hop_buf) || !aligned16(recv_base) || recv_stride_bytes % 16)
        return MW_ERR_ALIGNMENT;
    mw_ctx *hop = relay->hop;
    if (recv_stride_bytes && recv_capacity_rows * hop->cfg.row_bytes > recv_stride_bytes) return MW_ERR_CAPACITY;
    if (hop->planned_T == 0) return MW_OK;
    RowsArgs f;
    f.x = (const uint8_t *)x;
    f.send = (uint8_t *)send_buf;
    f.hop_buf = (uint8_t *)hop_buf;
    f.recv = (uint8_t *)recv_base;
    f.row_bytes = hop->cfg.row_bytes;
    f.recv_stride = recv_stride_bytes;
    f.recv_capacity_rows = recv_capacity_rows;
    f.hop_capacity_rows = hop_capacity_rows;
    f.send_capacity_rows = send_capacity_rows;
    f.Tm = relay->Tm;
    f.Kd = hop->Kd;
    // near-equal pieces of at most kRelayMaxThreads 16-byte vectors; smaller ones while the grid would leave SMs idle
    const int64_t vecs = f.row_bytes / 16;
    int64_t pieces = (vecs + kRelayMaxThreads - 1) / kRelayMaxThreads;
    while ((int64_t)hop->planned_T * pieces < 4 * (int64_t)hop->sm_count && (vecs + pieces - 1) / pieces > 128) pieces *= 2;
    int threads = (int)(((vecs + pieces - 1) / pieces + 31) / 32 * 32);
    if (threads < MW_MAX_TOPK) threads = MW_MAX_TOPK;              // thread i resolves next hop i and forwarded copy i
    f.piece_bytes = threads * 16;
    f.pieces = (int)((f.row_bytes + f.piece_bytes - 1) / f.piece_bytes);
    if ((int64_t)hop->planned_T * f.pieces > 0x7fffffff) return MW_ERR_CAPACITY;
    f.src_index = hop->d.mw_row_token;
    f.row_ndest = hop->d.row_ndest;
    f.f1_rank = relay->f1_rank; f.f1_pos = relay->f1_pos; f.f1_flat = relay->f1_flat;
    f.s2_n = relay->s2_n; f.s2_cnt = relay->s2_cnt; f.s2_rank = relay->s2_rank; f.s2_pos = relay->s2_pos; f.s2_flat = relay->s2_flat;
    f.totals = hop->d.totals;
    const cudaError_t e = mw_launch(k_relay_rows, dim3((unsigned)((int64_t)hop->planned_T * f.pieces)), dim3(threads), 0,
                                    (cudaStream_t)stream, !(hop->cfg.flags & MW_FLAG_NO_OVERLAP), f);
    hop->launches += 1;
    if (e != cudaSuccess) { cudaGetLastError(); return MW_ERR_CUDA; }
    return MW_OK;
}

}  // extern "C"
