// Combine: the reverse of dispatch (paper, Section 2.3.2: results return from the experts to the
// sender; no redundant data, so MultiWrite leaves this step unchanged).  Declared in include/mw.h.
//
// y[t] = sum over the destinations of token t, ascending rank, of w[t, i] * z[rank_i][slot_i], bf16 rows,
// fp32 accumulation by fused multiply-add in that order, one rounding to bf16 (nearest even) at the end.
// HBM-bound gather: sum |D_t| rows read, T rows written.  A block handles (token, piece of the row) items;
// a thread owns 8 consecutive elements; many small blocks per SM keep enough row loads in flight.
#include "mw_internal.cuh"

namespace {

constexpr int kCombineMaxThreads = 256;
constexpr int kCombineMinBlocks = 6;                    // 40 registers per thread: 48 warps per SM measured fastest
constexpr int kCombineBatch = 4;                        // row loads a thread has in flight at once
constexpr int kCombineMaxDest = 64;                     // = MW_MAX_TOPK

struct CombineArgs {
    const uint8_t *z;
    int64_t z_stride, row_bytes;
    const float *weights;
    uint8_t *y;
    int T, Kd, pieces;          // a row is cut into `pieces` pieces of blockDim.x * 16 bytes (the last may be ragged)
    const int32_t *token_ndest, *dest_rank, *dest_pos, *rank_offsets;
    const mw_totals *totals;
};

__device__ __forceinline__ uint4 ldg16(const uint8_t *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// float -> bf16 bits, round to nearest even; NaN becomes the quiet NaN 0x7FC0
__device__ __forceinline__ uint32_t f32_to_bf16(float f)
{
    uint32_t u = __float_as_uint(f);
    if ((u & 0x7fffffffu) > 0x7f800000u) return 0x7fc0u;
    u += 0x7fffu + ((u >> 16) & 1u);
    return u >> 16;
}

// Descriptor of destination i of one token, fetched by thread i.
struct CombineDesc {
    const uint8_t *src;
    float w;
};

__device__ __forceinline__ CombineDesc combine_fetch(const CombineArgs &a, int t, int i)
{
    CombineDesc d = {nullptr, 0.0f};
    if (i >= a.Kd) return d;
    const int r = a.dest_rank[(int64_t)t * a.Kd + i], p = a.dest_pos[(int64_t)t * a.Kd + i];
    if (r < 0) return d;                                                    // beyond the token's destinations
    d.w = a.weights ? a.weights[(int64_t)t * a.Kd + i] : 1.0f;
    d.src = a.z + (a.z_stride ? (int64_t)r * a.z_stride + (int64_t)p * a.row_bytes
                              : ((int64_t)a.rank_offsets[r] + p) * a.row_bytes);
    return d;
}

// One block per (token, piece) item, the pieces of a row adjacent in the grid.  Thread i fetches the descriptor of destination i; all threads then load
// their 16 bytes of every destination's row (kCombineBatch loads in flight per thread) and accumulate in rank order.
__global__ void __launch_bounds__(kCombineMaxThreads, kCombineMinBlocks) k_combine(const __grid_constant__ CombineArgs a)
{
    __shared__ const uint8_t *src_s[kCombineMaxDest];
    __shared__ float w_s[kCombineMaxDest];
    if (a.totals->status != MW_OK) return;      // the plan failed: its arrays are not to be trusted
    const int tid = threadIdx.x;
    // 32-bit on purpose: a 64-bit division here sits on the path to the first load and cost 12 % of the run time
    const int t = blockIdx.x / a.pieces, piece = blockIdx.x % a.pieces;
    const int nd = a.token_ndest[t];
    {
        const CombineDesc d = combine_fetch(a, t, tid);
        if (tid < a.Kd) { src_s[tid] = d.src; w_s[tid] = d.w; }
    }
    __syncthreads();
    const int64_t off = ((int64_t)piece * blockDim.x + tid) * 16;
    if (off >= a.row_bytes) return;
    float acc[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) acc[k] = 0.0f;
    for (int i0 = 0; i0 < nd; i0 += kCombineBatch) {
        uint4 v[kCombineBatch];
#pragma unroll
        for (int j = 0; j < kCombineBatch; ++j)
            if (i0 + j < nd) v[j] = ldg16(src_s[i0 + j] + off);
#pragma unroll
        for (int j = 0; j < kCombineBatch; ++j) {
            if (i0 + j >= nd) break;
            const float w = w_s[i0 + j];
            const uint32_t q[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                acc[2 * k] = fmaf(w, __uint_as_float(q[k] << 16), acc[2 * k]);              // bf16 -> f32: bits << 16
                acc[2 * k + 1] = fmaf(w, __uint_as_float(q[k] & 0xffff0000u), acc[2 * k + 1]);
            }
        }
    }
    uint4 o;
    o.x = nd ? (f32_to_bf16(acc[0]) | (f32_to_bf16(acc[1]) << 16)) : 0u;
    o.y = nd ? (f32_to_bf16(acc[2]) | (f32_to_bf16(acc[3]) << 16)) : 0u;
    o.z = nd ? (f32_to_bf16(acc[4]) | (f32_to_bf16(acc[5]) << 16)) : 0u;
    o.w = nd ? (f32_to_bf16(acc[6]) | (f32_to_bf16(acc[7]) << 16)) : 0u;
    *(uint4 *)(a.y + (int64_t)t * a.row_bytes + off) = o;
}

}  // namespace

extern "C" int mw_combine(mw_ctx *ctx, const void *z_base, int64_t z_stride_bytes, const float *weights, void *y, void *stream)
{
    if (!ctx || !z_base || !y || z_stride_bytes < 0) return MW_ERR_INVALID_ARG;
    MW_REFUSE_IF_POISONED(ctx);
    if (ctx->planned_T < 0) return MW_ERR_NO_PLAN;
    if (((uintptr_t)z_base & 15u) || ((uintptr_t)y & 15u) || z_stride_bytes % 16 || ((uintptr_t)weights & 3u)) return MW_ERR_ALIGNMENT;
    const int T = ctx->planned_T;
    if (T == 0) return MW_OK;
    CombineArgs a;
    a.z = (const uint8_t *)z_base; a.z_stride = z_stride_bytes; a.row_bytes = ctx->cfg.row_bytes;
    a.weights = weights; a.y = (uint8_t *)y;
    a.T = T; a.Kd = ctx->Kd;
    // pieces of at most 256 vectors of 16 bytes, sized so that the last one is as full as the others
    const int64_t vecs = ctx->cfg.row_bytes / 16;
    a.pieces = (int)((vecs + kCombineMaxThreads - 1) / kCombineMaxThreads);
    if ((int64_t)T * a.pieces > 0x7fffffff) return MW_ERR_CAPACITY;
    int threads = (int)(((vecs + a.pieces - 1) / a.pieces + 31) / 32 * 32);
    if (threads < kCombineMaxDest) threads = kCombineMaxDest;              // thread i fetches the descriptor of destination i
    a.token_ndest = ctx->d.token_ndest; a.dest_rank = ctx->d.dest_rank; a.dest_pos = ctx->d.dest_pos;
    a.rank_offsets = ctx->d.rank_offsets; a.totals = ctx->d.totals;
    const cudaError_t e = mw_launch(k_combine, dim3((unsigned)((int64_t)T * a.pieces)), dim3(threads), 0,
                                    (cudaStream_t)stream, false, a);
    ctx->launches += 1;
    if (e != cudaSuccess) { cudaGetLastError(); return MW_ERR_CUDA; }
    return MW_OK;
}
