// mw_group_tokens_static: destination bitmaps and grouping of tokens for callers that cannot
// allocate device memory.  A variant of the bitmap/grouping kernel of the plan whose scratch (the
// table keyed by bitmap, and one slot index per token) lives in a fixed array inside the library
// image instead of a workspace obtained from cudaMalloc.  Declared and documented in include/mw.h.
#include <mutex>

#include "mw_internal.cuh"

namespace {

constexpr int kSlots = 2 * MW_STATIC_MAX_TOKENS;   // table size (power of two), load factor <= 0.5
constexpr int kEmpty = -1;
constexpr int kNoLeader = 0x7fffffff;
constexpr int kMaxDevices = 64;

struct StaticScratch {
    int32_t slot_rep[kSlots];      // token that first claimed the slot (identifies the stored bitmap)
    int32_t slot_leader[kSlots];   // smallest token index with that bitmap
    int32_t slot_count[kSlots];    // tokens with that bitmap
    int32_t token_slot[MW_STATIC_MAX_TOKENS];
};

// Lives in every GPU that loads the library, for the life of the process (448 KB).  In host code
// this name is only a handle for cudaGetSymbolAddress; kernels receive the device address.
static __device__ __align__(256) unsigned char g_static_scratch[sizeof(StaticScratch)];

std::mutex g_setup_mutex;
StaticScratch *g_scratch_of_device[kMaxDevices];   // device address of the array, per device ordinal

// The array keeps whatever the previous call left: start every call from an empty table.
__global__ void k_static_clear(StaticScratch *s, int32_t *status)
{
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < kSlots; i += gridDim.x * blockDim.x) {
        s->slot_rep[i] = kEmpty;
        s->slot_leader[i] = kNoLeader;
        s->slot_count[i] = 0;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) *status = MW_OK;
}

__global__ void __launch_bounds__(256) k_static_mask(StaticScratch *s, const int32_t *ids, const int32_t *e2r, int T,
                                                     int K, int E, int R, int W, uint64_t *token_mask,
                                                     int32_t *token_ndest, int32_t *status)
{
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    const int32_t *my = ids + (int64_t)t * K;
    uint64_t *m = token_mask + (int64_t)t * W;
    int nd = 0, bad = 0;
    uint64_t h = 0x2545f4914f6cdd1dull;
    // the token's words in token_mask are private to this thread: cleared, then one pass over the expert slots
    // (every id and table entry is loaded once, whatever W is), then read back for the count and the hash
    for (int w = 0; w < W; ++w) m[w] = 0;
    for (int k = 0; k < K; ++k) {
        const int id = my[k];
        if (id == -1) continue;
        if (id < 0 || id >= E) { bad = 1; continue; }
        const int r = e2r[id];
        if (r < 0 || r >= R) { bad = 1; continue; }
        m[r >> 6] |= 1ull << (r & 63);
    }
    for (int w = 0; w < W; ++w) {
        const uint64_t word = m[w];
        nd += __popcll(word);
        h = mix64(h, word);
    }
    token_ndest[t] = nd;
    if (bad) atomicCAS(status, MW_OK, MW_ERR_BAD_INDEX);
    int slot = kEmpty;
    if (nd > 0) {
        __threadfence();
        slot = (int)(h & (uint64_t)(kSlots - 1));
        for (int probes = 0; probes < kSlots; ++probes) {
            const int cur = atomicCAS(s->slot_rep + slot, kEmpty, t);
            if (cur == kEmpty) break;
            __threadfence();
            const uint64_t *o = token_mask + (int64_t)cur * W;
            bool same = true;
            for (int w = 0; w < W; ++w) same &= (__ldcg(o + w) == m[w]);
            if (same) break;
            slot = (slot + 1) & (kSlots - 1);
        }
        atomicMin(s->slot_leader + slot, t);
        atomicAdd(s->slot_count + slot, 1);
    }
    s->token_slot[t] = slot;
}

__global__ void __launch_bounds__(256) k_static_resolve(const StaticScratch *s, int T, int32_t *token_leader,
                                                        int32_t *token_group_size)
{
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    const int slot = s->token_slot[t];
    token_leader[t] = slot < 0 ? -1 : s->slot_leader[slot];
    token_group_size[t] = slot < 0 ? 0 : s->slot_count[slot];
}

// Device address of the array on the current device; looked up once per device.
int scratch_for_current_device(StaticScratch **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MW_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_of_device[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) { cudaGetLastError(); return MW_ERR_CUDA; }
        g_scratch_of_device[dev] = (StaticScratch *)p;
    }
    *out = g_scratch_of_device[dev];
    return MW_OK;
}

}  // namespace

extern "C" int mw_group_tokens_static(const int32_t *topk_ids, const int32_t *expert_to_rank, int32_t T, int32_t K,
                                      int32_t E, int32_t R, uint64_t *token_mask, int32_t *token_ndest,
                                      int32_t *token_leader, int32_t *token_group_size, int32_t *status, void *stream)
{
    if (T < 0 || K < 1 || K > MW_MAX_TOPK || E < 1 || R < 1 || R > MW_MAX_RANKS || !status ||
        (T > 0 && (!topk_ids || !expert_to_rank || !token_mask || !token_ndest || !token_leader || !token_group_size)))
        return MW_ERR_INVALID_ARG;
    if (T > MW_STATIC_MAX_TOKENS) return MW_ERR_CAPACITY;   // the fixed scratch holds at most this many tokens
    StaticScratch *s = nullptr;
    const int rc = scratch_for_current_device(&s);
    if (rc != MW_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    const int W = (R + 63) / 64;
    k_static_clear<<<64, 256, 0, st>>>(s, status);
    if (T > 0) {
        const int blocks = (T + 255) / 256;
        k_static_mask<<<blocks, 256, 0, st>>>(s, topk_ids, expert_to_rank, T, K, E, R, W, token_mask, token_ndest, status);
        k_static_resolve<<<blocks, 256, 0, st>>>(s, T, token_leader, token_group_size);
    }
    return cudaGetLastError() == cudaSuccess ? MW_OK : MW_ERR_CUDA;
}
