// Source-side planning kernels: destination bitmaps with per-rank dedup, grouping of tokens by
// identical bitmap, per-group and per-rank counts with exclusive prefix sums, and every token's
// send row and receive slots.  (Paper: Section 4.1, metadata encoding at the source; Section 5.1,
// task decomposition in cs_send.  The slot layout rules are stated in mw.h.)
//
// Two ways to run the same three phases:
//   k_plan_fused  one launch, one block per 256-token tile, all blocks resident, the
//                 phases separated by two bounded grid barriers; a token's values stay in the
//                 registers of "its" thread from phase to phase.  Taken whenever the tiles fit on
//                 the SMs (T <= 256 x SM count).
//   multi-pass    three kernels chained on one stream, for larger T (or MW_FLAG_PLAN_MULTIPASS):
//   k_plan_mask   one thread per token: bitmap words, |D_t|, insertion of the bitmap into an
//                 open-addressed table whose slot value is the smallest token index seen
//                 (atomicMin), which makes the group "leader" independent of thread order;
//   k_plan_tile   one block per 256-token tile, tiles taken in ticket order: a rank x token
//                 bit matrix in shared memory gives every (token, rank) its position inside
//                 the tile, the per-tile histogram of R rank counts (+ leader count, + group
//                 size sum) is combined across tiles by a decoupled look-back scan, and the
//                 last tile turns the grand totals into rank_offsets and the byte accounting;
//   k_plan_final  one thread per token: group id / offset looked up at the leader, rank inside
//                 the group, send row, inverse maps, per-row delivery descriptors; also restores
//                 the table to its empty state for the next plan.
#include "mw_internal.cuh"

namespace {

constexpr int kEmpty = -1;
constexpr unsigned long long kEmptyKey = ~0ull;
constexpr int kNoLeader = 0x7fffffff;
constexpr unsigned kFlagAgg = 1u, kFlagPrefix = 2u;

struct PlanArgs {
    const int32_t *ids, *e2r;
    int T, K, E, R, W, Kd, src_rank, ntiles, NC, hs_mask, Tm;
    int relay_src, relay_P;   // relay_P > 0: a rank stands for its next hop as seen from relay_src (first level of a relayed dispatch)
    int64_t row_bytes;
    uint32_t skew_epoch;      // test hook: added to the epoch a look-back expects in its predecessors' records (0 normally)
    uint32_t skew_bar;        // test hook: added to the arrival count the grid barriers wait for (0 normally)
    int spin_limit;           // look-back polls before a tile gives up (2^20: about a second)
    int bar_spin_limit;       // polls of the arrival counter before a block gives up at a grid barrier
    const uint8_t *pf_base;   // rows to bring into L2 while the plan runs (fused plan only), or null
    int64_t pf_bytes;
    mw_dev d;
};

__device__ __forceinline__ void set_status(int *status, int err) { atomicCAS(status, 0, err); }

// The running counts of a context's plans live in device memory (mw_dev::plan_state), so that a plan launch carries no
// host-side state and a captured launch can be replayed: every block reads them when it starts; the plan's last tile
// advances them when everything that depends on them is done.  Plans of a context never overlap.
struct PlanCounters {
    uint32_t epoch;        // number of this plan, 30 bits (look-back records carry it, so they need no clearing)
    uint32_t wait_epoch;   // epoch expected in predecessors' records
    uint32_t ticket_base;  // tile tickets handed out by all previous multi-kernel plans
    uint32_t bar_base;     // grid-barrier arrivals made by all previous fused plans (plus the test skew)
};

__device__ __forceinline__ PlanCounters load_counters(const PlanArgs &a)
{
    const volatile mw_plan_state *st = a.d.plan_state;
    const uint32_t plans = st->plans, tickets = st->tickets, bars = st->bars;
    PlanCounters pc;
    pc.epoch = (plans + 1u) & 0x3fffffffu;
    pc.wait_epoch = (pc.epoch + a.skew_epoch) & 0x3fffffffu;
    pc.ticket_base = tickets;
    pc.bar_base = bars + a.skew_bar;
    return pc;
}

// Called by one thread of the plan's last tile, after every block has read the counters.
__device__ __forceinline__ void advance_counters(const PlanArgs &a, uint32_t tickets_taken, uint32_t barrier_arrivals)
{
    mw_plan_state *st = a.d.plan_state;
    st->plans += 1u;
    st->tickets += tickets_taken;
    st->bars += barrier_arrivals;
}

// The 30-bit epoch is about to start a new lap: the last tile of the lap's last plan wipes the look-back records, once
// every look-back of the plan is done (all threads of the block call this).
__device__ __forceinline__ void wipe_records_at_lap_end(const PlanArgs &a, uint32_t epoch)
{
    if (epoch != 0x3fffffffu) return;
    const size_t n = (size_t)((a.Tm + MW_TILE - 1) / MW_TILE) * (size_t)a.NC;
    for (size_t i = threadIdx.x; i < n; i += blockDim.x) a.d.tile_state[i] = 0ull;
}

// A wait gave up: the plan under way is invalid, and it will not restore the shared scratch (bitmap table, counters)
// to the state the next plan expects.  The flag makes every later plan on the context refuse to run until mw_reset
// has re-initialised the scratch, also when the host has not looked at the status in between.
__device__ __forceinline__ void give_up(const PlanArgs &a, int *status)
{
    set_status(status, MW_ERR_TIMEOUT);
    *(volatile unsigned int *)a.d.gave_up = 1u;
    __threadfence();                         // both are visible before anything this thread publishes afterwards
}
// True (and the slot's accounting says MW_ERR_TIMEOUT) if an earlier plan on this context gave up.
__device__ __forceinline__ bool refuses_to_plan(const PlanArgs &a)
{
    if (*(volatile const unsigned int *)a.d.gave_up == 0u) return false;
    if (blockIdx.x == 0 && threadIdx.x == 0) a.d.totals->status = MW_ERR_TIMEOUT;
    return true;
}


// Finds (or claims) the table slot of a bitmap.  A slot holds (32-bit hash tag, first token that
// claimed it); a probe that meets another tag moves on after one CAS, and the full bitmap is only
// compared when the tags agree.  Returns -1 if the table is full (cannot happen at load <= 1/8).
template <class SameFn>
__device__ __forceinline__ int table_insert(unsigned long long *slot_key, int hs_mask, uint64_t h, int t, SameFn same_as)
{
    const uint32_t tag = (uint32_t)(h >> 32);
    const unsigned long long mine = ((unsigned long long)tag << 32) | (uint32_t)t;
    int slot = (int)(h & (uint64_t)hs_mask);
    for (int probes = 0; probes <= hs_mask; ++probes) {
        const unsigned long long cur = atomicCAS(slot_key + slot, kEmptyKey, mine);
        if (cur == kEmptyKey) return slot;                                // claimed an empty slot
        if ((uint32_t)(cur >> 32) == tag) {
            __threadfence();
            if (same_as((int)(uint32_t)cur)) return slot;                 // slot already holds this bitmap
        }
        slot = (slot + 1) & hs_mask;
    }
    return -1;
}

// One-word bitmaps with fewer than 64 bits set can never equal the all-ones empty marker, so the bitmap itself
// is the key: no tag, no comparison with another token's bitmap, and nothing that must be visible beforehand.
__device__ __forceinline__ int table_insert_word(unsigned long long *slot_key, int hs_mask, uint64_t h, unsigned long long word)
{
    int slot = (int)(h & (uint64_t)hs_mask);
    for (int probes = 0; probes <= hs_mask; ++probes) {
        const unsigned long long cur = atomicCAS(slot_key + slot, kEmptyKey, word);
        if (cur == kEmptyKey || cur == word) return slot;
        slot = (slot + 1) & hs_mask;
    }
    return -1;
}

// ------------------------------------------------------------------------------------------
// Kernel 1: bitmaps (Section 4.1: bit r set <=> rank r is a target) and the bitmap table.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(MW_TILE) k_plan_mask(PlanArgs a)
{
    if (refuses_to_plan(a)) return;
    const PlanCounters pc = load_counters(a);
    const int t = blockIdx.x * MW_TILE + threadIdx.x;
    mw_acc *acc = a.d.acc + (pc.epoch & 1u);
    int valid = 0, self_only = 0, bad = 0;
    if (t < a.T) {
        const int32_t *my = a.ids + (int64_t)t * a.K;
        uint64_t *m = a.d.token_mask + (int64_t)t * a.W;
        int nd = 0;
        uint64_t h = 0x2545f4914f6cdd1dull, self_word = 0;
        for (int w = 0; w < a.W; ++w) {
            uint64_t word = 0;
            for (int k = 0; k < a.K; ++k) {
                const int id = my[k];
                if (id == -1) continue;                               // padding slot
                if (id < 0 || id >= a.E) { bad |= (w == 0); continue; }
                int r = a.e2r[id];
                if (r < 0 || r >= a.R) { bad |= (w == 0); continue; }
                if (a.relay_P > 0) r = mw_next_hop(r, a.relay_src, a.relay_P);    // one copy per distinct next hop (Section 4.1)
                valid += (w == 0);
                if ((r >> 6) == w) word |= 1ull << (r & 63);          // OR = per-rank dedup
            }
            m[w] = word;
            nd += __popcll(word);
            h = mix64(h, word);
            if (a.src_rank >= 0 && (a.src_rank >> 6) == w) self_word = word & (1ull << (a.src_rank & 63));
        }
        a.d.token_ndest[t] = nd;
        self_only = (nd == 1 && self_word != 0);
        int slot = kEmpty;
        if (nd > 0) {
            __threadfence();                                          // bitmap visible before the slot is claimed
            const int W = a.W;
            const uint64_t *masks = a.d.token_mask;
            slot = table_insert(a.d.slot_key, a.hs_mask, h, t, [=](int other) {
                bool same = true;
                for (int w = 0; w < W; ++w) same &= (__ldcg(masks + (int64_t)other * W + w) == m[w]);
                return same;
            });
            if (slot < 0) { set_status(&acc->status, MW_ERR_CAPACITY); a.d.token_ndest[t] = 0; }
            else { atomicMin(a.d.slot_leader + slot, t); atomicAdd(a.d.slot_count + slot, 1); }
        }
        a.d.token_slot[t] = slot;
    }
    valid = __reduce_add_sync(0xffffffffu, valid);
    self_only = __reduce_add_sync(0xffffffffu, self_only);
    bad = __reduce_or_sync(0xffffffffu, (unsigned)bad);
    if ((threadIdx.x & 31) == 0) {
        if (valid) atomicAdd(&acc->valid_slots, (unsigned long long)valid);
        if (self_only) atomicAdd(&acc->self_only, (unsigned)self_only);
        if (bad) set_status(&acc->status, MW_ERR_BAD_INDEX);
    }
}

// Exclusive prefix sum over the 256 threads of a block; `total` is returned to every thread.
__device__ __forceinline__ int block_excl_scan(int v, int *warp_sums /* [8] shared */, int &total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { int n = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += n; }
    __syncthreads();                       // protects warp_sums from a previous use
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    int before = 0, sum = 0;
#pragma unroll
    for (int w = 0; w < MW_TILE / 32; ++w) { int s = warp_sums[w]; if (w < warp) before += s; sum += s; }
    total = sum;
    return before + incl - v;
}

__device__ __forceinline__ unsigned long long pack_state(uint32_t epoch, unsigned flag, uint32_t value)
{
    return ((unsigned long long)((epoch << 2) | flag) << 32) | value;
}

// ------------------------------------------------------------------------------------------
// Kernel 2: per-tile histogram + decoupled look-back scan over tiles; positions inside regions.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(MW_TILE) k_plan_tile(PlanArgs a)
{
    extern __shared__ uint32_t sm[];
    uint32_t *bits = sm;                          // [R, 8]  bit i of word w: token 32 w + i of the tile targets rank r
    uint32_t *pre = bits + (size_t)a.R * 8;       // [R, 8]  tokens of the tile before word w that target rank r
    int *cnt = (int *)(pre + (size_t)a.R * 8);    // [NC]    this tile's counters
    int *base = cnt + a.NC;                       // [NC]    sum of the counters of all earlier tiles
    __shared__ int warp_sums[MW_TILE / 32];
    __shared__ int s_tile;

    if (refuses_to_plan(a)) return;
    const PlanCounters pc = load_counters(a);      // read before the ticket is taken: the tile with the last ticket advances them
    const int tid = threadIdx.x;
    mw_acc *acc = a.d.acc + (pc.epoch & 1u);
    // Tiles are numbered in the order blocks start, so a tile only ever waits for tiles that are already running.
    if (tid == 0) s_tile = (int)(atomicAdd(a.d.ticket, 1u) - pc.ticket_base);
    for (int i = tid; i < a.R * 8; i += MW_TILE) bits[i] = 0;
    __syncthreads();
    const int tile = s_tile;
    const int t = tile * MW_TILE + tid;
    const bool active = t < a.T;
    const int nd = active ? a.d.token_ndest[t] : 0;
    int leader = -1, gcount = 0;
    if (nd > 0) {
        const int slot = a.d.token_slot[t];
        leader = a.d.slot_leader[slot];
        gcount = a.d.slot_count[slot];
    }
    const bool is_leader = nd > 0 && leader == t;
    if (active) { a.d.token_leader[t] = leader; a.d.token_gcount[t] = gcount; }

    const uint64_t *m = a.d.token_mask + (int64_t)t * a.W;
    const int wi = tid >> 5;
    const uint32_t bit = 1u << (tid & 31);
    if (nd > 0)
        for (int w = 0; w < a.W; ++w)
            for (uint64_t word = m[w]; word; word &= word - 1)
                atomicOr(bits + (size_t)(w * 64 + __ffsll((long long)word) - 1) * 8 + wi, bit);
    __syncthreads();
    for (int r = tid; r < a.R; r += MW_TILE) {
        int run = 0;
#pragma unroll
        for (int w8 = 0; w8 < 8; ++w8) { pre[r * 8 + w8] = run; run += __popc(bits[r * 8 + w8]); }
        cnt[r] = run;
    }
    int lead_total, gc_total;
    const int lead_excl = block_excl_scan(is_leader ? 1 : 0, warp_sums, lead_total);
    const int gc_excl = block_excl_scan(is_leader ? gcount : 0, warp_sums, gc_total);
    if (tid == 0) { cnt[a.R] = lead_total; cnt[a.R + 1] = gc_total; }
    __syncthreads();

    // Decoupled look-back, one thread per counter.  A record is one 64-bit word (epoch, flag, value),
    // so flag and value are always read together; the epoch makes records of earlier plans invisible.
    for (int c = tid; c < a.NC; c += MW_TILE) {
        const uint32_t mine = (uint32_t)cnt[c];
        volatile unsigned long long *rec = a.d.tile_state + (size_t)tile * a.NC + c;
        uint32_t excl = 0;
        if (tile == 0) {
            *rec = pack_state(pc.epoch, kFlagPrefix, mine);
        } else {
            *rec = pack_state(pc.epoch, kFlagAgg, mine);
            for (int j = tile - 1; j >= 0; --j) {
                volatile unsigned long long *prev = a.d.tile_state + (size_t)j * a.NC + c;
                unsigned long long s = 0;
                int spins = 0;
                for (; spins < a.spin_limit; ++spins) {
                    s = *prev;
                    const uint32_t hi = (uint32_t)(s >> 32);
                    if ((hi >> 2) == pc.wait_epoch && (hi & 3u) != 0) break;
                    __nanosleep(64);
                }
                if (spins == a.spin_limit) { give_up(a, &acc->status); break; }
                excl += (uint32_t)s;
                if (((uint32_t)(s >> 32) & 3u) == kFlagPrefix) break;
            }
            *rec = pack_state(pc.epoch, kFlagPrefix, excl + mine);
        }
        base[c] = (int)excl;
    }
    __syncthreads();

    if (active) {
        if (is_leader) { a.d.gid_at[t] = base[a.R] + lead_excl; a.d.goff_at[t] = base[a.R + 1] + gc_excl; }
        int i = 0;
        int32_t *dr = a.d.dest_rank + (int64_t)t * a.Kd, *dp = a.d.dest_pos + (int64_t)t * a.Kd;
        if (nd > 0)
            for (int w = 0; w < a.W; ++w)
                for (uint64_t word = m[w]; word; word &= word - 1) {
                    const int r = w * 64 + __ffsll((long long)word) - 1;
                    dr[i] = r;
                    dp[i] = base[r] + (int)pre[r * 8 + wi] + __popc(bits[r * 8 + wi] & (bit - 1));
                    ++i;
                }
        for (; i < a.Kd; ++i) { dr[i] = -1; dp[i] = -1; }
    }

    if (tile == a.ntiles - 1) {
        // This tile's inclusive prefix is the grand total of every counter.
        int carry = 0;
        for (int r0 = 0; r0 < a.R; r0 += MW_TILE) {
            const int r = r0 + tid;
            const int v = r < a.R ? base[r] + cnt[r] : 0;
            int total;
            const int excl = block_excl_scan(v, warp_sums, total);
            if (r < a.R) a.d.rank_offsets[r] = carry + excl;
            carry += total;
        }
        if (tid == 0) {
            const int64_t G = base[a.R] + cnt[a.R], Tn = base[a.R + 1] + cnt[a.R + 1], SD = carry;
            const int64_t self_copies = a.src_rank >= 0 ? base[a.src_rank] + cnt[a.src_rank] : 0;
            const int64_t sent_rows = Tn - (int64_t)acc->self_only;
            a.d.rank_offsets[a.R] = (int32_t)SD;
            a.d.group_offsets[G] = (int32_t)Tn;
            mw_totals tt;
            tt.T_nonempty = Tn;
            tt.G = G;
            tt.total_dest = SD;
            tt.mw_bytes = sent_rows * a.row_bytes;
            tt.unicast_bytes = (SD - self_copies) * a.row_bytes;
            tt.unicast_per_expert_bytes = (int64_t)acc->valid_slots * a.row_bytes;
            // Section 6.4: beyond 64 ranks the bitmap travels in the payload, once per 4096-byte packet
            tt.meta_bytes = a.R <= 64 ? 0 : sent_rows * ((a.row_bytes + 4095) / 4096) * (int64_t)(8 * a.W);
            tt.status = acc->status;
            tt.reserved = 0;
            *a.d.totals = tt;
            mw_acc *next = a.d.acc + ((pc.epoch + 1u) & 1u);
            next->valid_slots = 0; next->self_only = 0; next->status = 0;
            advance_counters(a, (uint32_t)a.ntiles, 0u);     // every tile has read them (it took its ticket afterwards)
        }
        wipe_records_at_lap_end(a, pc.epoch);                // this tile's look-back ended last: no record is needed any more
    }
}

// ------------------------------------------------------------------------------------------
// Rank of every token inside its group (number of members with a smaller token index), for one
// 256-token tile, computed by the whole block.  Only groups with more than one member need work:
//   - the tile's distinct multi-member leaders go into a small shared-memory hash (key = leader);
//     each entry has a 256-bit bitmap of the tile's members, whose popcount prefix gives the rank
//     inside the tile, and a counter of members seen in earlier tiles;
//   - every earlier tile, from the tile of the smallest such leader on, is read once (coalesced,
//     eight independent loads per round) and each value is looked up in the hash.
// A group's first member is its leader, so no member lives before the leader's tile.
// ------------------------------------------------------------------------------------------
constexpr int kRankSlots = 512;      // shared hash slots: at most 256 distinct leaders per tile
struct RankScratch {
    int key[kRankSlots];             // leader token index, -1 = empty
    int earlier[kRankSlots];         // members in earlier tiles
    uint32_t members[kRankSlots][8]; // bit i of word w: token 32 w + i of this tile is a member
    int first_tile;                  // smallest tile that holds one of the tile's multi-member leaders
};

__device__ __forceinline__ int rank_slot_find(const int *key, int leader)
{
    int e = (int)(((uint32_t)leader * 2654435761u) >> 23) & (kRankSlots - 1);
    while (true) {
        const int k = key[e];
        if (k == leader) return e;
        if (k == -1) return -1;
        e = (e + 1) & (kRankSlots - 1);
    }
}

// `leader` is -1 for a token without destinations; `gcount` its group size; `token_leader` is the
// global array holding the leader of every token (complete before this is called).  All threads of
// the block must call it.
__device__ int group_rank_in_tile(RankScratch *rs, const int32_t *token_leader, int tile, int leader, int gcount)
{
    const int tid = threadIdx.x;
    const bool multi = leader >= 0 && gcount > 1;
    if (!__syncthreads_or(multi)) return 0;                       // every group of this tile is a singleton
    for (int i = tid; i < kRankSlots; i += MW_TILE) {
        rs->key[i] = -1; rs->earlier[i] = 0;
#pragma unroll
        for (int w = 0; w < 8; ++w) rs->members[i][w] = 0;
    }
    if (tid == 0) rs->first_tile = tile;
    __syncthreads();
    int e = -1;
    if (multi) {
        e = (int)(((uint32_t)leader * 2654435761u) >> 23) & (kRankSlots - 1);
        while (true) {
            const int k = atomicCAS(rs->key + e, -1, leader);
            if (k == -1 || k == leader) break;
            e = (e + 1) & (kRankSlots - 1);
        }
        atomicOr(&rs->members[e][tid >> 5], 1u << (tid & 31));
        atomicMin(&rs->first_tile, leader / MW_TILE);
    }
    __syncthreads();
    const int first_tile = rs->first_tile;
    for (int j0 = first_tile; j0 < tile; j0 += 8) {
        int v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = (j0 + i < tile) ? __ldcg(token_leader + (int64_t)(j0 + i) * MW_TILE + tid) : -1;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (v[i] < 0) continue;
            const int f = rank_slot_find(rs->key, v[i]);
            if (f >= 0) atomicAdd(rs->earlier + f, 1);
        }
    }
    __syncthreads();
    int within = 0;
    if (multi) {
        within = rs->earlier[e];
        const int wi = tid >> 5;
        for (int w = 0; w < wi; ++w) within += __popc(rs->members[e][w]);
        within += __popc(rs->members[e][wi] & ((1u << (tid & 31)) - 1u));
    }
    return within;
}

// ------------------------------------------------------------------------------------------
// Kernel 3: group ids and send rows, inverse maps, delivery descriptors, table clean-up.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(MW_TILE) k_plan_final(PlanArgs a)
{
    __shared__ RankScratch rank_scratch;
    const int t = blockIdx.x * MW_TILE + threadIdx.x;
    const mw_totals *tot = a.d.totals;
    if (tot->status == MW_ERR_TIMEOUT) return;      // a look-back gave up (now or in an earlier plan): nothing below can be trusted
    const int Tn = (int)tot->T_nonempty, G = (int)tot->G, SD = (int)tot->total_dest;
    if (t <= a.T && t > G) a.d.group_offsets[t] = -1;
    if (t < a.T) {
        if (t >= Tn) a.d.mw_row_token[t] = -1;
        for (int i = 0; i < a.Kd; ++i)
            if ((int64_t)t * a.Kd + i >= SD) a.d.rank_tokens[(int64_t)t * a.Kd + i] = -1;
        for (int w = 0; w < a.W; ++w)
            if (t >= G) a.d.group_mask[(int64_t)t * a.W + w] = 0;
    }
    const int leader = t < a.T ? a.d.token_leader[t] : -1;
    const int gcount = leader >= 0 ? a.d.token_gcount[t] : 0;
    const int within = group_rank_in_tile(&rank_scratch, a.d.token_leader, blockIdx.x, leader, gcount);
    if (t >= a.T) return;
    if (leader < 0) { a.d.token_group[t] = -1; a.d.token_mw_row[t] = -1; return; }
    const int g = a.d.gid_at[leader], goff = a.d.goff_at[leader];
    const int row = goff + within;
    a.d.token_group[t] = g;
    a.d.token_mw_row[t] = row;
    a.d.mw_row_token[row] = t;
    const int nd = a.d.token_ndest[t];
    a.d.row_ndest[row] = nd;
    if (leader == t) {
        a.d.group_offsets[g] = goff;
        for (int w = 0; w < a.W; ++w) a.d.group_mask[(int64_t)g * a.W + w] = a.d.token_mask[(int64_t)t * a.W + w];
    }
    for (int i = 0; i < a.Kd; ++i) {
        const int r = a.d.dest_rank[(int64_t)t * a.Kd + i], p = a.d.dest_pos[(int64_t)t * a.Kd + i];
        a.d.row_dest_rank[(int64_t)i * a.Tm + row] = r;
        a.d.row_dest_pos[(int64_t)i * a.Tm + row] = p;
        int at = -1;
        if (r >= 0) {
            at = a.d.rank_offsets[r] + p;
            a.d.rank_tokens[at] = t;
        }
        a.d.row_dest_flat[(int64_t)i * a.Tm + row] = at;
    }
    // leave the bitmap table empty for the next plan
    const int slot = a.d.token_slot[t];
    a.d.slot_key[slot] = kEmptyKey;
    a.d.slot_leader[slot] = kNoLeader;
    a.d.slot_count[slot] = 0;
}

// ------------------------------------------------------------------------------------------
// Fused plan: the three phases in one launch.
// ------------------------------------------------------------------------------------------
constexpr int kLookBack = 8;                  // predecessors a look-back reads per round trip (16 measured slower: more records not ready yet)

__device__ __forceinline__ unsigned int ld_volatile_u32(const unsigned int *p)
{
    unsigned int v;
    asm volatile("ld.volatile.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Grid barrier in two halves, so that work which does not depend on the other blocks can run between
// them.  Every block always arrives, so the running count of arrivals stays exact even after a
// block has given up waiting.
__device__ __forceinline__ void grid_barrier_arrive(unsigned int *counter)
{
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(counter, 1u);
    }
}

// A block that is still `alive` waits until the counter reaches `target`; returns false for a block
// that gave up (now or before).  With a single block, block-level ordering is all that is needed.
__device__ bool grid_barrier_wait(const PlanArgs &a, unsigned int target, bool alive, int *status)
{
    __shared__ int s_alive;
    if (gridDim.x == 1) {
        __syncthreads();
        return alive;
    }
    if (threadIdx.x == 0) {
        int ok = alive ? 1 : 0;
        if (ok) {
            int spins = 0;
            while ((int)(ld_volatile_u32(a.d.gbar) - target) < 0) {
                if (++spins > a.bar_spin_limit) { ok = 0; give_up(a, status); break; }
                __nanosleep(32);
            }
        }
        __threadfence();
        s_alive = ok;
    }
    __syncthreads();
    return s_alive != 0;
}

template <int WT>
__global__ void __launch_bounds__(MW_TILE) k_plan_fused(PlanArgs a)
{
    extern __shared__ uint32_t sm[];
    uint32_t *bits = sm;
    uint32_t *pre = bits + (size_t)a.R * 8;
    int *cnt = (int *)(pre + (size_t)a.R * 8);
    int *base = cnt + a.NC;
    __shared__ int warp_sums[MW_TILE / 32];
    __shared__ RankScratch rank_scratch;

    const int tid = threadIdx.x, tile = blockIdx.x;
    grid_launch_dependents();      // the pack kernel may set itself up while the plan runs
    if (tile >= a.ntiles) {
        // Blocks beyond the tiles take no part in the plan.  The plan is a chain of round trips on a few SMs and
        // leaves the memory system idle, so these blocks ask L2 for the hidden rows the pack step reads next.
        // One request covers 16 KB.  Measured on B200 (4096 rows of 14336 bytes, 16 plan tiles): requests of 8 to 16 KB
        // from every thread of the first blocks cost the plan 3.7 us and save the pack step 6 us; 2 to 4 KB requests, or
        // fewer requesting threads, save less; 32 KB and larger requests stall the requesting SMs for tens of microseconds.
        constexpr int64_t kPiece = 16384;
        const int64_t first = ((int64_t)(tile - a.ntiles) * MW_TILE + tid) * kPiece;
        const int64_t stride = (int64_t)((int)gridDim.x - a.ntiles) * MW_TILE * kPiece;
        for (int64_t off = first; off < a.pf_bytes; off += stride) {
            const uint32_t n = (uint32_t)min(kPiece, a.pf_bytes - off);       // a multiple of 16 (rows are)
            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(a.pf_base + off), "r"(n) : "memory");
        }
        return;
    }
    if (refuses_to_plan(a)) return;      // uniform over the grid (the flag only changes between plans): no block waits for another
    const PlanCounters pc = load_counters(a);
    const int t = tile * MW_TILE + tid;
    const bool active = t < a.T;
    mw_acc *acc = a.d.acc + (pc.epoch & 1u);
    for (int i = tid; i < a.R * 8; i += MW_TILE) bits[i] = 0;

    // ---- phase A: bitmap (Section 4.1: bit r set <=> rank r is a target) and the bitmap table ----
    uint64_t m[WT];
#pragma unroll
    for (int w = 0; w < WT; ++w) m[w] = 0;
    int nd = 0, slot = kEmpty;
    {
        int valid = 0, bad = 0, self_only = 0;
        if (active) {
            const int32_t *my = a.ids + (int64_t)t * a.K;
            for (int k0 = 0; k0 < a.K; k0 += 8) {
                int id[8], r[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) id[j] = (k0 + j < a.K) ? my[k0 + j] : -1;      // 8 independent loads
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const bool ok = id[j] >= 0 && id[j] < a.E;
                    bad |= (id[j] != -1 && !ok);
                    r[j] = ok ? a.e2r[id[j]] : -1;                                          // 8 independent loads
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const bool ok = r[j] >= 0 && r[j] < a.R;
                    bad |= (id[j] >= 0 && id[j] < a.E && !ok);
                    valid += ok;
                    if (a.relay_P > 0 && ok) r[j] = mw_next_hop(r[j], a.relay_src, a.relay_P);   // one copy per distinct next hop (Section 4.1)
                    const uint64_t rank_bit = ok ? 1ull << (r[j] & 63) : 0ull;
#pragma unroll
                    for (int w = 0; w < WT; ++w) m[w] |= rank_bit & equal_mask64(r[j] >> 6, w);   // OR = per-rank dedup
                }
            }
            uint64_t h = 0x2545f4914f6cdd1dull;
            uint64_t *mg = a.d.token_mask + (int64_t)t * a.W;
#pragma unroll
            for (int w = 0; w < WT; ++w)
                if (w < a.W) { mg[w] = m[w]; nd += __popcll(m[w]); h = mix64(h, m[w]); }
            a.d.token_ndest[t] = nd;
            if (a.src_rank >= 0 && nd == 1) {
#pragma unroll
                for (int w = 0; w < WT; ++w)
                    self_only |= (int)((m[w] & equal_mask64(a.src_rank >> 6, w)) >> (a.src_rank & 63)) & 1;
            }
            if (nd > 0) {
                if (WT == 1 && a.Kd < 64) {
                    slot = table_insert_word(a.d.slot_key, a.hs_mask, h, m[0]);
                } else {
                    __threadfence();                                  // bitmap visible before the slot is claimed
                    const int W = a.W;
                    const uint64_t *masks = a.d.token_mask;
                    slot = table_insert(a.d.slot_key, a.hs_mask, h, t, [&](int other) {
                        bool same = true;
#pragma unroll
                        for (int w = 0; w < WT; ++w)
                            if (w < W) same &= (__ldcg(masks + (int64_t)other * W + w) == m[w]);
                        return same;
                    });
                }
                if (slot < 0) { set_status(&acc->status, MW_ERR_CAPACITY); nd = 0; a.d.token_ndest[t] = 0; }
                else { atomicMin(a.d.slot_leader + slot, t); atomicAdd(a.d.slot_count + slot, 1); }
            }
        }
        valid = __reduce_add_sync(0xffffffffu, valid);
        self_only = __reduce_add_sync(0xffffffffu, self_only);
        bad = __reduce_or_sync(0xffffffffu, (unsigned)bad);
        if ((tid & 31) == 0) {
            if (valid) atomicAdd(&acc->valid_slots, (unsigned long long)valid);
            if (self_only) atomicAdd(&acc->self_only, (unsigned)self_only);
            if (bad) set_status(&acc->status, MW_ERR_BAD_INDEX);
        }
    }
    // Decoupled look-back over tiles for counters [c0, c1): one thread per counter, kLookBack predecessors
    // fetched per round trip.  A record is one 64-bit word (epoch, flag, value), so flag and value are
    // always read together; the epoch makes records of earlier plans invisible.
    auto look_back = [&](int c0, int c1) {
        for (int c = c0 + tid; c < c1; c += MW_TILE) {
            const uint32_t mine = (uint32_t)cnt[c];
            volatile unsigned long long *rec = a.d.tile_state + (size_t)tile * a.NC + c;
            uint32_t excl = 0;
            if (tile == 0) {
                *rec = pack_state(pc.epoch, kFlagPrefix, mine);
            } else {
                *rec = pack_state(pc.epoch, kFlagAgg, mine);
                bool done = false;
                for (int j = tile - 1; j >= 0 && !done; j -= kLookBack) {
                    unsigned long long s[kLookBack];
#pragma unroll
                    for (int i = 0; i < kLookBack; ++i)
                        s[i] = (j - i >= 0) ? *(volatile unsigned long long *)(a.d.tile_state + (size_t)(j - i) * a.NC + c) : 0ull;
#pragma unroll
                    for (int i = 0; i < kLookBack; ++i) {
                        if (done || j - i < 0) continue;
                        int spins = 0;
                        while (true) {
                            const uint32_t hi = (uint32_t)(s[i] >> 32);
                            if ((hi >> 2) == pc.wait_epoch && (hi & 3u) != 0) break;
                            if (++spins > a.spin_limit) { give_up(a, &acc->status); done = true; break; }
                            __nanosleep(64);
                            s[i] = *(volatile unsigned long long *)(a.d.tile_state + (size_t)(j - i) * a.NC + c);
                        }
                        if (done) break;
                        excl += (uint32_t)s[i];
                        if (((uint32_t)(s[i] >> 32) & 3u) == kFlagPrefix) done = true;
                    }
                }
                *rec = pack_state(pc.epoch, kFlagPrefix, excl + mine);
            }
            base[c] = (int)excl;
        }
    };

    // ---- phase B1 (needs only this tile's bitmaps, so it runs between the two halves of the first grid
    //      barrier and overlaps the barrier's latency): positions inside the tile, rank histogram, look-back ----
    const int wi = tid >> 5;
    const uint32_t bit = 1u << (tid & 31);
    grid_barrier_arrive(a.d.gbar);  // this tile's bitmaps are in the table (also orders the clearing of the bit matrix)
    if (nd > 0) {
#pragma unroll 1
        for (int w = 0; w < a.W; ++w)
            for (uint64_t word = bitmap_word(m, w); word; word &= word - 1)
                atomicOr(bits + (size_t)(w * 64 + __ffsll((long long)word) - 1) * 8 + wi, bit);
    }
    __syncthreads();
    for (int r = tid; r < a.R; r += MW_TILE) {
        int run = 0;
#pragma unroll
        for (int w8 = 0; w8 < 8; ++w8) { pre[r * 8 + w8] = run; run += __popc(bits[r * 8 + w8]); }
        cnt[r] = run;
    }
    __syncthreads();
    look_back(0, a.R);
    __syncthreads();
    bool alive = grid_barrier_wait(a, pc.bar_base + (unsigned)a.ntiles, true, &acc->status);

    // ---- phase B2: leaders and group sizes are final; every tile publishes its two totals ----
    int leader = -1, gcount = 0, lead_excl = 0, gc_excl = 0;
    int64_t SD_last = 0, self_copies = 0;          // thread 0 of the last tile
    if (alive) {
        if (nd > 0) { leader = __ldcg(a.d.slot_leader + slot); gcount = __ldcg(a.d.slot_count + slot); }
        const bool is_leader = nd > 0 && leader == t;
        if (active) a.d.token_leader[t] = leader;
        int lead_total, gc_total;
        lead_excl = block_excl_scan(is_leader ? 1 : 0, warp_sums, lead_total);
        gc_excl = block_excl_scan(is_leader ? gcount : 0, warp_sums, gc_total);
        // group id and offset relative to the tile, stored at the leader; the sums over earlier tiles are added
        // by whoever reads them, after the barrier (no second look-back chain)
        if (is_leader) { a.d.gid_at[t] = lead_excl; a.d.goff_at[t] = gc_excl; }
        if (tid == 0) a.d.tile_agg[tile] = ((unsigned long long)(uint32_t)gc_total << 32) | (uint32_t)lead_total;
        if (tile == a.ntiles - 1) {
            // this tile's inclusive prefix is the grand total of every rank counter
            int carry = 0;
            for (int r0 = 0; r0 < a.R; r0 += MW_TILE) {
                const int r = r0 + tid;
                const int v = r < a.R ? base[r] + cnt[r] : 0;
                int total;
                const int excl = block_excl_scan(v, warp_sums, total);
                if (r < a.R) a.d.rank_offsets[r] = carry + excl;
                carry += total;
            }
            if (tid == 0) {
                a.d.rank_offsets[a.R] = carry;
                SD_last = carry;
                self_copies = a.src_rank >= 0 ? base[a.src_rank] + cnt[a.src_rank] : 0;
            }
        }
    }
    // The (rank, slot) pairs of every token are only read by later kernels: they are stored while the second
    // barrier is in flight (arrive, store, wait), off the critical path.
    grid_barrier_arrive(a.d.gbar);
    if (alive && active) {
        int32_t *dr = a.d.dest_rank + (int64_t)t * a.Kd, *dp = a.d.dest_pos + (int64_t)t * a.Kd;
        if (a.Kd == 8) {
            // the usual top-8: the token's eight (rank, slot) pairs leave as four 16-byte stores instead of sixteen
            int rr[8], pp[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) { rr[i] = -1; pp[i] = -1; }
            if (nd > 0) {
                int i = 0;
#pragma unroll 1
                for (int w = 0; w < a.W; ++w)
                    for (uint64_t word = bitmap_word(m, w); word; word &= word - 1) {
                        const int r = w * 64 + __ffsll((long long)word) - 1;
                        const int p = base[r] + (int)pre[r * 8 + wi] + __popc(bits[r * 8 + wi] & (bit - 1));
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            if (j == i) { rr[j] = r; pp[j] = p; }
                        ++i;
                    }
            }
            ((int4 *)dr)[0] = make_int4(rr[0], rr[1], rr[2], rr[3]);
            ((int4 *)dr)[1] = make_int4(rr[4], rr[5], rr[6], rr[7]);
            ((int4 *)dp)[0] = make_int4(pp[0], pp[1], pp[2], pp[3]);
            ((int4 *)dp)[1] = make_int4(pp[4], pp[5], pp[6], pp[7]);
        } else {
            int i = 0;
            if (nd > 0) {
#pragma unroll 1
                for (int w = 0; w < a.W; ++w)
                    for (uint64_t word = bitmap_word(m, w); word; word &= word - 1) {
                        const int r = w * 64 + __ffsll((long long)word) - 1;
                        dr[i] = r;
                        dp[i] = base[r] + (int)pre[r * 8 + wi] + __popc(bits[r * 8 + wi] & (bit - 1));
                        ++i;
                    }
            }
            for (; i < a.Kd; ++i) { dr[i] = -1; dp[i] = -1; }
        }
    }
    alive = grid_barrier_wait(a, pc.bar_base + 2u * (unsigned)a.ntiles, alive, &acc->status);
    if (!alive) {
        if (tid == 0) set_status(&a.d.totals->status, MW_ERR_TIMEOUT);
        return;
    }

    // ---- phase C: group ids, send rows, inverse maps, delivery descriptors, table clean-up ----
    // Every block reads all tiles' totals (one record each, one round trip) and scans them in shared memory.
    __shared__ int tile_lead_pre[MW_TILE], tile_gc_pre[MW_TILE];
    int G, Tn;
    {
        const unsigned long long ag = tid < a.ntiles ? __ldcg(a.d.tile_agg + tid) : 0ull;
        const int plan_status = __ldcg(&acc->status);
        for (int r = tid; r <= a.R; r += MW_TILE) cnt[r] = __ldcg(a.d.rank_offsets + r);      // see below
        tile_lead_pre[tid] = block_excl_scan((int)(uint32_t)ag, warp_sums, G);
        tile_gc_pre[tid] = block_excl_scan((int)(uint32_t)(ag >> 32), warp_sums, Tn);
        if (tile == a.ntiles - 1 && tid == 0) {
            const int64_t sent_rows = (int64_t)Tn - (int64_t)acc->self_only;
            a.d.group_offsets[G] = Tn;
            mw_totals tt;
            tt.T_nonempty = Tn; tt.G = G; tt.total_dest = SD_last;
            tt.mw_bytes = sent_rows * a.row_bytes;
            tt.unicast_bytes = (SD_last - self_copies) * a.row_bytes;
            tt.unicast_per_expert_bytes = (int64_t)acc->valid_slots * a.row_bytes;
            // Section 6.4: beyond 64 ranks the bitmap travels in the payload, once per 4096-byte packet
            tt.meta_bytes = a.R <= 64 ? 0 : sent_rows * ((a.row_bytes + 4095) / 4096) * (int64_t)(8 * a.W);
            tt.status = plan_status;
            tt.reserved = 0;
            *a.d.totals = tt;
            mw_acc *next = a.d.acc + ((pc.epoch + 1u) & 1u);
            next->valid_slots = 0; next->self_only = 0; next->status = 0;
            advance_counters(a, 0u, 2u * (uint32_t)a.ntiles);   // every block is past the second barrier: all have read them
        }
        if (tile == a.ntiles - 1) wipe_records_at_lap_end(a, pc.epoch);      // all look-backs ended before the first barrier
        if (plan_status == MW_ERR_TIMEOUT) return;      // a look-back gave up somewhere: nothing below can be trusted
    }
    // cnt[] now holds the region starts (the tile's own counts are no longer needed); the barriers of the scans
    // above order those stores before their use below
    const int SD = cnt[a.R];
    // tails: every index up to T (inclusive for group_offsets) is covered by some thread of the grid
    for (int u = t; u <= a.T; u += a.ntiles * MW_TILE) {
        if (u > G) a.d.group_offsets[u] = -1;
        if (u < a.T) {
            if (u >= Tn) a.d.mw_row_token[u] = -1;
            for (int i = 0; i < a.Kd; ++i)
                if ((int64_t)u * a.Kd + i >= SD) a.d.rank_tokens[(int64_t)u * a.Kd + i] = -1;
            if (u >= G)
                for (int w = 0; w < a.W; ++w) a.d.group_mask[(int64_t)u * a.W + w] = 0;
        }
    }
    const int within = group_rank_in_tile(&rank_scratch, a.d.token_leader, tile, nd > 0 ? leader : -1, gcount);
    if (!active) return;
    if (nd == 0) { a.d.token_group[t] = -1; a.d.token_mw_row[t] = -1; return; }
    // the leader's values are relative to its tile; a leader has its own in registers
    const int lt = leader / MW_TILE;
    const int g = tile_lead_pre[lt] + (leader == t ? lead_excl : __ldcg(a.d.gid_at + leader));
    const int goff = tile_gc_pre[lt] + (leader == t ? gc_excl : __ldcg(a.d.goff_at + leader));
    const int row = goff + within;
    a.d.token_group[t] = g;
    a.d.token_mw_row[t] = row;
    a.d.mw_row_token[row] = t;
    a.d.row_ndest[row] = nd;
    if (leader == t) {
        a.d.group_offsets[g] = goff;
#pragma unroll
        for (int w = 0; w < WT; ++w)
            if (w < a.W) a.d.group_mask[(int64_t)g * a.W + w] = m[w];
    }
    {
        int i = 0;
#pragma unroll 1
        for (int w = 0; w < a.W; ++w)
            for (uint64_t word = bitmap_word(m, w); word; word &= word - 1) {
                const int r = w * 64 + __ffsll((long long)word) - 1;
                const int p = base[r] + (int)pre[r * 8 + wi] + __popc(bits[r * 8 + wi] & (bit - 1));
                a.d.row_dest_rank[(int64_t)i * a.Tm + row] = r;
                a.d.row_dest_pos[(int64_t)i * a.Tm + row] = p;
                const int at = cnt[r] + p;
                a.d.row_dest_flat[(int64_t)i * a.Tm + row] = at;
                a.d.rank_tokens[at] = t;
                ++i;
            }
        for (; i < a.Kd; ++i) {
            a.d.row_dest_rank[(int64_t)i * a.Tm + row] = -1;
            a.d.row_dest_pos[(int64_t)i * a.Tm + row] = -1;
            a.d.row_dest_flat[(int64_t)i * a.Tm + row] = -1;
        }
    }
    a.d.slot_key[slot] = kEmptyKey;
    a.d.slot_leader[slot] = kNoLeader;
    a.d.slot_count[slot] = 0;
}

size_t tile_smem_bytes(const mw_ctx *ctx) { return ((size_t)ctx->cfg.R * 16 + 2 * (size_t)ctx->NC) * sizeof(uint32_t); }

}  // namespace

int mw_plan_smem_setup(mw_ctx *ctx)
{
    const size_t need = tile_smem_bytes(ctx);
    if (need > (size_t)ctx->max_smem_optin) return MW_ERR_INVALID_ARG;
    if (need > 48 * 1024) {
        const int n = (int)need;
        if (cudaFuncSetAttribute(k_plan_tile, cudaFuncAttributeMaxDynamicSharedMemorySize, n) != cudaSuccess ||
            cudaFuncSetAttribute(k_plan_fused<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, n) != cudaSuccess ||
            cudaFuncSetAttribute(k_plan_fused<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, n) != cudaSuccess ||
            cudaFuncSetAttribute(k_plan_fused<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, n) != cudaSuccess ||
            cudaFuncSetAttribute(k_plan_fused<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, n) != cudaSuccess)
            return MW_ERR_CUDA;
    }
    return MW_OK;
}

int mw_plan_launch(mw_ctx *ctx, const int32_t *topk_ids, const int32_t *expert_to_rank, int32_t T, const void *rows, cudaStream_t st)
{
    PlanArgs a;
    a.ids = topk_ids; a.e2r = expert_to_rank;
    a.T = T; a.K = ctx->cfg.K; a.E = ctx->cfg.E; a.R = ctx->cfg.R; a.W = ctx->W; a.Kd = ctx->Kd;
    a.src_rank = ctx->cfg.src_rank;
    a.relay_src = ctx->relay_src; a.relay_P = ctx->relay_P;
    a.ntiles = T > 0 ? (T + MW_TILE - 1) / MW_TILE : 1;
    a.NC = ctx->NC; a.hs_mask = ctx->HS - 1; a.Tm = ctx->cfg.max_tokens;
    a.row_bytes = ctx->cfg.row_bytes;
    ctx->epoch += 1;                     // identifies the plan on the host (which plan a slot holds); the kernels count for themselves
    a.d = ctx->d;
    a.spin_limit = ctx->spin_limit;
    a.bar_spin_limit = ctx->bar_spin_limit;
    a.skew_epoch = (ctx->test_skew & MW_TEST_SKEW_LOOKBACK) ? 1u : 0u;       // records nobody writes
    a.skew_bar = (ctx->test_skew & MW_TEST_SKEW_BARRIER) ? 1u : 0u;          // a count nobody reaches
    ctx->test_skew &= ~(uint32_t)(MW_TEST_SKEW_LOOKBACK | MW_TEST_SKEW_BARRIER);
    const int blocks = a.ntiles;
    ctx->planned_T = T;
    ctx->plan_epoch = ctx->epoch;
    // rows to bring into L2 meanwhile: the first half-L2 of them (the pack step reads them in ascending order)
    a.pf_base = (const uint8_t *)rows;
    ctx->prefetched = nullptr;
    a.pf_bytes = rows ? (int64_t)T * ctx->cfg.row_bytes : 0;
    if (a.pf_bytes > ctx->l2_bytes / 2) a.pf_bytes = (ctx->l2_bytes / 2) & ~(int64_t)15;
    if (blocks <= ctx->sm_count && blocks <= MW_TILE && !(ctx->cfg.flags & MW_FLAG_PLAN_MULTIPASS)) {
        // One launch, at most one block per SM, phases separated by grid barriers.  The blocks wait for
        // one another, so all of them must become resident: an ordinary launch achieves that as soon
        // as earlier kernels of the stream have drained (the grid never exceeds the SM count and needs
        // a fraction of an SM each); blocks of other streams that occupy an SM are short-lived copy blocks.
        // Should other work keep SMs occupied for about a second, the barrier gives up with
        // MW_ERR_TIMEOUT instead of hanging (mw_reset then makes the context usable again;
        // MW_FLAG_PLAN_MULTIPASS avoids the residency assumption altogether).
        // The plan is not launched as a programmatic dependent of the previous kernel: measured on
        // B200 that costs about 30 us per step, while the pack kernel that follows does overlap its
        // start-up with the plan.
        void (*fn)(PlanArgs) = ctx->W <= 1 ? k_plan_fused<1> : ctx->W <= 2 ? k_plan_fused<2>
                             : ctx->W <= 4 ? k_plan_fused<4> : k_plan_fused<16>;
        // with rows to prefetch, one more block for every SM the tiles leave free
        const int extra = a.pf_bytes > 0 ? ctx->sm_count - blocks : 0;
        if (extra > 0 && a.pf_bytes == (int64_t)T * ctx->cfg.row_bytes) ctx->prefetched = rows;     // all of them fit
        const cudaError_t e = mw_launch(fn, dim3(blocks + extra), dim3(MW_TILE), tile_smem_bytes(ctx), st, false, a);
        if (e == cudaSuccess) {
            ctx->launches += 1;
            return MW_OK;
        }
        cudaGetLastError();   // the launch was refused: take the multi-pass route
        ctx->prefetched = nullptr;
    }
    k_plan_mask<<<blocks, MW_TILE, 0, st>>>(a);
    k_plan_tile<<<blocks, MW_TILE, tile_smem_bytes(ctx), st>>>(a);
    // one extra thread beyond T so that group_offsets[T] is covered
    k_plan_final<<<(T + 1 + MW_TILE - 1) / MW_TILE, MW_TILE, 0, st>>>(a);
    ctx->launches += 3;
    return cudaGetLastError() == cudaSuccess ? MW_OK : MW_ERR_CUDA;
}
