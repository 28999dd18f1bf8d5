/*
 * mwo -- CPU oracle for the MultiWrite dispatch / AllGather pack-and-deliver path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, sequential statement of
 * what the path computes.  It shares no code with the CUDA library and is never
 * used by it; only the tests, the smoke check and the benchmark's CPU-baseline leg
 * may call it.
 *
 * What is being computed (paper, Section 4.3.1): MultiWrite(S, M, B_S) writes the
 * content of the source buffer B_S into the target buffer B_i of every destination
 * D_i in M.  For MoE dispatch (Sections 1 and 2.3.2) the destinations of a token
 * are the nodes that host its gate-selected top-k experts; the destination set is
 * carried as a bitmap with one bit per rank, ranks numbered from zero
 * (Section 4.1, "Encoding scheme of metadata"; Section 6.4 for more than 64 ranks).
 * The unicast comparison sends one copy per destination (Section 2.2).  The
 * AllGather form (Section 5.2) delivers every rank's shard to every rank.
 *
 * The paper fixes the *content* each destination must end up with; it leaves the
 * slot layout open.  The layout used here (also listed in the design notes):
 *   - bit (r mod 64) of 64-bit word (r / 64) stands for rank r, least significant
 *     bit first; bits at or above R are zero;
 *   - the destination set is per rank: several experts of one token on the same
 *     rank set one bit;
 *   - a group is the set of all tokens with a bit-identical, non-empty bitmap;
 *     groups are numbered by first occurrence while walking tokens 0..T-1;
 *   - inside a group, and inside every receive region, rows keep ascending token
 *     order;
 *   - an expert id of -1 is padding; any other id outside [0,E), or a table entry
 *     outside [0,R), is ignored and reported as MWO_ERR_BAD_INDEX;
 *   - a token whose bitmap is empty gets no group, no send row and no bytes;
 *   - src_rank >= 0 names the sender's own rank: its bit is still delivered, but
 *     that copy is local and is left out of both transmitted-byte counts.
 *
 * Parity pins for every function live in tests/test_oracle_*.py (brute-force
 * enumeration of (token, rank) pairs written independently in Python, closed
 * forms, library counting-sort / bincount / concatenate special cases, the
 * constants printed in the paper).  The numbering rules themselves (first
 * occurrence, ascending token order) are this implementation's reading, not the
 * paper's: parity for those choices is pinned only to the independent brute force.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define MWO_OK 0
#define MWO_ERR_INVALID_ARG (-1)
#define MWO_ERR_BAD_INDEX (-5)

typedef struct {
    int64_t T_nonempty;               /* T' : tokens with a non-empty destination set        */
    int64_t G;                        /* number of distinct non-empty destination sets       */
    int64_t total_dest;               /* sum over tokens of |D_t| (rows delivered)           */
    int64_t mw_bytes;                 /* bytes transmitted when each row is sent once        */
    int64_t unicast_bytes;            /* bytes transmitted with one copy per destination     */
    int64_t unicast_per_expert_bytes; /* bytes if one copy were sent per valid expert slot   */
    int64_t meta_bytes;               /* in-payload bitmap bytes when R > 64 (Section 6.4)   */
    int32_t status;
    int32_t reserved;
} mwo_totals;

static int mwo_words(int32_t R) { return (R + 63) / 64; }

static int popcount64(uint64_t v)
{
    int c = 0;
    while (v) { v &= v - 1; ++c; }
    return c;
}

/*
 * Plan: bitmaps, groups, offsets, slots, byte accounting.
 *
 * Output arrays (caller allocated, Kd = min(K, R), W = ceil(R / 64)):
 *   token_mask   [T, W]   token_ndest [T]   token_group [T]   token_mw_row [T]
 *   mw_row_token [T]      (first T' entries defined, rest -1)
 *   group_offsets[T + 1]  (first G + 1 entries defined, rest -1)
 *   group_mask   [T, W]   (first G rows defined, rest 0)
 *   rank_offsets [R + 1]  rank_tokens [T * Kd] (first total_dest defined, rest -1)
 *   dest_rank    [T, Kd]  dest_pos    [T, Kd]  (-1 padded)
 */
int mwo_plan(const int32_t *topk_ids, const int32_t *expert_to_rank,
             int32_t T, int32_t K, int32_t E, int32_t R, int64_t row_bytes, int32_t src_rank,
             uint64_t *token_mask, int32_t *token_ndest, int32_t *token_group,
             int32_t *token_mw_row, int32_t *mw_row_token, int32_t *group_offsets,
             uint64_t *group_mask, int32_t *rank_offsets, int32_t *rank_tokens,
             int32_t *dest_rank, int32_t *dest_pos, mwo_totals *totals)
{
    if (T < 0 || K <= 0 || E <= 0 || R <= 0 || row_bytes <= 0 || src_rank >= R) return MWO_ERR_INVALID_ARG;
    const int W = mwo_words(R);
    const int Kd = K < R ? K : R;
    int32_t status = MWO_OK;
    int64_t valid_slots = 0;

    /* Step 1 -- destination bitmap per token (Section 4.1: one bit per rank, 1 = target). */
    for (int32_t t = 0; t < T; ++t) {
        uint64_t *m = token_mask + (int64_t)t * W;
        for (int w = 0; w < W; ++w) m[w] = 0;
        for (int32_t k = 0; k < K; ++k) {
            int32_t id = topk_ids[(int64_t)t * K + k];
            if (id == -1) continue;                         /* padding slot            */
            if (id < 0 || id >= E) { status = MWO_ERR_BAD_INDEX; continue; }
            int32_t r = expert_to_rank[id];
            if (r < 0 || r >= R) { status = MWO_ERR_BAD_INDEX; continue; }
            ++valid_slots;
            m[r / 64] |= (uint64_t)1 << (r % 64);            /* OR: per-rank dedup      */
        }
        int nd = 0;
        for (int w = 0; w < W; ++w) nd += popcount64(m[w]);
        token_ndest[t] = nd;
    }

    /* Step 2 -- groups of identical bitmap, numbered by first occurrence. */
    int64_t G = 0, Tn = 0;
    int32_t *group_count = (int32_t *)calloc((size_t)T + 1, sizeof(int32_t));
    if (!group_count) return MWO_ERR_INVALID_ARG;
    for (int64_t i = 0; i < (int64_t)T * W; ++i) group_mask[i] = 0;
    for (int32_t t = 0; t < T; ++t) {
        const uint64_t *m = token_mask + (int64_t)t * W;
        if (token_ndest[t] == 0) { token_group[t] = -1; continue; }
        int64_t g = 0;
        for (; g < G; ++g)
            if (memcmp(group_mask + g * W, m, (size_t)W * sizeof(uint64_t)) == 0) break;
        if (g == G) { memcpy(group_mask + G * W, m, (size_t)W * sizeof(uint64_t)); ++G; }
        token_group[t] = (int32_t)g;
        ++group_count[g];
        ++Tn;
    }

    /* Step 3 -- group offsets (exclusive prefix sum) and send rows in token order. */
    for (int32_t i = 0; i <= T; ++i) group_offsets[i] = -1;
    group_offsets[0] = 0;
    for (int64_t g = 0; g < G; ++g) group_offsets[g + 1] = group_offsets[g] + group_count[g];
    for (int32_t t = 0; t < T; ++t) mw_row_token[t] = -1;
    for (int64_t g = 0; g < G; ++g) group_count[g] = 0;       /* reuse as "members seen so far" */
    for (int32_t t = 0; t < T; ++t) {
        int32_t g = token_group[t];
        if (g < 0) { token_mw_row[t] = -1; continue; }
        int32_t row = group_offsets[g] + group_count[g]++;
        token_mw_row[t] = row;
        mw_row_token[row] = t;
    }
    free(group_count);

    /* Step 4 -- per-rank counts, offsets, and each token's slot in each receive region. */
    int32_t *rank_seen = (int32_t *)calloc((size_t)R, sizeof(int32_t));
    if (!rank_seen) return MWO_ERR_INVALID_ARG;
    for (int32_t t = 0; t < T; ++t)
        for (int32_t r = 0; r < R; ++r)
            if (token_mask[(int64_t)t * W + r / 64] >> (r % 64) & 1) ++rank_seen[r];
    rank_offsets[0] = 0;
    for (int32_t r = 0; r < R; ++r) rank_offsets[r + 1] = rank_offsets[r] + rank_seen[r];
    const int64_t total_dest = rank_offsets[R];
    for (int64_t i = 0; i < (int64_t)T * Kd; ++i) { rank_tokens[i] = -1; dest_rank[i] = -1; dest_pos[i] = -1; }
    for (int32_t r = 0; r < R; ++r) rank_seen[r] = 0;          /* reuse as "tokens seen so far" */
    for (int32_t t = 0; t < T; ++t) {
        int i = 0;
        for (int32_t r = 0; r < R; ++r) {
            if (!(token_mask[(int64_t)t * W + r / 64] >> (r % 64) & 1)) continue;
            dest_rank[(int64_t)t * Kd + i] = r;
            dest_pos[(int64_t)t * Kd + i] = rank_seen[r];
            rank_tokens[rank_offsets[r] + rank_seen[r]] = t;
            ++rank_seen[r];
            ++i;
        }
    }
    free(rank_seen);

    /* Step 5 -- transmitted bytes, exactly, from the plan. */
    int64_t sent_rows = 0, sent_copies = 0;
    for (int32_t t = 0; t < T; ++t) {
        int nd = token_ndest[t];
        if (src_rank >= 0 && (token_mask[(int64_t)t * W + src_rank / 64] >> (src_rank % 64) & 1)) --nd;
        if (nd > 0) ++sent_rows;
        sent_copies += nd;
    }
    totals->T_nonempty = Tn;
    totals->G = G;
    totals->total_dest = total_dest;
    totals->mw_bytes = sent_rows * row_bytes;
    totals->unicast_bytes = sent_copies * row_bytes;
    totals->unicast_per_expert_bytes = valid_slots * row_bytes;
    /* Section 6.4: above 64 ranks the bitmap rides in the payload, once per 4096-byte packet. */
    totals->meta_bytes = R <= 64 ? 0 : sent_rows * ((row_bytes + 4095) / 4096) * (int64_t)(8 * W);
    totals->status = status;
    totals->reserved = 0;
    return MWO_OK;
}

/* Region r of a receive area: explicit stride, or compact (stride 0: region r begins at row rank_offsets[r]). */
static uint8_t *region(uint8_t *recv_base, int64_t stride, const int32_t *rank_offsets, int32_t r, int64_t row_bytes)
{
    return stride ? recv_base + (int64_t)r * stride : recv_base + (int64_t)rank_offsets[r] * row_bytes;
}

/* MultiWrite send layout: row j holds the hidden row of token mw_row_token[j], each token once. */
void mwo_pack_mw(const uint8_t *x, int64_t row_bytes, const int32_t *mw_row_token, int64_t T_nonempty, uint8_t *send_mw)
{
    for (int64_t j = 0; j < T_nonempty; ++j)
        memcpy(send_mw + j * row_bytes, x + (int64_t)mw_row_token[j] * row_bytes, (size_t)row_bytes);
}

/* Unicast send layout: one copy per destination, rank-major, token order inside a rank. */
void mwo_pack_uc(const uint8_t *x, int64_t row_bytes, const int32_t *rank_tokens, int64_t total_dest, uint8_t *send_uc)
{
    for (int64_t i = 0; i < total_dest; ++i)
        memcpy(send_uc + i * row_bytes, x + (int64_t)rank_tokens[i] * row_bytes, (size_t)row_bytes);
}

/*
 * Deliver from the MultiWrite send buffer: every send row is written to every
 * destination named by its group's bitmap (Section 4.3.1; Section 4.3.3 with each
 * destination as its own next hop: one plain write per set bit).
 */
void mwo_deliver_mw(const uint8_t *send_mw, int64_t row_bytes, int64_t T_nonempty, int32_t R, int32_t K,
                    const int32_t *mw_row_token, const int32_t *token_group, const uint64_t *group_mask,
                    const int32_t *dest_pos, const int32_t *rank_offsets,
                    uint8_t *recv_base, int64_t recv_stride_bytes)
{
    const int W = mwo_words(R);
    const int Kd = K < R ? K : R;
    for (int64_t j = 0; j < T_nonempty; ++j) {
        int32_t t = mw_row_token[j];
        const uint64_t *m = group_mask + (int64_t)token_group[t] * W;
        int i = 0;
        for (int32_t r = 0; r < R; ++r) {
            if (!(m[r / 64] >> (r % 64) & 1)) continue;
            int64_t slot = dest_pos[(int64_t)t * Kd + i++];
            memcpy(region(recv_base, recv_stride_bytes, rank_offsets, r, row_bytes) + slot * row_bytes,
                   send_mw + j * row_bytes, (size_t)row_bytes);
        }
    }
}

/* Deliver from the unicast send buffer: region r receives its contiguous slice. */
void mwo_deliver_uc(const uint8_t *send_uc, int64_t row_bytes, int32_t R, const int32_t *rank_offsets,
                    uint8_t *recv_base, int64_t recv_stride_bytes)
{
    for (int32_t r = 0; r < R; ++r) {
        int64_t n = rank_offsets[r + 1] - rank_offsets[r];
        memcpy(region(recv_base, recv_stride_bytes, rank_offsets, r, row_bytes),
               send_uc + (int64_t)rank_offsets[r] * row_bytes, (size_t)(n * row_bytes));
    }
}

/*
 * Delivery straight from the definition, using only the router output and the
 * table: for each rank, walk tokens in ascending order and append the hidden row
 * of every token that selected an expert on that rank.
 */
void mwo_deliver_definition(const uint8_t *x, int64_t row_bytes, const int32_t *topk_ids, const int32_t *expert_to_rank,
                            int32_t T, int32_t K, int32_t E, int32_t R, const int32_t *rank_offsets,
                            uint8_t *recv_base, int64_t recv_stride_bytes)
{
    for (int32_t r = 0; r < R; ++r) {
        uint8_t *dst = region(recv_base, recv_stride_bytes, rank_offsets, r, row_bytes);
        int64_t n = 0;
        for (int32_t t = 0; t < T; ++t) {
            int hit = 0;
            for (int32_t k = 0; k < K && !hit; ++k) {
                int32_t id = topk_ids[(int64_t)t * K + k];
                if (id >= 0 && id < E && expert_to_rank[id] == r) hit = 1;
            }
            if (hit) memcpy(dst + (n++) * row_bytes, x + (int64_t)t * row_bytes, (size_t)row_bytes);
        }
    }
}

/*
 * AllGather (Section 5.2): R ranks each hold one shard of shard_bytes; afterwards
 * every destination rank holds shard_0 | shard_1 | ... | shard_{R-1}.
 *
 * Only destination ranks [dst_begin, dst_begin + dst_count) are materialised (the
 * full R x R result does not fit in memory for large shards); byte accounting is
 * always for the full domain.  A rank's own shard reaches its own region by a
 * local copy, never over the network (Section 2.3.1: N1 sends its partition seven
 * times in an 8-node domain), so it is delivered but not counted.
 *
 * layout 0 (MultiWrite): send_buf [R, shard_bytes] holds every shard once.
 * layout 1 (unicast):    send_buf [R, dst_count, shard_bytes]; slot (i, d) holds the
 *                        copy of shard i addressed to rank dst_begin + d.  The slot
 *                        with dst_begin + d == i is never transmitted; it is left
 *                        untouched and the self copy is taken from the shard itself.
 * Region d of recv (rank dst_begin + d) starts at recv_base + d * stride
 * (stride 0: compact, d * R * shard_bytes).
 */
int mwo_allgather(const uint8_t *shards, int32_t R, int64_t shard_bytes, int layout,
                  int32_t dst_begin, int32_t dst_count, uint8_t *send_buf,
                  uint8_t *recv_base, int64_t recv_stride_bytes, mwo_totals *totals)
{
    if (R <= 0 || shard_bytes <= 0 || dst_begin < 0 || dst_count < 0 || dst_begin + dst_count > R) return MWO_ERR_INVALID_ARG;
    if (layout != 0 && layout != 1) return MWO_ERR_INVALID_ARG;
    const int64_t stride = recv_stride_bytes ? recv_stride_bytes : (int64_t)R * shard_bytes;
    if (layout == 0) {
        for (int32_t i = 0; i < R; ++i)
            memcpy(send_buf + (int64_t)i * shard_bytes, shards + (int64_t)i * shard_bytes, (size_t)shard_bytes);
        for (int32_t i = 0; i < R; ++i)
            for (int32_t d = 0; d < dst_count; ++d)
                memcpy(recv_base + d * stride + (int64_t)i * shard_bytes,
                       send_buf + (int64_t)i * shard_bytes, (size_t)shard_bytes);
    } else {
        for (int32_t i = 0; i < R; ++i)
            for (int32_t d = 0; d < dst_count; ++d) {
                if (dst_begin + d == i) continue;
                memcpy(send_buf + ((int64_t)i * dst_count + d) * shard_bytes,
                       shards + (int64_t)i * shard_bytes, (size_t)shard_bytes);
            }
        for (int32_t i = 0; i < R; ++i)
            for (int32_t d = 0; d < dst_count; ++d) {
                const uint8_t *src = (dst_begin + d == i) ? shards + (int64_t)i * shard_bytes
                                                           : send_buf + ((int64_t)i * dst_count + d) * shard_bytes;
                memcpy(recv_base + d * stride + (int64_t)i * shard_bytes, src, (size_t)shard_bytes);
            }
    }
    if (totals) {
        const int W = mwo_words(R);
        memset(totals, 0, sizeof(*totals));
        totals->T_nonempty = R;
        totals->G = R;                                   /* every shard has its own destination set (all but itself) */
        totals->total_dest = (int64_t)R * R;             /* rows delivered, self copies included */
        totals->mw_bytes = R > 1 ? (int64_t)R * shard_bytes : 0;
        totals->unicast_bytes = (int64_t)R * (R - 1) * shard_bytes;
        totals->unicast_per_expert_bytes = totals->unicast_bytes;
        totals->meta_bytes = (R <= 64 || R == 1) ? 0 : (int64_t)R * ((shard_bytes + 4095) / 4096) * (8 * W);
        totals->status = MWO_OK;
    }
    return MWO_OK;
}

/*
 * Two-level (relayed) MultiWrite for dispatch: Section 3.2 and Section 4.3.3.
 *
 * Ranks are grouped into servers of ranks_per_server consecutive ranks.  The source (src_rank, a
 * member of the domain) writes directly to destinations inside its own server; for every other
 * server that holds at least one destination of a token it sends ONE copy to the rank with its own
 * index inside that server (Section 3.2), which then replicates the row to the destinations
 * inside its server (Section 3.2; Section 4.1 "Local forwarding table": one copy per distinct next hop;
 * Section 4.3.3: M is partitioned by next hop).
 */
int mwo_next_hop(int32_t r, int32_t src_rank, int32_t ranks_per_server)
{
    if (r / ranks_per_server == src_rank / ranks_per_server) return r;          /* same server: direct   */
    return (r / ranks_per_server) * ranks_per_server + src_rank % ranks_per_server;   /* same-index relay */
}

typedef struct {
    int64_t hop_rows;               /* rows written by the source: one per (token, distinct next hop)       */
    int64_t delivered_rows;         /* rows in the final receive regions (= flat total_dest)                */
    int64_t direct_bytes;           /* source -> destinations in its own server (own rank excluded)         */
    int64_t inter_multiwrite_bytes; /* source -> other servers, one copy per server that has a destination  */
    int64_t inter_unicast_bytes;    /* source -> other servers, one copy per remote destination (baseline)  */
    int64_t forward_bytes;          /* relays -> destinations in their server (the relay itself excluded)   */
    int64_t staged_rows;            /* hop rows whose next hop is not itself a destination of the token     */
    int32_t status;
    int32_t reserved;
} mwo_relay_totals;

/*
 * hop_of_expert [E]: next hop of every expert's rank (the table handed to the first-level plan);
 * entries whose rank is out of range are passed through unchanged so that the plan reports them.
 */
void mwo_relay_table(const int32_t *expert_to_rank, int32_t E, int32_t R, int32_t src_rank, int32_t ranks_per_server,
                     int32_t *hop_of_expert)
{
    for (int32_t e = 0; e < E; ++e) {
        int32_t r = expert_to_rank[e];
        hop_of_expert[e] = (r < 0 || r >= R) ? r : mwo_next_hop(r, src_rank, ranks_per_server);
    }
}

/*
 * Second level: every row that arrived in hop region h (rows of the first-level plan, token order) is
 * written to each final destination r of its token whose next hop is h, at the slot the flat plan gives
 * that (token, rank) pair.  Also the byte accounting per link class.
 *   hop_*   : first-level plan (computed by mwo_plan on hop_of_expert)
 *   flat_*  : flat plan (computed by mwo_plan on expert_to_rank)
 *   hop_buf : compact first-level receive area [hop_rows, row_bytes]
 */
void mwo_relay_expand(const uint8_t *hop_buf, int64_t row_bytes, int32_t T, int32_t R, int32_t K,
                      int32_t src_rank, int32_t ranks_per_server,
                      const int32_t *hop_rank_offsets, const int32_t *hop_rank_tokens,
                      const int32_t *flat_dest_rank, const int32_t *flat_dest_pos, const int32_t *flat_rank_offsets,
                      int32_t flat_status, uint8_t *recv_base, int64_t recv_stride_bytes, mwo_relay_totals *totals)
{
    const int Kd = K < R ? K : R;
    memset(totals, 0, sizeof(*totals));
    for (int32_t h = 0; h < R; ++h) {
        for (int32_t q = hop_rank_offsets[h]; q < hop_rank_offsets[h + 1]; ++q) {
            const int32_t t = hop_rank_tokens[q];
            const int remote = h / ranks_per_server != src_rank / ranks_per_server;
            int is_dest = 0;
            ++totals->hop_rows;
            if (remote) totals->inter_multiwrite_bytes += row_bytes;
            for (int i = 0; i < Kd; ++i) {
                const int32_t r = flat_dest_rank[(int64_t)t * Kd + i];
                if (r < 0 || mwo_next_hop(r, src_rank, ranks_per_server) != h) continue;
                if (recv_base)
                    memcpy(region(recv_base, recv_stride_bytes, flat_rank_offsets, r, row_bytes) +
                               (int64_t)flat_dest_pos[(int64_t)t * Kd + i] * row_bytes,
                           hop_buf + (int64_t)q * row_bytes, (size_t)row_bytes);
                ++totals->delivered_rows;
                if (r == h) is_dest = 1;
                if (remote) {
                    totals->inter_unicast_bytes += row_bytes;
                    if (r != h) totals->forward_bytes += row_bytes;
                } else if (r != src_rank) {
                    totals->direct_bytes += row_bytes;
                }
            }
            if (!is_dest) ++totals->staged_rows;
        }
    }
    totals->status = flat_status;
    (void)T;
}

/*
 * The same two levels with the receive buffer serving as the relay buffer (Section 6.4, memory usage: the relay's
 * buffer is the receive buffer that exists anyway, so relaying needs no memory of its own).  A copy whose next hop h
 * is itself a destination of the token is written by the first level straight into its final slot of region(h); the
 * relay then forwards it from there.  Only a copy whose next hop is NOT a destination of the token (a pure relay)
 * needs a place outside the receive regions: it goes to its row of the hop area, laid out as before (region of hop h
 * at the first-level offset of h), whose other rows are left untouched.
 *
 * First level: send row j of the first-level plan (token t) to every next hop h of the token.
 */
static int flat_slot_of(const int32_t *flat_dest_rank, const int32_t *flat_dest_pos, int32_t t, int Kd, int32_t r)
{
    for (int i = 0; i < Kd; ++i)
        if (flat_dest_rank[(int64_t)t * Kd + i] == r) return flat_dest_pos[(int64_t)t * Kd + i];
    return -1;                                           /* r is not a destination of t */
}

void mwo_relay_first_in_place(const uint8_t *send_mw, int64_t row_bytes, int64_t hop_T_nonempty, int32_t R, int32_t K,
                              const int32_t *hop_mw_row_token, const int32_t *hop_dest_rank, const int32_t *hop_dest_pos,
                              const int32_t *hop_rank_offsets,
                              const int32_t *flat_dest_rank, const int32_t *flat_dest_pos, const int32_t *flat_rank_offsets,
                              uint8_t *hop_buf, uint8_t *recv_base, int64_t recv_stride_bytes)
{
    const int Kd = K < R ? K : R;
    for (int64_t j = 0; j < hop_T_nonempty; ++j) {
        const int32_t t = hop_mw_row_token[j];
        for (int i = 0; i < Kd; ++i) {
            const int32_t h = hop_dest_rank[(int64_t)t * Kd + i];
            if (h < 0) break;
            const int slot = flat_slot_of(flat_dest_rank, flat_dest_pos, t, Kd, h);
            uint8_t *dst = slot >= 0
                ? region(recv_base, recv_stride_bytes, flat_rank_offsets, h, row_bytes) + (int64_t)slot * row_bytes
                : hop_buf + ((int64_t)hop_rank_offsets[h] + hop_dest_pos[(int64_t)t * Kd + i]) * row_bytes;
            memcpy(dst, send_mw + j * row_bytes, (size_t)row_bytes);
        }
    }
}

/* Second level: every relay forwards the copy it holds (in its own region if it is a destination of the token, else
 * in the hop area) to the other destinations of the token inside its server (Section 3.2; Section 4.1 step 5). */
void mwo_relay_forward_in_place(const uint8_t *hop_buf, int64_t row_bytes, int32_t R, int32_t K,
                                int32_t src_rank, int32_t ranks_per_server,
                                const int32_t *hop_rank_offsets, const int32_t *hop_rank_tokens,
                                const int32_t *flat_dest_rank, const int32_t *flat_dest_pos, const int32_t *flat_rank_offsets,
                                uint8_t *recv_base, int64_t recv_stride_bytes)
{
    const int Kd = K < R ? K : R;
    for (int32_t h = 0; h < R; ++h) {
        for (int32_t q = hop_rank_offsets[h]; q < hop_rank_offsets[h + 1]; ++q) {
            const int32_t t = hop_rank_tokens[q];
            const int slot = flat_slot_of(flat_dest_rank, flat_dest_pos, t, Kd, h);
            const uint8_t *held = slot >= 0
                ? region(recv_base, recv_stride_bytes, flat_rank_offsets, h, row_bytes) + (int64_t)slot * row_bytes
                : hop_buf + (int64_t)q * row_bytes;
            for (int i = 0; i < Kd; ++i) {
                const int32_t r = flat_dest_rank[(int64_t)t * Kd + i];
                if (r < 0 || r == h || mwo_next_hop(r, src_rank, ranks_per_server) != h) continue;
                memcpy(region(recv_base, recv_stride_bytes, flat_rank_offsets, r, row_bytes) +
                           (int64_t)flat_dest_pos[(int64_t)t * Kd + i] * row_bytes,
                       held, (size_t)row_bytes);
            }
        }
    }
}

/*
 * Paired-relay AllGather on a full mesh with two communication domains (Section 3.1, Section 5.2).
 *
 * R = 2n ranks; ranks [0, n) form one domain, [n, 2n) the other; rank r is paired with (r + n) mod 2n.
 * Each domain runs its own AllGather: afterwards every rank holds the n shards of its own domain,
 * in rank order.  A shard of shard_bytes is split in two segments: bytes [0, direct_bytes) travel on
 * the direct links to the n - 1 other members of the domain; bytes [direct_bytes, shard_bytes) go to
 * the paired rank of the other domain, which forwards them to those n - 1 members.
 *   layout 0 (MultiWrite): the relayed segment crosses the pair link once;
 *   layout 1 (unicast relay): it crosses the pair link n - 1 times, one copy per final destination.
 * relay_buf [R, copies, relay_bytes] (copies = 1 or n - 1): region p holds what rank p received from its
 * partner.  recv [R, n * shard_bytes].  Link loads are in bytes per directed link; every link has the
 * same bandwidth in the paper's model, so the transfer time is max_link_bytes / w.
 */
typedef struct {
    int64_t direct_link_bytes;    /* load of each used intra-domain link                       */
    int64_t pair_link_bytes;      /* load of each pair link (source -> its partner)            */
    int64_t forward_link_bytes;   /* load of each link partner -> member of the other domain   */
    int64_t max_link_bytes;       /* the bottleneck                                            */
    int64_t total_bytes;          /* all bytes put on links by all ranks                       */
} mwo_pair_totals;

int mwo_paired_allgather(const uint8_t *shards, int32_t R, int64_t shard_bytes, int64_t direct_bytes, int layout,
                         uint8_t *relay_buf, uint8_t *recv, mwo_pair_totals *totals)
{
    if (R < 2 || R % 2 || shard_bytes <= 0 || direct_bytes < 0 || direct_bytes > shard_bytes || (layout != 0 && layout != 1))
        return MWO_ERR_INVALID_ARG;
    const int32_t n = R / 2;
    const int64_t relay_bytes = shard_bytes - direct_bytes;
    const int64_t copies = layout == 0 ? 1 : n - 1;
    for (int32_t r = 0; r < R; ++r) {
        const int32_t dom = r / n, partner = (r + n) % R;
        const uint8_t *mine = shards + (int64_t)r * shard_bytes;
        /* own copy: local, not on any link */
        memcpy(recv + ((int64_t)r * n + r % n) * shard_bytes, mine, (size_t)shard_bytes);
        /* direct segment to the other members of the domain */
        for (int32_t q = 0; q < n; ++q) {
            const int32_t d = dom * n + q;
            if (d == r) continue;
            memcpy(recv + ((int64_t)d * n + r % n) * shard_bytes, mine, (size_t)direct_bytes);
        }
        /* relayed segment: to the partner (once, or once per final destination) ... */
        for (int64_t c = 0; c < copies; ++c)
            memcpy(relay_buf + ((int64_t)partner * copies + c) * relay_bytes, mine + direct_bytes, (size_t)relay_bytes);
        /* ... which forwards it to the other members of the source's domain */
        int64_t k = 0;
        for (int32_t q = 0; q < n; ++q) {
            const int32_t d = dom * n + q;
            if (d == r) continue;
            const int64_t c = layout == 0 ? 0 : k;
            memcpy(recv + ((int64_t)d * n + r % n) * shard_bytes + direct_bytes,
                   relay_buf + ((int64_t)partner * copies + c) * relay_bytes, (size_t)relay_bytes);
            ++k;
        }
    }
    if (totals) {
        totals->direct_link_bytes = n > 1 ? direct_bytes : 0;
        totals->pair_link_bytes = n > 1 ? copies * relay_bytes : 0;
        totals->forward_link_bytes = n > 1 ? relay_bytes : 0;
        int64_t m = totals->direct_link_bytes;
        if (totals->pair_link_bytes > m) m = totals->pair_link_bytes;
        if (totals->forward_link_bytes > m) m = totals->forward_link_bytes;
        totals->max_link_bytes = m;
        totals->total_bytes = (int64_t)R * ((n - 1) * direct_bytes + totals->pair_link_bytes + (n - 1) * totals->forward_link_bytes);
    }
    return MWO_OK;
}

/* The split that makes the direct links and the pair link finish together (Section 5.2 step 1), rounded
 * down to a multiple of 16 bytes: direct = shard * c / (1 + c) with c copies on the pair link. */
int64_t mwo_balanced_direct_bytes(int64_t shard_bytes, int32_t n, int layout)
{
    const int64_t c = layout == 0 ? 1 : n - 1;
    if (n <= 1) return shard_bytes;
    return (shard_bytes * c / (1 + c)) / 16 * 16;
}

/*
 * The split for links of two bandwidth classes (Section 5.2 step 1: the shard is cut in two by the measured
 * bandwidth ratio of the links; Section 3.1 for the traffic each link carries).  Links inside a domain run at
 * w_direct, links between the domains (the pair link and the relay's forwarding links) at w_pair, in the same
 * unit.  With d direct bytes a direct link is busy for d / w_direct and the pair link, which carries c copies of
 * the rest (c = 1 for MultiWrite, n - 1 for the unicast relay), for c (s - d) / w_pair; the forwarding links carry
 * one copy each and are never slower than the pair link.  Both finish together at
 *     d = s c w_direct / (w_pair + c w_direct),
 * taken in double precision and rounded down to a multiple of 16 bytes.  Equal bandwidths give the split of
 * mwo_balanced_direct_bytes.  Non-positive bandwidths or n <= 1: everything goes direct.
 */
int64_t mwo_split_direct_bytes(int64_t shard_bytes, int32_t n, int layout, double w_direct, double w_pair)
{
    if (n <= 1 || !(w_direct > 0.0) || !(w_pair > 0.0)) return shard_bytes;
    const double c = layout == 0 ? 1.0 : (double)(n - 1);
    const double d = floor((double)shard_bytes * c * w_direct / (w_pair + c * w_direct));
    int64_t bytes = (int64_t)d / 16 * 16;
    if (bytes > shard_bytes) bytes = shard_bytes / 16 * 16;
    return bytes;
}

/*
 * Combine: the reverse of dispatch (Section 2.3.2: the expert outputs travel back to the ranks that sent
 * the tokens; the step carries no redundant data, so MultiWrite does not change it).
 *
 * Reading taken: every destination rank r of token t returns one row z[r][dest_pos(t, r)] of bf16
 * values (its local experts' contribution), in the slot the dispatch delivered the token to; the source
 * forms  y[t] = sum over the destinations of t, in ascending rank order, of w[t, i] * z[r_i][slot_i]
 * with the sum carried in double precision here and rounded once to bf16 (round to nearest even).
 * weights == NULL means all ones.  A token without destinations gets a row of zeros.
 */
static double bf16_to_double(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* double -> bf16 bits, one rounding (nearest even), bf16 = sign, 8 exponent bits, 7 fraction bits */
static uint16_t double_to_bf16(double x)
{
    if (isnan(x)) return 0x7FC0;
    uint16_t sign = signbit(x) ? 0x8000 : 0;
    double a = fabs(x);
    if (a == 0.0) return sign;
    if (isinf(a)) return sign | 0x7F80;
    int e;
    frexp(a, &e);                                   /* a = m * 2^e, m in [0.5, 1)  ->  a in [2^(e-1), 2^e) */
    int ex = e - 1;                                 /* unbiased exponent of a                               */
    if (ex < -126) ex = -126;                       /* subnormal range: fixed scale                         */
    double q = nearbyint(ldexp(a, 7 - ex));         /* significand in units of 2^(ex-7), ties to even       */
    if (q >= 256.0) { q = 128.0; ++ex; }            /* rounding carried into the next binade                */
    if (ex > 127) return sign | 0x7F80;
    if (q < 128.0) return sign | (uint16_t)q;       /* subnormal (or zero)                                  */
    return sign | (uint16_t)(((ex + 127) << 7) | ((int)q - 128));
}

void mwo_combine(const uint8_t *z_base, int64_t z_stride_bytes, const float *weights, int32_t T, int32_t R, int32_t K,
                 int64_t row_bytes, const int32_t *dest_rank, const int32_t *dest_pos, const int32_t *rank_offsets,
                 uint8_t *y)
{
    const int Kd = K < R ? K : R;
    const int64_t H = row_bytes / 2;
    for (int32_t t = 0; t < T; ++t) {
        uint16_t *out = (uint16_t *)(y + (int64_t)t * row_bytes);
        for (int64_t c = 0; c < H; ++c) {
            double acc = 0.0;
            int any = 0;
            for (int i = 0; i < Kd; ++i) {
                const int32_t r = dest_rank[(int64_t)t * Kd + i];
                if (r < 0) break;
                const uint8_t *row = region((uint8_t *)z_base, z_stride_bytes, rank_offsets, r, row_bytes) +
                                     (int64_t)dest_pos[(int64_t)t * Kd + i] * row_bytes;
                const double w = weights ? (double)weights[(int64_t)t * Kd + i] : 1.0;
                acc += w * bf16_to_double(((const uint16_t *)row)[c]);
                any = 1;
            }
            out[c] = any ? double_to_bf16(acc) : 0;
        }
    }
}

/*
 * The same combine with the precision of the accelerator path stated operation by operation (the paper
 * fixes none; Section 2.3.2 only names the step): the sum is carried in IEEE binary32, starting from +0,
 * one fused multiply-add  acc = fma(w[t, i], z, acc)  per destination in ascending rank order (the product
 * is not rounded on its own), and the binary32 sum is rounded once to bf16 (nearest even).  fmaf() of C99
 * is correctly rounded, so every step below is exactly defined and the result is unique bit for bit.
 * mwo_combine (binary64 sum) stays the accuracy reference: the two differ by at most the accumulated
 * binary32 rounding errors plus one bf16 unit in the last place.
 */
void mwo_combine_f32(const uint8_t *z_base, int64_t z_stride_bytes, const float *weights, int32_t T, int32_t R, int32_t K,
                     int64_t row_bytes, const int32_t *dest_rank, const int32_t *dest_pos, const int32_t *rank_offsets,
                     uint8_t *y)
{
    const int Kd = K < R ? K : R;
    const int64_t H = row_bytes / 2;
    for (int32_t t = 0; t < T; ++t) {
        uint16_t *out = (uint16_t *)(y + (int64_t)t * row_bytes);
        for (int64_t c = 0; c < H; ++c) {
            float acc = 0.0f;
            int any = 0;
            for (int i = 0; i < Kd; ++i) {
                const int32_t r = dest_rank[(int64_t)t * Kd + i];
                if (r < 0) break;
                const uint8_t *row = region((uint8_t *)z_base, z_stride_bytes, rank_offsets, r, row_bytes) +
                                     (int64_t)dest_pos[(int64_t)t * Kd + i] * row_bytes;
                const float w = weights ? weights[(int64_t)t * Kd + i] : 1.0f;
                const float z = (float)bf16_to_double(((const uint16_t *)row)[c]);      /* exact: bf16 is a subset of binary32 */
                acc = fmaf(w, z, acc);
                any = 1;
            }
            out[c] = any ? double_to_bf16((double)acc) : 0;                             /* binary32 -> binary64 is exact: one rounding */
        }
    }
}

/*
 * Group-major receive order (Section 4.3.1: one MultiWrite writes ONE source buffer B_S into ONE target buffer
 * B_i at every destination D_i; Section 4.3.2: the call takes an array of remote buffer addresses).
 * With the receive region of rank r laid out group by group (groups in id order, members in token order), the
 * group g is exactly one such call: B_S = send_mw[group_offsets[g] .. +size), B_i = region(D_i)[start .. +size)
 * with start = group_dest_offset[g][i].
 *
 *   group_dest_rank   [G, Kd]  destination ranks of group g, ascending, -1 padded
 *   group_dest_offset [G, Kd]  first slot of the group's block inside the region of that rank, -1 padded
 *   dest_pos_gm       [T, Kd]  slot of token t in the region of its i-th destination rank, -1 padded
 * Rows of the three arrays beyond G (or T) are not touched.  Region sizes are those of the plan (rank_offsets).
 */
void mwo_group_major(int32_t T, int32_t R, int32_t K, int64_t G, const uint64_t *group_mask, const int32_t *group_offsets,
                     const int32_t *token_group, const int32_t *token_mw_row,
                     int32_t *group_dest_rank, int32_t *group_dest_offset, int32_t *dest_pos_gm)
{
    const int W = mwo_words(R);
    const int Kd = K < R ? K : R;
    int32_t *filled = (int32_t *)calloc((size_t)R, sizeof(int32_t));      /* slots used so far in each region */
    if (!filled) return;
    for (int64_t g = 0; g < G; ++g) {
        const int32_t size = group_offsets[g + 1] - group_offsets[g];
        int i = 0;
        for (int32_t r = 0; r < R; ++r) {
            if (!(group_mask[g * W + r / 64] >> (r % 64) & 1)) continue;
            group_dest_rank[g * Kd + i] = r;
            group_dest_offset[g * Kd + i] = filled[r];
            filled[r] += size;
            ++i;
        }
        for (; i < Kd; ++i) { group_dest_rank[g * Kd + i] = -1; group_dest_offset[g * Kd + i] = -1; }
    }
    free(filled);
    for (int32_t t = 0; t < T; ++t) {
        const int32_t g = token_group[t];
        for (int i = 0; i < Kd; ++i) {
            if (g < 0 || group_dest_rank[(int64_t)g * Kd + i] < 0) { dest_pos_gm[(int64_t)t * Kd + i] = -1; continue; }
            const int32_t within = token_mw_row[t] - group_offsets[g];
            dest_pos_gm[(int64_t)t * Kd + i] = group_dest_offset[(int64_t)g * Kd + i] + within;
        }
    }
}

/* One MultiWrite per group: the group's slice of the send buffer goes, as one block, to every destination. */
void mwo_deliver_group_major(const uint8_t *send_mw, int64_t row_bytes, int32_t R, int32_t K, int64_t G,
                             const int32_t *group_offsets, const int32_t *group_dest_rank, const int32_t *group_dest_offset,
                             const int32_t *rank_offsets, uint8_t *recv_base, int64_t recv_stride_bytes)
{
    const int Kd = K < R ? K : R;
    for (int64_t g = 0; g < G; ++g) {
        const int64_t size = group_offsets[g + 1] - group_offsets[g];
        const uint8_t *b_s = send_mw + (int64_t)group_offsets[g] * row_bytes;
        for (int i = 0; i < Kd; ++i) {
            const int32_t r = group_dest_rank[g * Kd + i];
            if (r < 0) continue;
            uint8_t *b_i = region(recv_base, recv_stride_bytes, rank_offsets, r, row_bytes) +
                           (int64_t)group_dest_offset[g * Kd + i] * row_bytes;
            memcpy(b_i, b_s, (size_t)(size * row_bytes));
        }
    }
}

/*
 * Expert index of the receive regions (Section 2.3.2: a token goes to the nodes that host its selected experts;
 * on arrival each local expert must find its tokens).  A row is stored once per rank, so a token chosen by two
 * experts of one rank cannot sit in two places: the region keeps its order and every expert gets a list instead.
 *
 *   expert_offsets [E + 1]  exclusive prefix sum of the number of distinct tokens that selected expert e
 *                           (experts whose table entry is outside [0, R) count nothing)
 *   expert_token   [T * K]  for each expert in id order, its tokens in ascending order; -1 beyond the total
 *   expert_slot    [T * K]  the slot of that token inside the region of the expert's rank (token-major order)
 * Returns the total number of (token, expert) pairs.
 */
int64_t mwo_expert_index(const int32_t *topk_ids, const int32_t *expert_to_rank, int32_t T, int32_t K, int32_t E, int32_t R,
                         const int32_t *dest_rank, const int32_t *dest_pos,
                         int32_t *expert_offsets, int32_t *expert_token, int32_t *expert_slot)
{
    const int Kd = K < R ? K : R;
    int64_t P = 0;
    for (int32_t e = 0; e < E; ++e) {
        expert_offsets[e] = (int32_t)P;
        const int32_t r = expert_to_rank[e];
        if (r < 0 || r >= R) continue;
        for (int32_t t = 0; t < T; ++t) {
            int hit = 0;
            for (int32_t k = 0; k < K; ++k) hit |= (topk_ids[(int64_t)t * K + k] == e);
            if (!hit) continue;
            int32_t slot = -1;
            for (int i = 0; i < Kd; ++i)
                if (dest_rank[(int64_t)t * Kd + i] == r) slot = dest_pos[(int64_t)t * Kd + i];
            expert_token[P] = t;
            expert_slot[P] = slot;
            ++P;
        }
    }
    expert_offsets[E] = (int32_t)P;
    for (int64_t i = P; i < (int64_t)T * K; ++i) { expert_token[i] = -1; expert_slot[i] = -1; }
    return P;
}
