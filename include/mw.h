/*
 * mw.h -- C ABI of the MultiWrite dispatch / AllGather pack-and-deliver library (CUDA, sm_100a).
 *
 * The library emulates a communication domain of R ranks as R receive regions in one
 * GPU's memory and performs, on the device, the source-side and relay-side work of
 * the paper's MultiWrite semantic:
 *
 *   MultiWrite(S, M, B_S), M = {(D_i, B_i)}: the content of the source buffer B_S is
 *   written into the target buffer B_i of every destination D_i   (Section 4.3.1).
 *
 * For MoE dispatch the destinations of a token are the ranks hosting its top-k experts
 * (Sections 1, 2.3.2); the destination set travels as a bitmap, one bit per rank, ranks
 * numbered from zero (Section 4.1; Section 6.4 for more than 64 ranks).  The unicast
 * layout sends one copy per destination (Section 2.2) and is kept as the comparison.
 *
 * Conventions for every call
 *   - All pointers marked "device" are CUDA device pointers valid on the context's
 *     device; "host" pointers are ordinary host memory.  `stream` is a cudaStream_t
 *     passed as void* (NULL = the legacy default stream).
 *   - The caller owns every buffer it passes.  The context owns the plan metadata and
 *     its scratch, all allocated in mw_create; no other call allocates device memory,
 *     except mw_dispatch_host, which uses staging buffers allocated in mw_create when
 *     MW_FLAG_HOST_STAGING is set.
 *   - Calls are asynchronous on `stream` unless stated otherwise; results are defined
 *     once the stream has completed ("atomic per destination, no ordering between
 *     destinations", Section 4.3.4).  A context must be driven from one stream at a time.
 *   - Every call returns MW_OK or a negative MW_ERR_* code.  Errors that the host can
 *     see (null pointer, misalignment, sizes beyond the configured maxima) are returned
 *     at once and nothing is launched.  Errors that depend on device data (an expert id
 *     outside {-1} U [0,E), a table entry outside [0,R), a row that would land beyond a
 *     buffer's capacity, a wait that gave up) are recorded in mw_totals.status on the
 *     device, the offending write is suppressed, and mw_get_totals reports them.
 *     Nothing traps or aborts.
 *
 * Layout rules (the paper fixes the bytes each destination receives; the slots are this
 * library's choice)
 *   - rank r is bit (r mod 64), least significant first, of 64-bit word (r / 64);
 *     W = ceil(R / 64) words per bitmap; bits >= R are zero;
 *   - destination sets are per rank: experts of one token on the same rank set one bit;
 *   - a group is the set of all tokens with the same non-empty bitmap; groups are numbered
 *     by first occurrence in token order; rows of a group, and rows of a receive region,
 *     keep ascending token order;
 *   - expert id -1 is padding and is skipped; a token whose bitmap is empty has no group,
 *     no send row (token_group = token_mw_row = -1) and moves no bytes.
 */
#ifndef MW_H_
#define MW_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define MW_API __attribute__((visibility("default")))
#else
#define MW_API
#endif

#define MW_OK                0
#define MW_ERR_INVALID_ARG  (-1)  /* null pointer, size out of range, unknown layout          */
#define MW_ERR_ALIGNMENT    (-2)  /* pointer, stride or row size not a multiple of 16 bytes   */
#define MW_ERR_CAPACITY     (-3)  /* a buffer cannot hold the rows the plan assigns to it     */
#define MW_ERR_CUDA         (-4)  /* a CUDA runtime call failed                               */
#define MW_ERR_BAD_INDEX    (-5)  /* expert id or expert->rank entry out of range (ignored)   */
#define MW_ERR_TIMEOUT      (-6)  /* a bounded device-side wait gave up; the plan is invalid  */
                                  /* and the context refuses further work until mw_reset      */
#define MW_ERR_NO_PLAN      (-7)  /* dispatch called before any plan                          */

#define MW_LAYOUT_MULTIWRITE 0    /* send buffer holds each row once (one row per group member) */
#define MW_LAYOUT_UNICAST    1    /* send buffer holds one copy per destination                */

#define MW_FLAG_HOST_STAGING   0x1u  /* allocate device staging so mw_dispatch_host can be used */
#define MW_FLAG_PLAN_MULTIPASS 0x2u  /* always take the tiled multi-kernel plan, even for small T (its tiles take   */
                                     /* tickets, so it does not need all its blocks resident at once)               */
#define MW_FLAG_NO_OVERLAP     0x10u /* do not let a kernel's start-up overlap the previous kernel's tail */
#define MW_FLAG_COPY_BULK      0x40u /* persistent grid, bulk (TMA) loads into shared memory and bulk stores out of it; */
                                     /* without it row copies run one block per (row, piece) with plain 16-byte loads   */
                                     /* and stores, which measured fastest on B200                                      */
#define MW_FLAG_SHORT_WAITS    0x80u /* device-side waits give up after about a millisecond instead of about a second   */
                                     /* (for latency-critical hosts that prefer an early MW_ERR_TIMEOUT, and for tests) */

#define MW_MAX_RANKS   1024
#define MW_MAX_TOPK    64
#define MW_STATIC_MAX_TOKENS 16384   /* largest T of mw_group_tokens_static */

typedef struct mw_ctx mw_ctx;   /* opaque: configuration, device workspace, plan metadata */

typedef struct {
    int32_t  R;           /* ranks in the emulated domain, 1..MW_MAX_RANKS                         */
    int32_t  E;           /* experts (length of expert_to_rank), >= 1                              */
    int32_t  K;           /* router top-k (columns of topk_ids), 1..MW_MAX_TOPK                    */
    int32_t  max_tokens;  /* largest T any mw_plan call will pass, >= 1                            */
    int64_t  row_bytes;   /* B: bytes per hidden row, a positive multiple of 16                    */
    int32_t  src_rank;    /* sender's own rank, or -1 if it is outside the domain (Section 2.3.1:  */
                          /* the copy to oneself is local and not counted as transmitted)          */
    int32_t  device;      /* CUDA device ordinal                                                   */
    uint32_t flags;       /* MW_FLAG_*                                                             */
    uint32_t reserved;
} mw_config;

/* Exact byte accounting of the last plan (64-bit integers; no measurement involved). */
typedef struct {
    int64_t T_nonempty;               /* T': tokens with at least one destination                   */
    int64_t G;                        /* distinct non-empty destination sets = MultiWrite groups    */
    int64_t total_dest;               /* sum over tokens of |D_t| = rows delivered                   */
    int64_t mw_bytes;                 /* transmitted when every row is sent once (Section 1)        */
    int64_t unicast_bytes;            /* transmitted with one copy per destination (Section 2.2)    */
    int64_t unicast_per_expert_bytes; /* one copy per valid expert slot (no per-rank dedup)         */
    int64_t meta_bytes;               /* bitmap bytes carried in the payload when R > 64, one       */
                                      /* bitmap per 4096-byte packet (Section 6.4); 0 otherwise     */
    int32_t status;                   /* MW_OK or the first device-side MW_ERR_* of plan/dispatch   */
    int32_t reserved;
} mw_totals;

/*
 * Device pointers into the context's workspace, valid until mw_destroy; contents are those
 * of the latest mw_plan once its stream work has completed.  Kd = min(K, R).
 * Entries past the defined prefix hold -1 (masks: 0).
 */
typedef struct {
    const uint64_t  *token_mask;    /* [T, W]    destination bitmap of each token                   */
    const int32_t   *token_ndest;   /* [T]       |D_t|                                              */
    const int32_t   *token_group;   /* [T]       group id, -1 if D_t is empty                       */
    const int32_t   *token_mw_row;  /* [T]       row of the token in the MultiWrite send buffer     */
    const int32_t   *mw_row_token;  /* [T]       inverse of the above; first T' entries defined     */
    const int32_t   *group_offsets; /* [T + 1]   exclusive prefix sum of group sizes; G + 1 defined */
    const uint64_t  *group_mask;    /* [T, W]    bitmap of each group; first G rows defined         */
    const int32_t   *rank_offsets;  /* [R + 1]   exclusive prefix sum of rows per receive region    */
    const int32_t   *rank_tokens;   /* [T * Kd]  token of every delivered row, region-major         */
    const int32_t   *dest_rank;     /* [T, Kd]   ascending destination ranks of the token, -1 pad   */
    const int32_t   *dest_pos;      /* [T, Kd]   slot of the token inside that rank's region        */
    const mw_totals *totals;        /* device copy of the accounting                                */
    int32_t T, W, Kd, reserved;
} mw_plan_view;

/*
 * Creates a context: validates the configuration, selects cfg->device, allocates all
 * device workspace (sized for max_tokens and the worst case of Kd destinations per token).
 * Corresponds to the paper's initialisation module, which loads the node configuration
 * (Section 5.1, cs_ini).  Synchronous.  *out is NULL on failure.
 */
MW_API int mw_create(mw_ctx **out, const mw_config *cfg);

/* Frees everything mw_create allocated.  Synchronises the device first.  NULL is accepted. */
MW_API int mw_destroy(mw_ctx *ctx);

/*
 * Makes a context usable again after MW_ERR_TIMEOUT.  The device-side waits of this library (a plan tile waiting
 * for the counts of the tiles before it, a plan block waiting at a grid barrier, a tile of mw_group_major waiting
 * for the sums of the tiles before it, a copy pipeline waiting for a bulk load) are bounded; when one gives up, mw_totals.status says MW_ERR_TIMEOUT, the kernels that follow skip
 * their work, and from the mw_get_totals that reported it every call on the context except mw_get_totals,
 * mw_reset and mw_destroy returns MW_ERR_TIMEOUT.  (A plan can run into this when other work keeps the GPU's SMs
 * occupied for about a second, so that its blocks cannot all become resident.)  mw_reset waits for the device,
 * empties the scratch the plans share (their running counts included); no plan exists afterwards (the next
 * call must be a plan).  Nothing is reallocated.  Synchronous.
 */
MW_API int mw_reset(mw_ctx *ctx);

/*
 * Source-side planning (Section 4.1 step 1: the source turns the destination information
 * into bitmap metadata; Section 5.1, cs_send: task decomposition).  From the router output
 * it builds bitmaps, groups, per-group and per-rank counts with exclusive prefix sums, every
 * token's send row and receive slots, and the byte accounting.
 *
 *   topk_ids        device, int32 [T, K] row-major; -1 = padding
 *   expert_to_rank  device, int32 [E], values in [0, R)  (the preconfigured table of Section 4.1)
 *   T               0 <= T <= max_tokens
 *   view            host, optional: receives the workspace pointers (same every call)
 */
MW_API int mw_plan(mw_ctx *ctx, const int32_t *topk_ids, const int32_t *expert_to_rank, int32_t T,
            mw_plan_view *view, void *stream);

/*
 * mw_plan with one more argument: the hidden rows x (device, [T, row_bytes], 16-byte aligned; may be NULL when T is 0) that the pack step
 * will load into the send buffer next (Section 5.2 step 1).  Same plan, same results.  Planning is a chain of
 * dependent steps on a few SMs and leaves the memory system idle, so the launch carries extra blocks that ask
 * the L2 cache for the first rows of x (up to half the cache) meanwhile; mw_pack / mw_dispatch then find them
 * there.  x is only read.  It must not be written by work that runs concurrently with the plan.
 */
MW_API int mw_plan_prefetch(mw_ctx *ctx, const int32_t *topk_ids, const int32_t *expert_to_rank, int32_t T,
                     const void *x, mw_plan_view *view, void *stream);

/*
 * Planning one batch ahead.  A plan is a short chain of dependent steps on a few SMs and moves almost no data, while
 * pack and deliver are bound by memory bandwidth; the source-side preparation of the next write can therefore run
 * while the replication of the current one is in flight (Section 5.1: cs_send prepares work requests while the
 * relay thread copies and forwards).  The context holds two plan slots:
 *
 *   mw_plan_next   plans a batch into the slot the data path is NOT using, on a stream the library owns.  The plan
 *                  starts once everything submitted to `stream` so far has completed (its inputs are ready, and the
 *                  copy kernels that read that slot two batches ago are done) and then runs concurrently with whatever
 *                  is submitted to `stream` afterwards.  x (optional, may be NULL) as in mw_plan_prefetch.
 *   mw_plan_swap   makes that plan the current one: `stream` waits for it (no host synchronisation) and every call
 *                  that "uses the latest plan" now uses it; `view` (optional) receives its arrays.  MW_ERR_NO_PLAN when
 *                  no mw_plan_next is outstanding.  Views and plan arrays of the slot swapped out stay valid until the
 *                  next mw_plan_next overwrites them.
 *
 * Steady state, batch i (one stream, one context):
 *     mw_plan_swap(ctx, &view, s);                          the plan of batch i, issued one iteration ago
 *     mw_plan_next(ctx, ids[i+1], e2r, T[i+1], x[i+1], s);  before the copies of batch i are submitted
 *     mw_pack(ctx, x[i], ...s);  mw_deliver(ctx, ...s);     run while batch i+1 is being planned
 * The inputs of a pending mw_plan_next must not be overwritten before the matching mw_plan_swap's stream work.
 * mw_plan, mw_plan_prefetch and mw_plan_dispatch plan into the current slot and may be mixed with the pair above
 * (plans are ordered among themselves by the library); an outstanding mw_plan_next stays outstanding.
 */
MW_API int mw_plan_next(mw_ctx *ctx, const int32_t *topk_ids, const int32_t *expert_to_rank, int32_t T, const void *x,
                        void *stream);
MW_API int mw_plan_swap(mw_ctx *ctx, mw_plan_view *view, void *stream);

/* Fills `view` with the workspace pointers of the context and the T of its latest plan (no device work). */
MW_API int mw_get_plan_view(mw_ctx *ctx, mw_plan_view *view);

/* Waits for `stream`, then copies the accounting of the latest plan to host memory. */
MW_API int mw_get_totals(mw_ctx *ctx, mw_totals *host_out, void *stream);

/*
 * Pack: fill the send buffer from the hidden rows, using the latest plan (Section 5.2 step 1: every rank first
 * copies its own data into a send buffer allocated beforehand).
 *   MW_LAYOUT_MULTIWRITE  send_buf[j] = x[mw_row_token[j]],            j < T'
 *   MW_LAYOUT_UNICAST     send_buf[rank_offsets[r] + i] = x[rank_tokens[rank_offsets[r] + i]]
 *   x         device, [T, row_bytes], 16-byte aligned
 *   send_buf  device, send_capacity_rows * row_bytes bytes, 16-byte aligned; rows beyond the
 *             capacity are not written and set MW_ERR_CAPACITY in the status
 */
MW_API int mw_pack(mw_ctx *ctx, const void *x, int layout, void *send_buf, int64_t send_capacity_rows, void *stream);

/*
 * Deliver: expand the send buffer into the R receive regions (Section 4.1 steps 3-5 and
 * Section 4.3.3 with every destination as its own next hop: the relay reads the payload it
 * holds and writes one copy per set bit of the bitmap).
 *   MW_LAYOUT_MULTIWRITE  for each send row j and each set bit r of its group's bitmap:
 *                         region(r)[dest_pos(token, r)] = send_buf[j]
 *   MW_LAYOUT_UNICAST     region(r)[i] = send_buf[rank_offsets[r] + i]
 * Both give region(r) = the rows of all tokens bound for r, in ascending token order.
 *   recv_base           device, 16-byte aligned
 *   recv_stride_bytes   > 0: region(r) starts at recv_base + r * stride (multiple of 16) and holds
 *                       at most recv_capacity_rows rows;
 *                       0: compact, region(r) starts at row rank_offsets[r] and the whole area
 *                       holds at most recv_capacity_rows rows
 */
MW_API int mw_deliver(mw_ctx *ctx, int layout, const void *send_buf, void *recv_base, int64_t recv_stride_bytes,
               int64_t recv_capacity_rows, void *stream);

/*
 * mw_deliver with every receive region named by its own base address, the form the paper gives its interface
 * (Section 4.3.2: used like a standard write, but accepts an array of remote buffer addresses instead of one;
 * Section 4.3.1: the payload is written into buffer B_i at every destination D_i).
 *   recv_ptrs           device, array of R addresses (8-byte aligned array); entry r is the start of region(r),
 *                       16-byte aligned, room for recv_capacity_rows rows.  Entries of ranks that receive nothing
 *                       are not looked at.  The addresses are read on the device: a null or misaligned entry of a
 *                       rank that does receive rows sets MW_ERR_INVALID_ARG / MW_ERR_ALIGNMENT in the accounting
 *                       status (mw_get_totals) and that region is not written.
 * Same rows in the same order as mw_deliver.
 */
MW_API int mw_deliver_ptrs(mw_ctx *ctx, int layout, const void *send_buf, void *const *recv_ptrs,
                    int64_t recv_capacity_rows, void *stream);

/*
 * The whole data movement of one dispatch, with the results of mw_pack followed by mw_deliver (same send buffer,
 * same receive regions, bit for bit) but in one pass: every hidden row is read once and written to its send
 * slot(s) and to all its receive slots.  With MW_FLAG_COPY_BULK it is the two calls in sequence.
 */
MW_API int mw_dispatch(mw_ctx *ctx, const void *x, int layout, void *send_buf, int64_t send_capacity_rows,
                void *recv_base, int64_t recv_stride_bytes, int64_t recv_capacity_rows, void *stream);

/*
 * mw_plan followed by mw_dispatch in one call (same arguments, same results, the context is left
 * in the same state).  For small batches in the MultiWrite layout (T <= 1024, R <= 256, min(K, R)
 * <= 16: the batch sizes of Section 6.3, from the decode-sized ones, where the paper finds the
 * replication overhead to outweigh the savings, up to its batch of 1k) the three kernels are
 * replaced by a single launch in which every block recomputes the plan in shared memory and then
 * moves its share of the rows (256 threads per block up to 128 tokens, 1024 beyond); larger
 * batches, the unicast layout and contexts created with MW_FLAG_PLAN_MULTIPASS take the
 * ordinary three-kernel route (planning through mw_plan_prefetch).
 * The single launch keeps no state on the host, so a call captured into a CUDA graph may be replayed
 * (new ids and rows in the same buffers).  So may mw_plan / mw_plan_prefetch followed by mw_pack, mw_deliver or
 * mw_dispatch: the running counts of the tiled plan (epoch of its look-back records, barrier arrivals, tile tickets)
 * live on the device and are advanced by the plan kernels themselves.  (mw_plan_next / mw_plan_swap use a second
 * stream and events; capturing them is not covered here.)
 */
MW_API int mw_plan_dispatch(mw_ctx *ctx, const int32_t *topk_ids, const int32_t *expert_to_rank, int32_t T,
                            const void *x, int layout, void *send_buf, int64_t send_capacity_rows, void *recv_base,
                            int64_t recv_stride_bytes, int64_t recv_capacity_rows, mw_plan_view *view, void *stream);

/*
 * AllGather pack + deliver (Section 5.2): R ranks each contribute one shard of shard_bytes;
 * every destination rank ends with shard_0 | shard_1 | ... | shard_{R-1}.  Uses cfg.R only.
 *   shards       device, [R, shard_bytes] contiguous, 16-byte aligned; shard_bytes multiple of 16
 *   layout       MW_LAYOUT_MULTIWRITE: send_buf [R, shard_bytes], every shard once;
 *                MW_LAYOUT_UNICAST:    send_buf [R, dst_rank_count, shard_bytes]; slot (i, d) is the
 *                copy of shard i addressed to rank dst_rank_begin + d; the slot addressed to
 *                rank i itself is never written (that copy is local: Section 2.3.1)
 *   recv_base    device; region d (rank dst_rank_begin + d) starts at recv_base + d * stride,
 *                stride = recv_stride_bytes, or R * shard_bytes when 0
 *   dst_rank_begin, dst_rank_count   the window of destination ranks that is materialised
 *                (the full R x R result need not fit in memory); accounting is for the full domain
 *   host_totals  host, optional: receives the accounting (filled synchronously, no device work)
 */
MW_API int mw_allgather_pack(mw_ctx *ctx, const void *shards, int64_t shard_bytes, int layout, void *send_buf,
                      void *recv_base, int64_t recv_stride_bytes, int32_t dst_rank_begin, int32_t dst_rank_count,
                      mw_totals *host_totals, void *stream);

/*
 * Combine: the reverse of dispatch (Section 2.3.2: results return from the experts to their senders;
 * the step carries no redundant data and is not changed by MultiWrite).  Uses the latest plan.
 * Every destination rank r of token t has put one bf16 row into z at the slot the dispatch delivered
 * the token to (same compact or strided layout as the receive area); the source computes
 *     y[t] = sum over the destinations of t, in ascending rank order, of weights[t, i] * z[r_i][slot_i]
 * with fp32 accumulation by fused multiply-add in that order and one rounding to bf16 (nearest even).
 * Rows are row_bytes / 2 bf16 values; this is the only call that interprets the payload.
 *   z_base          device, 16-byte aligned; z_stride_bytes as recv_stride_bytes of mw_deliver (0 = compact)
 *   weights         device float32 [T, Kd] (entry i belongs to the i-th destination rank, ascending), or
 *                   NULL for all ones
 *   y               device, [T, row_bytes]; a token without destinations gets zeros
 */
MW_API int mw_combine(mw_ctx *ctx, const void *z_base, int64_t z_stride_bytes, const float *weights, void *y, void *stream);

/*
 * Group-major receive order.  Section 4.3.1 defines MultiWrite(S, M, B_S) as writing ONE source buffer B_S into
 * ONE target buffer B_i at every destination D_i, and Section 4.3.2 gives the call an array of remote buffer
 * addresses.  With the region of every rank laid out group by group (groups in id order, members in ascending
 * token order) each group of the latest plan is exactly one such call:
 *     B_S = send buffer rows [group_offsets[g], group_offsets[g + 1])      (MultiWrite layout)
 *     D_i = group_dest_rank[g][i],   B_i = region(D_i) rows [group_dest_offset[g][i], + size of the group)
 * mw_group_major derives these arrays from the latest plan (region sizes and rank_offsets are unchanged; only
 * the order of the rows inside a region differs from mw_deliver's token-major order):
 *     group_dest_rank    device int32 [max_tokens, Kd]   first G rows defined, -1 padded
 *     group_dest_offset  device int32 [max_tokens, Kd]   first G rows defined, -1 padded
 *     dest_pos_gm        device int32 [max_tokens, Kd]   first T rows: slot of token t at its i-th destination
 * The arrays belong to the context and are overwritten by the next mw_group_major.  view (host, optional)
 * receives their addresses.  mw_deliver_group_major expands the MultiWrite-layout send buffer into regions in
 * that order (arguments as mw_deliver); it needs mw_group_major to have run after the latest plan
 * (else MW_ERR_NO_PLAN).
 */
typedef struct mw_group_major_view {
    int32_t *group_dest_rank;
    int32_t *group_dest_offset;
    int32_t *dest_pos_gm;
    int32_t  Kd;
    int32_t  reserved;
} mw_group_major_view;

MW_API int mw_group_major(mw_ctx *ctx, mw_group_major_view *view, void *stream);
MW_API int mw_deliver_group_major(mw_ctx *ctx, const void *send_buf, void *recv_base, int64_t recv_stride_bytes,
                           int64_t recv_capacity_rows, void *stream);

/*
 * Expert index of the receive regions (Section 2.3.2: a token is sent to the nodes that host its selected
 * experts; each local expert then has to find its tokens).  A row is stored once per rank, so the regions keep
 * their order and every expert gets a list.  Uses the latest plan; topk_ids / expert_to_rank must be the arrays
 * that plan was made from.
 *     expert_offsets  device int32 [E + 1]  exclusive prefix sum of the number of distinct tokens that selected
 *                                           expert e (experts whose table entry is outside [0, R) count nothing)
 *     expert_token    device int32 [T * K]  per expert in id order, its tokens ascending; -1 beyond the total
 *     expert_slot     device int32 [T * K]  slot of that token in the region of the expert's rank (token-major
 *                                           order, i.e. the order mw_deliver and mw_dispatch produce)
 * MW_ERR_CAPACITY when E is too large for the kernel's shared memory (36 bytes per expert) or for
 * the per-tile count table (max_tokens / 256 x E entries, at most 256 MB).
 */
MW_API int mw_expert_index(mw_ctx *ctx, const int32_t *topk_ids, const int32_t *expert_to_rank, int32_t *expert_offsets,
                    int32_t *expert_token, int32_t *expert_slot, void *stream);

/*
 * Paired-relay AllGather with segment split (the paired relaying of Section 3.1; Section 5.2): cfg.R = 2n
 * ranks on a full mesh form two domains, [0, n) and [n, 2n); rank r is paired with (r + n) mod 2n.
 * Each domain gathers its own n shards: afterwards the receive region of every rank holds the shards
 * of its domain in rank order.  Bytes [0, direct_bytes) of a shard go on the direct links to the other
 * members of the domain; bytes [direct_bytes, shard_bytes) go to the paired rank, which forwards them
 * to those members.  MW_LAYOUT_MULTIWRITE: the relayed segment crosses the pair link once;
 * MW_LAYOUT_UNICAST: n - 1 times, one copy per final destination.
 *   shards      device, [R, shard_bytes]; shard_bytes and direct_bytes multiples of 16
 *   relay_buf   device, [R, copies, shard_bytes - direct_bytes], copies = 1 or n - 1: region p is what
 *               rank p received from its partner
 *   recv_base   device, [R, n * shard_bytes]
 *   host_totals host, optional: bytes per directed link (every link has the same bandwidth in the
 *               paper's model, so the transfer time is max_link_bytes / bandwidth)
 */
typedef struct {
    int64_t direct_link_bytes;    /* load of each used intra-domain link                     */
    int64_t pair_link_bytes;      /* load of each pair link (source -> its partner)          */
    int64_t forward_link_bytes;   /* load of each link partner -> member of the other domain */
    int64_t max_link_bytes;       /* the bottleneck                                          */
    int64_t total_bytes;          /* all bytes put on links by all ranks                     */
} mw_pair_totals;

MW_API int mw_paired_allgather(mw_ctx *ctx, const void *shards, int64_t shard_bytes, int64_t direct_bytes, int layout,
                               void *relay_buf, void *recv_base, mw_pair_totals *host_totals, void *stream);

/* The split that lets the direct links and the pair link finish together (Section 5.2 step 1, equal link
 * bandwidths): shard_bytes * c / (1 + c) with c copies on the pair link, rounded down to a multiple of 16. */
MW_API int64_t mw_pair_balanced_direct_bytes(int64_t shard_bytes, int32_t ranks_per_domain, int layout);

/* The same split for links of two bandwidth classes (Section 5.2 step 1: the shard is cut by the measured bandwidth
 * ratio): links inside a domain run at w_direct, links between the domains at w_pair (same unit, both > 0).  A direct
 * link carries d bytes and the pair link c copies of the rest, so both finish together at
 * d = shard_bytes * c * w_direct / (w_pair + c * w_direct), evaluated in double precision and rounded down to a
 * multiple of 16.  Equal bandwidths give mw_pair_balanced_direct_bytes; a non-positive bandwidth or a single-rank
 * domain returns shard_bytes (everything direct).  Host arithmetic only. */
MW_API int64_t mw_pair_split_direct_bytes(int64_t shard_bytes, int32_t ranks_per_domain, int layout, double w_direct,
                                          double w_pair);

/*
 * One whole dispatch from host memory (plan, pack, deliver) for callers whose data lives on
 * the host: copies topk_ids, expert_to_rank and x to the device, runs mw_plan and mw_dispatch
 * into context-owned staging, and copies the compact receive area (total_dest rows), the
 * rank offsets and the accounting back.  Needs MW_FLAG_HOST_STAGING.  Synchronises `stream`.
 *   recv_host              host, at least recv_capacity_rows * row_bytes bytes
 *   rank_offsets_host      host, int32 [R + 1]
 * Pinned host memory makes the copies asynchronous; pageable memory also works.
 */
MW_API int mw_dispatch_host(mw_ctx *ctx, const int32_t *topk_ids_host, const int32_t *expert_to_rank_host,
                     const void *x_host, int32_t T, int layout, void *recv_host, int64_t recv_capacity_rows,
                     int32_t *rank_offsets_host, mw_totals *totals_host, void *stream);

/* ------------------------------------------------------------------------------------------------
 * Two-level (relayed) MultiWrite dispatch: Section 3.2 (oversubscribed inter-server bandwidth),
 * Section 4.1 "Local forwarding table" (one copy per distinct next hop) and Section 4.3.3 (M is
 * partitioned by next hop; a relay re-issues the write for its part).
 *
 * The R ranks form servers of ranks_per_server consecutive ranks; the source is rank cfg.src_rank
 * (it must be a member of the domain).  A destination in the source's own server is its own next
 * hop; every other server's next hop is the rank with the source's index inside that server (Section 3.2),
 * which forwards the row to the destinations inside its server.  First level: an ordinary MultiWrite plan over
 * next-hop sets; every hidden row is packed once per group of identical next-hop set and one copy goes to each
 * next hop.  The receive buffer is the relay buffer (Section 6.4: relaying needs no memory of its own): a copy
 * whose next hop is itself a destination of the token lands in its final slot of that rank's receive region;
 * only a copy held by a pure relay (a next hop that is not a destination) is staged in the hop area.  Second
 * level: every relay forwards the copy it holds to the token's other destinations inside its server, at the
 * slots of the flat plan, so the final receive regions are byte-identical to those of mw_dispatch.  Byte
 * accounting is per link class.
 * ------------------------------------------------------------------------------------------------ */
typedef struct mw_relay mw_relay;   /* opaque: two plans (next hops, final destinations) and the second-level descriptors */

typedef struct {
    int64_t hop_rows;               /* rows the source writes: one per (token, distinct next hop)            */
    int64_t delivered_rows;         /* rows in the final receive regions (= total_dest of the flat plan)     */
    int64_t direct_bytes;           /* source -> destinations in its own server (its own rank excluded)      */
    int64_t inter_multiwrite_bytes; /* source -> other servers: one copy per server holding a destination    */
    int64_t inter_unicast_bytes;    /* the same traffic with one copy per remote destination (the baseline)  */
    int64_t forward_bytes;          /* relays -> destinations in their server (the relay itself excluded)    */
    int64_t staged_rows;            /* hop rows whose next hop is not a destination of the token: the only   */
                                    /* copies that need room outside the receive regions                     */
    int32_t status;                 /* MW_OK or the first device-side MW_ERR_* of either plan or the dispatch */
    int32_t reserved;
} mw_relay_totals;

/* cfg as for mw_create, with 0 <= cfg->src_rank < R and R a multiple of ranks_per_server.  Synchronous. */
MW_API int mw_relay_create(mw_relay **out, const mw_config *cfg, int32_t ranks_per_server);
MW_API int mw_relay_destroy(mw_relay *relay);

/* After MW_ERR_TIMEOUT in mw_relay_totals.status: mw_reset for both inner contexts.  Synchronous. */
MW_API int mw_relay_reset(mw_relay *relay);

/* Plans both levels (inputs as for mw_plan; the two plans run concurrently, one of them on a stream the library
 * owns, and `stream` waits for both).  Asynchronous on `stream`. */
MW_API int mw_relay_plan(mw_relay *relay, const int32_t *topk_ids, const int32_t *expert_to_rank, int32_t T, void *stream);

/* Waits for `stream`, then copies the per-link accounting of the latest mw_relay_plan / mw_relay_dispatch. */
MW_API int mw_relay_get_totals(mw_relay *relay, mw_relay_totals *host_out, void *stream);

/*
 * Pack (each row once per group of identical next-hop set) and first-level deliver in one pass, then the relays'
 * forwarding.
 *   send_buf   device, send_capacity_rows rows
 *   hop_buf    device, hop area of hop_capacity_rows rows, laid out per next hop (region of next hop h starts at
 *              the first-level rank offset of h, one row per token that passes through h); only the rows of copies
 *              held by pure relays are written (mw_relay_totals.staged_rows of them), the others are left untouched
 *   recv_base, recv_stride_bytes, recv_capacity_rows   as for mw_deliver
 */
MW_API int mw_relay_dispatch(mw_relay *relay, const void *x, void *send_buf, int64_t send_capacity_rows, void *hop_buf,
                             int64_t hop_capacity_rows, void *recv_base, int64_t recv_stride_bytes,
                             int64_t recv_capacity_rows, void *stream);

/* The two inner contexts (first level: next hops; flat: final destinations), e.g. to read their plan views. */
MW_API int mw_relay_contexts(mw_relay *relay, mw_ctx **hop_ctx, mw_ctx **flat_ctx);

/*
 * Bitmaps and token grouping without any allocation.  (The paper has no counterpart for this
 * entry point; it exists for a class of callers, not for a step of the method.)
 *
 * Some hosts of this library may not allocate device memory themselves: a serving process that
 * hands the whole GPU to its framework's memory pool at start-up leaves nothing for a later
 * cudaMalloc, and a caller on a latency-critical path cannot afford the device-wide
 * synchronisation an allocation or free may imply.  Such callers cannot use mw_create.  This call
 * allocates nothing, neither through CUDA nor through any library: its scratch (the table keyed by
 * bitmap and one slot index per token, 448 KB) is a fixed array inside the library image, present
 * on every GPU that loads the library until the process exits.  The caller passes all inputs and
 * all outputs.
 *
 * It computes, for the current device and on `stream`, the first part of the plan:
 *   token_mask        device, uint64 [T, W], W = ceil(R / 64): destination bitmap (same rules as mw_plan)
 *   token_ndest       device, int32 [T]: |D_t|
 *   token_leader      device, int32 [T]: smallest token index whose bitmap equals this token's
 *                     (the first member of its group), -1 if the bitmap is empty
 *   token_group_size  device, int32 [T]: number of tokens with that bitmap, 0 if empty
 *   status            device, int32 [1]: MW_OK, or MW_ERR_BAD_INDEX if an id or table entry was
 *                     out of range (such slots are ignored)
 * Inputs as for mw_plan: topk_ids device int32 [T, K], expert_to_rank device int32 [E].  With T = 0 only
 * `status` is written and every other pointer may be NULL.
 *
 * Limits and rules
 *   - T <= MW_STATIC_MAX_TOKENS; a larger T returns MW_ERR_CAPACITY and launches nothing.
 *   - The first call on each device looks up the device address of the array (one CUDA runtime
 *     query, no allocation); make that first call before starting any stream capture.  The address
 *     is remembered per device ordinal for the life of the process: it does not survive a
 *     cudaDeviceReset of that device, after which this entry point must not be used again.
 *   - All calls on a device share the one array, which still holds the previous call's contents;
 *     every call therefore begins by emptying the table on `stream`.  Two calls whose GPU work
 *     overlaps (different streams, or different host threads without ordering) race on the array
 *     and give undefined results: order them on one stream or with events.
 *   - Returns MW_ERR_INVALID_ARG for null pointers or sizes out of range, MW_ERR_CUDA if the
 *     runtime fails; asynchronous otherwise.
 */
MW_API int mw_group_tokens_static(const int32_t *topk_ids, const int32_t *expert_to_rank, int32_t T, int32_t K,
                                  int32_t E, int32_t R, uint64_t *token_mask, int32_t *token_ndest,
                                  int32_t *token_leader, int32_t *token_group_size, int32_t *status, void *stream);

/*
 * Convenience for reading plan metadata: waits for `stream`, then copies `bytes` from a device
 * pointer of the plan view (or any device memory of the context's device) into host memory.
 */
MW_API int mw_read_device(mw_ctx *ctx, void *host_dst, const void *device_src, int64_t bytes, void *stream);

/*
 * Test hook for the give-up paths of the bounded device-side waits (nothing faults, traps or hangs: a wait simply
 * runs out).  The bits apply to the next launch that contains the wait and are cleared by it:
 *   MW_TEST_SKEW_LOOKBACK   the next plan's tiles look for predecessor records of an epoch nobody writes
 *   MW_TEST_SKEW_BARRIER    the next fused plan's grid barriers wait for one arrival more than there are blocks
 *   MW_TEST_SKEW_BULK_LOAD  the next launch of the bulk-copy engine announces every load 16 bytes too large, so
 *                           no pipeline stage ever completes
 *   MW_TEST_SKEW_GROUP_MAJOR the next mw_group_major's tiles look for records of another call
 * Use with MW_FLAG_SHORT_WAITS, or each wait takes about a second to give up.  The outcome is MW_ERR_TIMEOUT in
 * mw_totals.status; recover with mw_reset.
 */
#define MW_TEST_SKEW_LOOKBACK  0x1u
#define MW_TEST_SKEW_BARRIER   0x2u
#define MW_TEST_SKEW_BULK_LOAD 0x4u
#define MW_TEST_SKEW_GROUP_MAJOR 0x8u
MW_API int mw_test_skew_waits(mw_ctx *ctx, uint32_t what);

/* Number of kernels this context has launched since mw_create (for launch accounting). */
MW_API int64_t mw_kernel_launches(const mw_ctx *ctx);

/* Static description of an error code. */
MW_API const char *mw_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* MW_H_ */
