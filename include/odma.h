/*
 * odma.h - C ABI of libodma: on-demand contiguous KV-cache allocation (ODMA) and the
 * decode-attention path that streams the resulting slabs on NVIDIA B200 (sm_100a).
 *
 * The allocator follows the paper's design section (Section III): a request's KV cache
 * lives in ONE contiguous slab whose size is the request's length bucket; bucket
 * boundaries are re-derived from a sliding window of realised lengths (Section III-C,
 * Eq. 2); a Large Bucket (safety pool) absorbs high-uncertainty requests and requests that
 * outgrow their slab (Section III-D); reserve/release are the allocator's API (Section
 * III-E).  The GPU kernels are the consumer the contiguous layout exists for (Section
 * III-A: contiguous blocks so that attention streams at peak bandwidth).
 *
 * Conventions
 *  - Every function returns an int32 status (ODMA_OK = 0); nothing throws.
 *  - "dev" pointers are CUDA device pointers, "host" pointers are ordinary host memory.
 *  - The pool's device memory belongs to the caller; the library never allocates or
 *    frees it.  The library owns only small device scratch (split partials, staging for
 *    odma_decode_step_host), allocated in odma_pool_create and freed in
 *    odma_pool_destroy.
 *  - Kernel launchers are asynchronous on the given stream (a cudaStream_t passed as
 *    void*; NULL = the legacy default stream).  All device work of one pool must be
 *    issued on one stream, or be ordered by the caller: a slab released on the host may
 *    be handed out again while an earlier kernel still reads it otherwise.  The decode
 *    kernels are launched with programmatic stream serialization and read queries, new
 *    rows and (after another decode launch of this library) slab rows only once the
 *    kernels ahead of them have completed; a caller that writes pool memory, q, k_new or
 *    v_new with kernels of its own must not let those signal their dependents early
 *    (no programmatic launch trigger before the writes are done).  Decode steps
 *    (odma_decode_step, odma_decode_step_host) issued directly one after the other on
 *    DIFFERENT layers run concurrently: layers share no K/V rows, and the second does not wait
 *    for the first.  The q, k_new, v_new of a step must therefore not be outputs of the decode
 *    step issued directly before it, and their out buffers must not overlap (in a model the
 *    projections between two layers' attention are kernels of the caller: a step issued
 *    behind any other kernel or copy starts only when that operation has completed).
 *  - Host-side calls are not thread-safe; serialise calls on one pool.
 *  - Lengths and capacities are in tokens.  One token occupies
 *    layers * 2 * kv_heads * head_dim * elem_bytes bytes of the pool.
 *
 * Pool layout in device memory
 *    The pool is layers*2 arrays (layer-major, K then V), each of T*kv_heads rows of
 *    head_dim elements (T = pool capacity in tokens).  A slab {base, cap} owns rows
 *    [base*kv_heads, (base+cap)*kv_heads) of every array, head-major inside the slab:
 *        row(head, t) = base*kv_heads + head*cap + t,            0 <= t < cap
 *    so the keys (or values) of one (request, layer, head) are one contiguous run of
 *    len*head_dim*elem_bytes bytes.  Element address of array a = layer*2 + (0:K | 1:V):
 *        dev_base + ((a*T*kv_heads + row) * head_dim + d) * elem_bytes
 */
#ifndef ODMA_H_
#define ODMA_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ODMA_MAX_BUCKETS 8

enum {
    ODMA_OK = 0,
    ODMA_ERR_INVALID = 1,     /* bad argument, shape, alignment or configuration */
    ODMA_ERR_NOMEM = 2,       /* no free run of the needed size (main or safety region) */
    ODMA_ERR_UNKNOWN_REQ = 3, /* request id not live */
    ODMA_ERR_DUP_REQ = 4,     /* request id already live */
    ODMA_ERR_OVERFLOW = 5,    /* length beyond max_len, or beyond the slab on commit */
    ODMA_ERR_CUDA = 6,        /* a CUDA runtime or driver call failed */
    ODMA_ERR_TIMEOUT = 7,     /* a bounded device-side wait ran out (status word) */
    ODMA_ERR_TOO_LARGE = 8    /* odma_decode_attention_static: batch beyond its fixed scratch */
};

/* Element type of the pool's K/V rows.  ODMA_DTYPE_FP8_E4M3: one byte per element in the OCP
 * 8-bit floating-point format E4M3 (no infinities, largest value 448) with one fp32
 * dequantisation scale per layer for K and one for V (odma_set_kv_scales); queries, the rows
 * given to an append and the output are bf16 ("io type": bf16 for BF16 and FP8_E4M3 pools,
 * fp32 for F32 pools).  An 8-bit pool needs head_dim 128 and at most 8 query heads per KV
 * head; its decode runs on the tcgen05 kernel only. */
enum { ODMA_DTYPE_F32 = 0, ODMA_DTYPE_BF16 = 1, ODMA_DTYPE_FP8_E4M3 = 2 };

/* which tensor-core decode kernel a bf16 pool runs (odma_config.decode_kernel) */
enum { ODMA_DECODE_AUTO = 0, ODMA_DECODE_TCGEN05 = 1, ODMA_DECODE_MMA_SYNC = 2 };
enum { ODMA_READOUT_AUTO = 0, ODMA_READOUT_LATE = 1, ODMA_READOUT_AT_ONCE = 2 };

/* kernels that odma_profile_read can report */
enum { ODMA_K_APPEND = 0, ODMA_K_DECODE = 1, ODMA_K_COMBINE = 2, ODMA_K_MIGRATE = 3,
       ODMA_K_PROBE = 4, ODMA_K_COUNT = 5 };

typedef struct odma_pool odma_pool;   /* opaque */
typedef struct odma_paged odma_paged; /* opaque: a page-16 copy of the pool (ablation) */

/* Allocator and scratch configuration.  odma_config_default() fills the values the paper
 * states (Section III-B: gamma = 0.2, tau = 0.8; Section III-C: 4 buckets, 10,000-request
 * window, refresh every 1,000 requests) and this library's choices for what it leaves open. */
typedef struct odma_config {
    int32_t safety_pct;      /* share of the pool given to the Large Bucket, integer percent (10) */
    int32_t max_len;         /* longest KV length of a request; multiple of granule (32768) */
    int32_t granule;         /* G: slab bases and sizes are multiples of G tokens; must be 16 */
    int32_t window;          /* W: realised lengths kept for the quantiles (10000) */
    int32_t refresh;         /* R: boundaries re-derived every R completions (1000) */
    int32_t n_levels;        /* B: number of quantile levels / adaptive buckets (4) */
    int32_t p_num[ODMA_MAX_BUCKETS]; /* quantile levels p_i = p_num[i] / p_den ({1,2,3,4}/4) */
    int32_t p_den;
    int32_t gamma_permille;  /* gamma of L' = L(1 + gamma u), thousandths (200) */
    int32_t tau_permille;    /* tau: u > tau routes to the Large Bucket, thousandths (800) */
    int32_t growth;          /* migration asks for max(need, growth*len) tokens (2) */
    int32_t large_fixed;     /* 1: every Large Bucket slab has max_len tokens (0) */
    int32_t max_batch;       /* most requests per odma_build_tables call; sizes scratch (1024) */
    int32_t max_group;       /* most query heads per KV head; sizes scratch (8) */
    int32_t plan_ctas;       /* persistent CTAs the split plan targets; 0 = one per SM of the
                                current device (148 when the pool has no device memory) */
    int32_t fused_combine;   /* 1: the CTA that delivers the last piece of a split stream merges
                                the pieces inside the decode kernel; 0: a separate combine kernel
                                is launched after it (1) */
    int32_t fused_append;    /* 1: odma_decode_step / odma_decode_step_host let the bf16 decode
                                kernel take the step's new token from k_new / v_new and write
                                it into the slab itself (one launch per layer); 0: they launch
                                the append kernel first (1) */
    int32_t decode_kernel;   /* bf16 decode kernel: ODMA_DECODE_TCGEN05 the tcgen05 / tensor-memory
                                kernel, ODMA_DECODE_MMA_SYNC the mma.sync kernel, ODMA_DECODE_AUTO
                                the first for the layers of an odma_decode_step over several
                                layers and the second for single launches (0) */
    int32_t chain_launches;  /* 1: a decode step issued directly behind a decode step on another layer does
                                not wait for it (see "Conventions"); 0: every launch waits for the kernel
                                ahead of it (1) */
    int32_t span_layers;     /* 1: odma_decode_step over several layers is ONE launch of the tcgen05 kernel
                                when that kernel serves the pool and the split streams' partial results of
                                all layers fit the scratch: the CTAs walk layer after layer over the same
                                plan; 0: one launch per layer (1) */
    int32_t async_recal;     /* 1: a background thread owns the length window: odma_free only logs the
                                realised length, the thread applies the log in order and refreshes the
                                boundaries off the critical path (Sections III-E, IV-C); boundaries at
                                any moment are those of a prefix of the log, after odma_recal_flush
                                those of the whole log.  0: the refresh runs inside odma_free (0) */
    int32_t cluster_observe; /* 1: a completion's length goes only to the outbox read by
                                odma_drain_observations and enters the window through odma_observe
                                (every replica then feeds the same merged sequence and derives the
                                same boundaries: the bucket configuration a cluster manager keeps
                                consistent, Section III-E); 0: it enters the window at once (0) */
    int32_t readout;         /* tcgen05 kernel, 16-bit slabs: ODMA_READOUT_LATE an item's result is read out
                                of tensor memory and stored after the softmax of the first tile of the next
                                item of the same half of the CTA (same results; faster where a CTA works
                                through many short items, slower on few long ones), ODMA_READOUT_AT_ONCE as
                                soon as the item ends, ODMA_READOUT_AUTO late for launches in which a CTA
                                walks three items or more of at most 128 tokens on average (0) */
} odma_config;

typedef struct odma_slab {
    int32_t base_tok;  /* first token of the slab */
    int32_t cap_tok;   /* tokens it can hold */
    int32_t pool_id;   /* 0 main region, 1 Large Bucket */
    int32_t bucket_id; /* index of the boundary it was sized by, -1 in the Large Bucket */
    uint64_t epoch;    /* boundary epoch in force when the call returned */
} odma_slab;

typedef struct odma_stats {
    int64_t total_tokens, safety_tokens, main_tokens; /* T, S, M */
    int64_t live, reserved_live, used_live;           /* live requests, sum cap, sum len */
    int64_t completed, sum_len_completed, sum_cap_completed; /* utilisation = len / cap */
    int64_t migrations, nomem, routed_large;
    int64_t safety_live, safety_peak;                 /* tokens held in the Large Bucket */
    int64_t observed;                                 /* lengths logged so far */
    uint64_t epoch;
} odma_stats;

/* Host-side description of one built batch (plain data, owned by the caller).  The device
 * table it points to holds int32 words:
 *   base[n], cap[n], len[n] (length AFTER this step's append), cu_new[n+1] (prefix sum of
 *   the tokens appended this step), cta[n_ctas][12], items[n_items][8], combine[n_combine][4].
 *   cta     = {item_begin, item_end, 0, 0, copy of items[item_begin]}: CTA c works through
 *             items [item_begin, item_end), pieces of split streams first
 *   item    = {request, kv_head, first_token, n_tokens, flags (bit 0: the piece is the whole
 *              stream, written out directly; bit 1: the piece ends its stream), slot,
 *              first row of the piece inside one K/V array, combine record (-1 if direct)};
 *             slots number the pieces in plan order (longest streams first; the pieces of one
 *             cut stream are consecutive, in token order)
 *   combine = {request, kv_head, first_slot, n_slots}
 * The off_* fields are word offsets of those arrays inside d_table. */
typedef struct odma_tables {
    void* d_table;
    int32_t n, n_new_total, n_items, n_ctas, n_combine, words;
    int32_t off_base, off_cap, off_len, off_cu_new, off_cta, off_items, off_combine;
    int32_t tile_tokens;
    int32_t one_new_each; /* 1 when every request appends exactly one token (decode step) */
    int32_t reserved;
    int64_t kv_tokens; /* sum of len */
    uint64_t epoch;
} odma_tables;

void odma_config_default(odma_config* cfg);
const char* odma_strerror(int32_t code);

/* ---- pool (problem statement: one KV-cache pool carved into contiguous per-request slabs;
 *      Section I-C, Section III-A) --------------------------------------------------------
 * dev_base: device pointer to `bytes` bytes, 256-byte aligned, or NULL for a bookkeeping-only
 * pool (allocator calls work, every device call returns ODMA_ERR_INVALID).  T =
 * floor_G(bytes / token_bytes) tokens, the last floor_G(T*safety_pct/100) of them are the
 * Large Bucket.  head_dim*elem_bytes must be a multiple of 16.  cfg NULL = defaults.
 * Until odma_set_buckets or the first recalibration there is one bucket of max_len tokens.
 * With device memory the call allocates the library's scratch (cudaMalloc) and must run
 * with the pool's device current. */
int32_t odma_pool_create(void* dev_base, uint64_t bytes, int32_t layers, int32_t kv_heads,
                         int32_t head_dim, int32_t dtype, const odma_config* cfg, odma_pool** out);
int32_t odma_pool_destroy(odma_pool* pool);

/* ---- boundary refresh off the critical path and across replicas (Sections III-E, IV-C) ------
 * odma_recal_flush: returns once the background thread (async_recal) has applied every length
 * logged so far; a no-op otherwise.
 * odma_drain_observations: copies to `out` (host, room for `cap` values) the lengths of the
 * requests completed on this pool since the last drain, oldest first (at most `window` are
 * kept), and forgets them; *n = how many.
 * odma_observe: feeds `n` realised lengths (host; 0 <= length <= max_len) into the window as if
 * they had completed here, in the given order; every `refresh`-th observation re-derives the
 * boundaries (Eq. 2).  Replicas that exchange their drained lengths and observe the
 * concatenation in rank order hold identical windows and so identical boundaries. */
int32_t odma_recal_flush(odma_pool* pool);
int32_t odma_drain_observations(odma_pool* pool, int32_t* out, int32_t cap, int32_t* n);
int32_t odma_observe(odma_pool* pool, const int32_t* lengths, int32_t n);

/* Dequantisation scales of an ODMA_DTYPE_FP8_E4M3 pool (the 8-bit variant of the slab layout;
 * the paper's slabs hold the serving stack's 16-bit cache, Section IV-A): k_scale, v_scale:
 * host, [layers] fp32, finite and > 0.  A stored code c of layer l stands for value(c) *
 * scale[l]; an append stores the code nearest (ties to even, saturating at +-448) to
 * fp32(x) * (1.0f / scale[l]), product and reciprocal taken in fp32.  Default 1 for every
 * layer.  Takes effect for launches issued after the call; rows already stored keep their
 * codes.  ODMA_ERR_INVALID for another pool type or a bad scale. */
int32_t odma_set_kv_scales(odma_pool* pool, const float* k_scale, const float* v_scale);

/* ---- bucket boundaries (Section III-C, Eq. 2) ------------------------------------------
 * Static / initial boundaries: n in [1, ODMA_MAX_BUCKETS], strictly increasing multiples of
 * the granule, none above max_len.  They hold until the next recalibration. */
int32_t odma_set_buckets(odma_pool* pool, const int32_t* boundaries, int32_t n);
/* boundaries: host array of ODMA_MAX_BUCKETS entries; *n and *epoch receive count and epoch. */
int32_t odma_get_buckets(const odma_pool* pool, int32_t* boundaries, int32_t* n, uint64_t* epoch);

/* ---- reserve (Section III-E; bucket choice Section III-C; tail Section III-D) -----------
 * predicted_len is the predicted TOTAL length (prompt + generation).  The slab has the size
 * of the first boundary >= predicted_len and sits at the lowest free address of the main
 * region; a length beyond the last boundary is served from the Large Bucket with
 * ceil_G(predicted_len) tokens.  ODMA_ERR_NOMEM when nothing fits (ordinary requests never
 * spill into the Large Bucket), ODMA_ERR_DUP_REQ for a live id. */
int32_t odma_alloc(odma_pool* pool, uint64_t req, int32_t predicted_len, odma_slab* out);
/* Section III-B: inflate L' = ceil(L_hat * (1 + gamma*u)) and, when u > tau, take the slab
 * straight from the Large Bucket.  u_permille in [0, 1000]. */
int32_t odma_alloc_uncertain(odma_pool* pool, uint64_t req, int32_t l_hat, int32_t u_permille,
                             odma_slab* out);
/* Sections III-D and IV-C, reactive migration: if needed_len exceeds the slab, reserve a
 * Large Bucket slab of max(needed_len, growth*len) tokens (capped at max_len), launch the
 * copy of the request's len tokens (all layers, K and V) on `stream`, then release the old
 * slab.  *migrated = 1 when that happened.  ODMA_ERR_OVERFLOW beyond max_len;
 * ODMA_ERR_NOMEM leaves the old slab in place. */
int32_t odma_ensure_capacity(odma_pool* pool, uint64_t req, int32_t needed_len, void* stream,
                             odma_slab* out, int32_t* migrated);
/* release (Section III-E) and logging of the realised length (Section III-A): frees the
 * slab, pushes the request's length into the window and, on every R-th completion,
 * re-derives the boundaries.  New boundaries apply to later odma_alloc calls only
 * (Section IV-C). */
int32_t odma_free(odma_pool* pool, uint64_t req);

/* Host mirror of the lengths: after a step's kernels have been issued, add n_new[i] (NULL =
 * 1 each) tokens to each request's length.  ODMA_ERR_OVERFLOW if one would pass its slab
 * (nothing is changed then). */
int32_t odma_commit_step(odma_pool* pool, const uint64_t* reqs, int32_t n, const int32_t* n_new);
int32_t odma_get_slab(const odma_pool* pool, uint64_t req, odma_slab* out, int32_t* len);
int32_t odma_get_stats(const odma_pool* pool, odma_stats* out);

/* ---- per-step tables -------------------------------------------------------------------
 * Slab table, lengths and the split plan for a batch of n live requests, each about to
 * append n_new[i] tokens (NULL = 1 each; 0 allowed).  Every request must already have room
 * (odma_ensure_capacity).  The plan deals the batch's KV streams (one per request and KV
 * head, read in 64-token tiles) to the persistent CTAs in shares of equal cost: streams longer
 * than a share are cut into pieces, all others go whole, longest first, to the least loaded share.
 * odma_plan_host writes the table to host memory (no CUDA call); odma_build_tables writes
 * it to the caller's device buffer d_table with one asynchronous copy.  table_bytes must be
 * at least odma_tables_bytes(pool, n). */
uint64_t odma_tables_bytes(const odma_pool* pool, int32_t n);
int32_t odma_plan_host(odma_pool* pool, const uint64_t* reqs, const int32_t* n_new, int32_t n,
                       int32_t* host_table, uint64_t table_bytes, odma_tables* out);
int32_t odma_build_tables(odma_pool* pool, const uint64_t* reqs, const int32_t* n_new, int32_t n,
                          void* d_table, uint64_t table_bytes, void* stream, odma_tables* out);

/* ---- chunked prefill over the slabs (Section II-A: the prefill phase fills the cache with the
 *      prompt's keys and values before decoding starts) --------------------------------------
 * A chunk of n_new[i] >= 1 prompt tokens per request is appended with the ordinary calls
 * (odma_build_tables with n_new, odma_append_kv); its causal attention is then the decode
 * attention of one stream PER NEW TOKEN over the owner's slab: token j of request i attends
 * keys [0, len[i] + j] (len[i] = the committed length, the chunk not yet committed).  This
 * call plans those sum(n_new) streams (at most max_batch of them; ODMA_ERR_INVALID beyond)
 * and writes their table to d_table (device, table_bytes >= odma_tables_bytes(pool,
 * sum(n_new))); odma_decode_attention with the returned descriptor, q and out of shape
 * [sum(n_new), q_heads, head_dim] (tokens in request order, then position order), computes
 *   out[t][h] = softmax_{k <= pos(t)}(q[t][h] . K[h div g][k] / sqrt(head_dim)) V[h div g].
 * The descriptor appends nothing (n_new_total = 0).  A slab is read once per new token, from
 * L2 after the first; packing several tokens of a chunk into one tensor-core tile is not done. */
int32_t odma_build_prefill_tables(odma_pool* pool, const uint64_t* reqs, const int32_t* n_new, int32_t n,
                                  void* d_table, uint64_t table_bytes, void* stream, odma_tables* out);

/* ---- KV append (the per-step growth of each request's cache, Section II-A) --------------
 * Writes the step's new K and V rows of `layer` behind each request's existing tokens:
 * token j of request i goes to slab position len[i] - n_new[i] + j.  k_new, v_new: device,
 * [n_new_total, kv_heads, head_dim] in the pool's io type, requests in table order, 16-byte
 * aligned.  An 8-bit pool quantises the rows as odma_set_kv_scales describes. */
int32_t odma_append_kv(odma_pool* pool, int32_t layer, const odma_tables* tables,
                       const void* k_new, const void* v_new, void* stream);

/* ---- decode attention over the slabs (the bandwidth consumer, Sections III-A and V-B) ---
 * out[i][h] = softmax_j(q[i][h] . K_i[h div g][j] / sqrt(head_dim)) V_i[h div g], j < len[i],
 * g = q_heads / kv_heads (K_i, V_i of an 8-bit pool: the dequantised values).  q, out: device,
 * [n, q_heads, head_dim] in the pool's io type, 16-byte aligned; lse: device fp32 [n, q_heads] or NULL (natural-log sum of exp of the scaled
 * scores).  Accumulation and softmax are fp32.  Launches the split kernel and, when some
 * stream was split, the combine kernel. */
int32_t odma_decode_attention(odma_pool* pool, int32_t layer, const void* q, int32_t q_heads,
                              const odma_tables* tables, void* out, float* lse, void* stream);

/* One decode step of one layer from HOST buffers: builds the tables for reqs (one new token
 * each), takes h_q [n,q_heads,head_dim], h_k_new, h_v_new [n,kv_heads,head_dim], appends,
 * attends and leaves the result in h_out [n,q_heads,head_dim]; asynchronous on `stream`
 * (h_out is complete once the stream has been synchronised).  When all four buffers are
 * page-locked (cudaHostAlloc, cudaHostRegister, a framework's pinned tensors) and 16-byte
 * aligned, the kernel reads and writes them in place over the bus: the step is one launch and
 * no copy.  Otherwise the inputs are staged through the pool's device scratch (three
 * host-to-device copies) and the result is copied back.  Does not commit lengths. */
int32_t odma_decode_step_host(odma_pool* pool, int32_t layer, int32_t q_heads, const uint64_t* reqs,
                              int32_t n, const void* h_q, const void* h_k_new, const void* h_v_new,
                              void* h_out, void* stream);

/* The same step from DEVICE buffers, for n_layers consecutive layers starting at `layer`:
 * builds the tables once into the pool's own table buffer, then for each layer appends one
 * token per request and attends, all asynchronous on `stream`.  Buffers are layer-major:
 * d_q, d_out [n_layers, n, q_heads, head_dim]; d_k_new, d_v_new [n_layers, n, kv_heads,
 * head_dim]; lse device fp32 [n_layers, n, q_heads] or NULL.  tables_out (host, nullable)
 * receives the description of the built batch; its d_table stays valid until the next
 * odma_decode_step / odma_decode_step_host on this pool.  Does not commit lengths.
 * On a bf16 pool with fused_append the decode kernel appends the token itself (one launch per
 * layer, no append kernel).  Consecutive steps of the same batch (same requests, no slab
 * moved, grown by at most 32 tokens per request since the last full plan) reuse that plan: a
 * stream's last piece takes the growth, and for batches of up to 256 requests the lengths
 * travel with the kernel's arguments, so such a step copies no table; the length words of
 * d_table in device memory are then those of the last full plan. */
int32_t odma_decode_step(odma_pool* pool, int32_t layer, int32_t n_layers, int32_t q_heads,
                         const uint64_t* reqs, int32_t n, const void* d_q, const void* d_k_new,
                         const void* d_v_new, void* d_out, float* lse, void* stream,
                         odma_tables* tables_out);

/* ---- decode attention that allocates nothing (the paper has no counterpart: this entry point
 *      exists for how the library is deployed, not for the method) ------------------------
 * For callers that cannot allocate device memory when they reach this call: a serving
 * process whose memory manager has already claimed the whole GPU, a plug-in that runs under
 * a host framework which owns every allocation, code on a path where cudaMalloc (which
 * synchronises the device) is forbidden.  The result is the one odma_decode_attention
 * gives, but the partial results of split streams are kept in ONE fixed array of device
 * memory that is part of the library image (about 2.1 MB on every GPU that loads the
 * library, until the process exits) rather than in scratch allocated by odma_pool_create,
 * and the call itself performs no cudaMalloc, cudaFree or other allocating call.
 *   pool      any pool handle; it supplies the geometry only (layers, kv_heads, head_dim,
 *             dtype, capacity T).  A pool created with dev_base = NULL (its creation makes
 *             no CUDA call) is enough; plan the batch with odma_plan_host and copy the
 *             table words into device memory of your own.
 *   dev_base  device, 256-byte aligned: the KV memory, laid out as described at the top.
 *   tables    the descriptor odma_plan_host filled, with d_table set to your device copy
 *             of the table (16-byte aligned).
 *   q, out, lse, stream: as for odma_decode_attention.
 * Limits: at most 512 items in the plan (tables->n_items), at most 8 query heads per KV head,
 * head_dim 32, 64 or 128; beyond them the call returns ODMA_ERR_TOO_LARGE and launches
 * nothing.  It runs the plain-ALU decode kernel and the combine kernel for every dtype.
 * The first call on a device looks up the array's device address (a CUDA runtime query, no
 * allocation): make that first call before any stream capture, with the device current.
 * Every call on a GPU uses the same array and leaves its partial results there; a call
 * reads only slots it has written itself, so nothing needs clearing, but two calls whose
 * kernels overlap on the GPU (different streams, no ordering) race on it. */
int32_t odma_decode_attention_static(const odma_pool* pool, const void* dev_base, int32_t layer,
                                     const void* q, int32_t q_heads, const odma_tables* tables,
                                     void* out, float* lse, void* stream);

/* Synchronises `stream` and returns the device status word as an error code (ODMA_OK,
 * ODMA_ERR_TIMEOUT, or ODMA_ERR_CUDA for a failed stream), clearing it. */
int32_t odma_check_status(odma_pool* pool, void* stream);

/* Failure detection, exercised without a fault: launches a one-thread kernel whose only wait
 * can never be satisfied and gives up after limit_ms (1..1000); odma_check_status then returns
 * ODMA_ERR_TIMEOUT and the context stays usable.  Every wait of the decode kernels is bounded
 * the same way. */
int32_t odma_selftest_timeout(odma_pool* pool, int32_t limit_ms, void* stream);

/* ---- measurement aids -------------------------------------------------------------------
 * Streams exactly the bytes odma_decode_attention would read for `layer`, through the same
 * staging pipeline, and does no arithmetic: the ceiling for this access pattern. */
int32_t odma_read_probe(odma_pool* pool, int32_t layer, int32_t q_heads, const odma_tables* tables,
                        void* stream);
/* Per-kernel device time: while enabled every launch is bracketed by CUDA events on its
 * stream.  odma_profile_read synchronises and returns the summed milliseconds and the
 * number of launches of one kernel since profiling was enabled. */
int32_t odma_profile_enable(odma_pool* pool, int32_t on);
int32_t odma_profile_read(odma_pool* pool, int32_t kernel, double* total_ms, int64_t* launches);

/* ---- admission / serving simulator (the paper's evaluation protocol, Section V: Poisson
 *      arrivals into one KV pool; KV-cache utilisation = actual / reserved; throughput in
 *      output tokens per second) ----------------------------------------------------------------
 * Host only.  One model replica decodes in lock step over the pool; `reqs` (host, n entries,
 * arrival times non-decreasing) are admitted first come first served under one of three
 * reservation policies: ODMA_SIM_STATIC reserves max_len tokens per request (the static
 * worst-case baseline), ODMA_SIM_PAGED16 takes 16-token pages on demand (PagedAttention
 * accounting), ODMA_SIM_ODMA drives this pool's own allocator (odma_alloc, or
 * odma_alloc_uncertain when u_permille >= 0; odma_ensure_capacity with allocate-and-copy
 * migration; odma_free with boundary recalibration).  `pool` must be a pool without live
 * requests; a bookkeeping-only pool (dev_base NULL) is enough, no kernel is launched.
 * Rules: time in integer nanoseconds; the prompt is in place at admission; a decode step lasts
 * layers * (base_ns + kv_tokens * ps_per_token / 1000) with kv_tokens the keys attended by the
 * requests that generate in that step (fit base_ns and ps_per_token to measured launches);
 * admission stops at the first request that does not fit, at max_batch live requests, or at
 * one that has not arrived (with nobody live the clock jumps to the next arrival); a request
 * without room for its next token stalls for the step; when all stall, the youngest is
 * preempted (progress lost, back to the head of the queue) and nothing is admitted until a
 * live request completes; a request that cannot be placed in an empty pool, or stalls alone,
 * is dropped (failed).  Results are sums; utilisation = sum_actual / sum_reserved (capacity
 * held at completion), time-averaged utilisation = used_time / reserved_time, mean
 * concurrency = conc_time / makespan_ns, tokens per second = tokens_out / makespan_ns * 1e9. */
enum { ODMA_SIM_STATIC = 0, ODMA_SIM_PAGED16 = 1, ODMA_SIM_ODMA = 2 };
typedef struct odma_sim_request {
    int64_t arrival_ns;
    int32_t prompt;      /* KV tokens present at admission (>= 1) */
    int32_t total;       /* KV tokens at completion (> prompt) */
    int32_t predicted;   /* predicted total, as given to the allocator */
    int32_t u_permille;  /* predictor uncertainty in thousandths, -1: none */
} odma_sim_request;
typedef struct odma_sim_params {
    int32_t policy, max_batch, layers, reserved;
    int64_t base_ns, ps_per_token;
} odma_sim_params;
typedef struct odma_sim_result {
    int64_t completed, failed, tokens_out, tokens_lost, steps, makespan_ns, sum_actual, sum_reserved,
        conc_time, reserved_time, used_time, migrations, preemptions, stalls, deferred;
} odma_sim_result;
int32_t odma_sim_run(odma_pool* pool, const odma_sim_params* params, const odma_sim_request* reqs,
                     int32_t n, odma_sim_result* out);

/* ---- page-16 ablation (paging is the layout the paper argues against, Sections I, II-A) --
 * The same requests re-laid in 16-token pages: page p of (array a, head) is 16 rows at
 * ((a*n_pages + p)*kv_heads + head)*16 of the caller's buffer d_pages.  odma_paged_build
 * assigns ceil(len/16) pages to each request of `tables` (consecutive ids when shuffle_seed
 * is 0, a seeded permutation of all pages otherwise), writes the page table
 * [n][max_pages] to d_page_table and copies the slab contents of every layer into the
 * pages.  odma_decode_attention_paged is odma_decode_attention reading through it. */
int32_t odma_paged_create(odma_pool* pool, void* d_pages, uint64_t bytes, odma_paged** out);
int32_t odma_paged_destroy(odma_paged* paged);
int32_t odma_paged_build(odma_paged* paged, const odma_tables* tables, const int32_t* host_len,
                         uint64_t shuffle_seed, int32_t* d_page_table, int32_t max_pages,
                         void* stream);
int32_t odma_decode_attention_paged(odma_paged* paged, int32_t layer, const void* q,
                                    int32_t q_heads, const odma_tables* tables,
                                    const int32_t* d_page_table, int32_t max_pages, void* out,
                                    float* lse, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* ODMA_H_ */
