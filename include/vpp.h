/*
 * vpp.h -- C ABI of the B200 chunked-prefill attention library.
 *
 * The operation is the attention step inside a chunked prefill (the paper's
 * Eq. 1 with the causal rule of its Transformer background section, applied
 * per chunk as described in its "Chunked Prefill Pipeline Parallelism"
 * section): a packed chunk of query rows attends causally to itself and to
 * the whole prefix already held in a (paged) KV cache.  For request r with
 * prefix_len P and chunk_len C, query row i (0 <= i < C) of q-head h sits at
 * absolute position p = P + i and sees cached keys 0..p (inclusive) of
 * kv-head h / (num_q_heads / num_kv_heads):
 *
 *     s_j = softmax_scale * <q, k_j>,  out = sum_j softmax(s)_j * v_j,
 *     lse = ln sum_j exp(s_j)
 *
 * The cost of one chunk grows linearly with its prefix length: this is the
 * per-chunk imbalance the paper's V-shaped virtual-stage layout is built
 * around (its Eq. 2-3).
 *
 * General rules
 *  - Every pointer is a DEVICE pointer unless its comment says "host".
 *  - The caller owns every buffer; the library allocates no device memory
 *    in the entry points declared here.
 *  - All work is enqueued on `stream`; no entry point synchronises.
 *  - Entry points return VPP_OK or a negative vpp_status; vpp_last_error()
 *    gives a thread-local message for the most recent failure.
 *  - There is no CPU fallback: unsupported shapes return VPP_ERR_UNSUPPORTED.
 */
#ifndef VPP_H_
#define VPP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    VPP_OK = 0,
    VPP_ERR_INVALID_ARG = -1, /* null pointer, negative size, bad stride or alignment */
    VPP_ERR_UNSUPPORTED = -2, /* head dims / block size this build has no kernel for   */
    VPP_ERR_WORKSPACE = -3,   /* workspace missing or smaller than the size query      */
    VPP_ERR_CUDA = -4,        /* a CUDA runtime / driver call failed                   */
    VPP_ERR_TIMEOUT = -5      /* never returned by an entry point (none synchronises): the code a caller should
                                 map a device status of VPP_DEV_TIMEOUT to once it has read *status          */
} vpp_status;

/* Values the device writes to *status (0 = success). */
enum {
    VPP_DEV_OK = 0,
    VPP_DEV_BAD_LENGTHS = 1,  /* prefix_len/chunk_len negative, beyond max_seq_len, or sum != total_q */
    VPP_DEV_BAD_BLOCK = 2,    /* a block_table entry that is needed lies outside [0, num_blocks)       */
    VPP_DEV_TIMEOUT = 3       /* a bounded wait inside a kernel expired; outputs are undefined         */
};

typedef void *vpp_stream_t; /* a cudaStream_t */

/*
 * Arguments of vpp_chunk_attn_fwd.
 *
 * q            bf16 [total_q, num_q_heads, head_dim_qk], dense, packed request-major: the rows of
 *              request r start at sum_{r' < r} chunk_len[r'].  16-byte aligned.
 * k_cache      bf16; element (block b, slot t, kv-head g, feature d) lives at
 *              b*k_block_stride + t*k_token_stride + g*k_head_stride + d   (strides in ELEMENTS,
 *              feature stride 1; each stride a multiple of 8 elements; base 16-byte aligned).
 *              The usual layout [num_blocks, block_size, Hkv, Dqk] has strides
 *              (block_size*Hkv*Dqk, Hkv*Dqk, Dqk).
 * v_cache      same addressing with the v_* strides and head_dim_v features.  It may alias k_cache
 *              (absorbed MLA: V is the first head_dim_v features of each K row).
 *              The cache must ALREADY hold positions [0, prefix_len+chunk_len) of every request:
 *              the chunk's own K/V are written before this call.  Slots past that point inside a
 *              request's last block may hold anything (NaN included) and blocks the block table
 *              does not name are never read.
 * block_table  int32 [num_reqs, max_blocks_per_req]: physical block of logical block j of request r.
 *              NULL means contiguous: request r is "block" r and block_size is ignored (slot = token).
 *              Then EVERY request's region must really hold max_seq_len slots (the kernels fetch whole
 *              128-key tiles up to max_seq_len, so a loose bound would read past a shorter buffer):
 *              k_block_stride >= max_seq_len * k_token_stride (the same for v), the last region
 *              allocated in full.  With several requests the call checks the strides and returns
 *              VPP_ERR_INVALID_ARG otherwise; the size of the allocation itself cannot be checked.
 * prefix_len   int32 [num_reqs], tokens of the request already cached before this chunk.
 * chunk_len    int32 [num_reqs], query rows of the request in this call (0 allowed).
 * total_q      host copy of sum(chunk_len); sizes out, lse and the workspace.
 * max_seq_len  host upper bound on prefix_len[r] + chunk_len[r]; for a contiguous cache also the
 *              number of slots of each request's region (see block_table).
 * num_kv_splits  0: the library decides; 1: never split the key range; S > 1: split the key range of
 *              every query tile into up to S parts and merge them (split-KV).
 * out          bf16 [total_q, num_q_heads, head_dim_v], 16-byte aligned.
 * lse          fp32 [total_q, num_q_heads], natural log of sum_j exp(softmax_scale * <q,k_j>) over
 *              the visible keys; may be NULL.
 * workspace    at least vpp_chunk_attn_workspace_size(args) bytes, 256-byte aligned.  Contents need
 *              no initialisation and are clobbered.  Two calls that overlap on the GPU need two
 *              workspaces.
 * status       optional device int32.  Zeroed by the call; a nonzero VPP_DEV_* value afterwards
 *              means a device-side check failed and out/lse must not be used.
 *
 * Supported shapes: (head_dim_qk, head_dim_v) = (128, 128) with num_q_heads % num_kv_heads == 0, and
 * (576, 512) with num_kv_heads == 1; block_size a power of two >= 16 (or block_table == NULL).
 */
typedef struct {
    const void *q;
    const void *k_cache;
    const void *v_cache;
    int64_t k_block_stride, k_token_stride, k_head_stride;
    int64_t v_block_stride, v_token_stride, v_head_stride;
    const int32_t *block_table;
    const int32_t *prefix_len;
    const int32_t *chunk_len;
    int32_t num_reqs;
    int32_t max_blocks_per_req;
    int32_t block_size;
    int32_t num_blocks;
    int32_t total_q;
    int32_t max_seq_len;
    int32_t num_q_heads;
    int32_t num_kv_heads;
    int32_t head_dim_qk;
    int32_t head_dim_v;
    float softmax_scale;
    int32_t num_kv_splits;
    void *out;
    float *lse;
    void *workspace;
    size_t workspace_bytes;
    int32_t *status;
} vpp_chunk_attn_args;

/*
 * Bytes of workspace vpp_chunk_attn_fwd needs for these arguments (only the host-side scalar
 * fields are read).  Pure host arithmetic apart from one cached device-attribute query.
 * Returns 0 if the arguments are invalid.
 */
size_t vpp_chunk_attn_workspace_size(const vpp_chunk_attn_args *args);

/*
 * Chunked-prefill attention forward (the operation defined at the top of this file).
 * Enqueues: a work-decomposition kernel (query tiles x heads x key-range splits, ordered by
 * decreasing cost), the persistent attention kernel, and, when the key range was split, the
 * merge kernel.  Returns after enqueueing.
 * Errors: VPP_ERR_INVALID_ARG / VPP_ERR_UNSUPPORTED / VPP_ERR_WORKSPACE before anything is
 * enqueued; VPP_ERR_CUDA if a launch fails.
 */
vpp_status vpp_chunk_attn_fwd(const vpp_chunk_attn_args *args, vpp_stream_t stream);

/*
 * Merge of partial attention results computed over disjoint key sets (split-KV, or the
 * per-device partials of a context-parallel prefix):
 *     lse = ln sum_s exp(lse_s),   out = sum_s exp(lse_s - lse) * o_s
 * where each o_s is already normalised by its own split.  A split with lse_s = -inf contributes
 * nothing; a row whose splits are all -inf gets out = 0, lse = -inf.
 *
 * o_parts    fp32 [num_splits, total_q, num_q_heads, head_dim_v]
 * lse_parts  fp32 [num_splits, total_q, num_q_heads]
 * out        bf16 [total_q, num_q_heads, head_dim_v]
 * lse        fp32 [total_q, num_q_heads] or NULL
 * head_dim_v must be a multiple of 8, num_splits at most 64; pointers 16-byte aligned.
 */
vpp_status vpp_lse_merge(const float *o_parts, const float *lse_parts, int32_t num_splits,
                         int32_t total_q, int32_t num_q_heads, int32_t head_dim_v, void *out,
                         float *lse, vpp_stream_t stream);

/*
 * Chunked-prefill attention over a RANGE of the cached keys, giving partial results -- the building block
 * of a context-parallel prefix (the paper's background on context parallelism: the prefix KV cache is
 * sharded along the sequence): each shard holder evaluates Eq. 1 over its own keys, the partials of all
 * shards are gathered and vpp_lse_merge combines them.
 *
 * Same arguments as vpp_chunk_attn_fwd except that every query row only sees the keys at positions
 * [kv_begin, kv_end) of its request (still subject to the causal rule), and that the results are written
 * un-merged, in the layout vpp_lse_merge reads:
 *   o_part    fp32 [total_q, num_q_heads, head_dim_v]: softmax-weighted values over the keys seen (normalised
 *             within the range);  lse_part  fp32 [total_q, num_q_heads]: log-sum-exp over the keys seen.
 * Stacking the o_part / lse_part of S ranges that tile [0, prefix_len + chunk_len) along a leading dimension
 * gives vpp_lse_merge's o_parts / lse_parts, and its result equals vpp_chunk_attn_fwd's.
 * args->out, args->lse and args->num_kv_splits are ignored; the workspace is still needed (size query with
 * num_kv_splits = 1).  kv_begin must be a multiple of 128 and at most prefix_len[r] for every request with
 * query rows (so that each row sees at least one key: otherwise VPP_DEV_BAD_LENGTHS, nothing written); kv_end
 * must be a multiple of 128 or >= max_seq_len ("to the end").  Errors as vpp_chunk_attn_fwd.
 */
vpp_status vpp_chunk_attn_partial_fwd(const vpp_chunk_attn_args *args, int32_t kv_begin, int32_t kv_end,
                                      float *o_part, float *lse_part, vpp_stream_t stream);

/*
 * Same operation as vpp_chunk_attn_fwd, for callers that cannot obtain device memory themselves.
 * (The paper has no counterpart for this entry point: it is a packaging variant, not a method step.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a plugin called inside a framework's
 * captured or memory-planned region, a serving process whose device memory was handed out in full at
 * start-up, a host thread that must not take the allocator's lock.  Such a caller still passes every
 * input and output buffer; what it cannot supply is the workspace.  Here the workspace is a fixed
 * array of VPP_STATIC_SCRATCH_BYTES inside the library, so `args->workspace` and
 * `args->workspace_bytes` are ignored.
 *
 *  - The call allocates nothing: no cudaMalloc / cudaFree and no allocating library routine.
 *  - Every device that loads the library holds the array (VPP_STATIC_SCRATCH_BYTES) until the
 *    process exits.
 *  - The first call on each device looks up the array's device address (a one-time set-up that is
 *    not a stream operation); make that first call before starting any stream capture.  That look-up
 *    may also be the moment the CUDA runtime loads this part of the library onto the device and
 *    reserves the array, so make it at start-up, while device memory is still available: in a process
 *    that has already handed out all device memory it can fail (VPP_ERR_CUDA, "out of memory").
 *  - With num_kv_splits = 0 the library's own split choice is dropped (the launch runs unsplit) when its partials do
 *    not fit the array.
 *  - A launch whose vpp_chunk_attn_workspace_size exceeds VPP_STATIC_SCRATCH_BYTES is refused
 *    with VPP_ERR_WORKSPACE and nothing is enqueued; vpp_static_last_error() says how much was needed.
 *    (Split-KV partials dominate: 4 * num_kv_splits * total_q * num_q_heads * (head_dim_v + 1) bytes.)
 *  - All calls on a device share the one array, and it keeps whatever the previous call left there.
 *    Nothing in it has to start at zero -- the work-decomposition kernel rewrites the header, the work
 *    list and the per-row split counts of each launch before they are read -- but two calls that
 *    overlap on the GPU (different streams, or graphs replayed concurrently) race on it.  Serialise them.
 *  - Other errors and the meaning of *status are those of vpp_chunk_attn_fwd.
 */
#define VPP_STATIC_SCRATCH_BYTES (32u << 20)
vpp_status vpp_chunk_attn_fwd_static(const vpp_chunk_attn_args *args, vpp_stream_t stream);

/* Size of the built-in scratch array (VPP_STATIC_SCRATCH_BYTES of the library that was loaded). */
size_t vpp_static_scratch_bytes(void);

/* Thread-local detail of the last failure of vpp_chunk_attn_fwd_static on this host thread. */
const char *vpp_static_last_error(void);

/*
 * Paged KV-cache append: the step before vpp_chunk_attn_fwd in a chunked prefill (the paper's
 * "Chunked Prefill Pipeline Parallelism" section: every chunk's keys and values join the cache that
 * the later chunks attend to).  Row i of request r (0 <= i < chunk_len[r]) is written to position
 * prefix_len[r] + i of that request: block block_table[r][pos / block_size], slot pos % block_size
 * (block_table NULL: request r is block r and slot = pos).  Pure data movement, bit-exact.
 *
 * k_new        bf16 [total_q, num_kv_heads, head_dim_qk], dense, packed request-major like q. 16-byte aligned.
 * v_new        bf16 [total_q, num_kv_heads, head_dim_v], or NULL when the values are the leading features of
 *              the keys (v_cache aliases k_cache: absorbed MLA) -- then only the keys are written.
 * k_cache, v_cache, strides, block_table, prefix_len, chunk_len, num_reqs, max_blocks_per_req, block_size,
 * num_blocks, total_q: as in vpp_chunk_attn_args (the caches are written here, not read).  For a contiguous
 *              cache (block_table NULL) max_seq_len is the number of positions each request's region holds.
 * status       optional device int32, zeroed by the call.  VPP_DEV_BAD_LENGTHS: a negative length, a request
 *              that would outgrow its pages, or sum(chunk_len) != total_q -- nothing is written.
 *              VPP_DEV_BAD_BLOCK: a needed block_table entry outside [0, num_blocks) -- that row is skipped.
 * head dims must be multiples of 8 elements, num_reqs at most 8192.  Rows of one call never overlap, so the
 * result does not depend on scheduling.  Returns after enqueueing one kernel on `stream`.
 */
typedef struct {
    const void *k_new;
    const void *v_new;
    void *k_cache;
    void *v_cache;
    int64_t k_block_stride, k_token_stride, k_head_stride;
    int64_t v_block_stride, v_token_stride, v_head_stride;
    const int32_t *block_table;
    const int32_t *prefix_len;
    const int32_t *chunk_len;
    int32_t num_reqs;
    int32_t max_blocks_per_req;
    int32_t block_size;
    int32_t num_blocks;
    int32_t total_q;
    int32_t max_seq_len;
    int32_t num_kv_heads;
    int32_t head_dim_qk;
    int32_t head_dim_v;
    int32_t *status;
} vpp_kv_append_args;

vpp_status vpp_kv_append(const vpp_kv_append_args *args, vpp_stream_t stream);

/*
 * One chunk of one request with its query, its new keys/values and its results in HOST memory: the whole per-chunk
 * step of a chunked prefill (the paper's "Chunked Prefill Pipeline Parallelism" section: append the chunk's K/V to
 * the cache, then Eq. 1 over prefix + chunk) as a single call that also moves the data.  The chunk's rows are cut
 * into slices; slice i's rows go host -> device on a copy stream of the library, are appended (vpp_kv_append) and
 * attended (vpp_chunk_attn_fwd, prefix = prefix_len + the earlier slices) on `stream`, and its results go device ->
 * host on a second copy stream, so that the copies of a slice overlap the attention of its neighbours.  No
 * arithmetic happens outside those two entry points' kernels.
 *
 * q_host       bf16 [chunk_len, num_q_heads, head_dim_qk]   host, read
 * k_new_host   bf16 [chunk_len, num_kv_heads, head_dim_qk]  host, read: keys of the chunk's own tokens
 * v_new_host   bf16 [chunk_len, num_kv_heads, head_dim_v]   host, read; ignored when dev.v_cache == dev.k_cache (MLA)
 * out_host     bf16 [chunk_len, num_q_heads, head_dim_v]    host, written
 * lse_host     float [chunk_len, num_q_heads] or NULL       host, written
 *              Host buffers should be page-locked (copies from pageable memory do not overlap anything); they must
 *              stay valid until the work enqueued on `stream` has completed.
 * prefix_len, chunk_len   host scalars of the request; positions [0, prefix_len) are in the cache already.
 * slice_rows, num_slices  slice lengths in rows (positive, sum = chunk_len, at most VPP_HOST_MAX_SLICES), or NULL / 0:
 *              the library cuts the chunk into three runs of whole 128-row tiles that minimise what cannot overlap
 *              (first copy in, last copy out, idle tail of each launch's last wave); chunks of fewer than three
 *              tiles or ragged chunks go through as one slice.  vpp_chunk_attn_host_plan returns that choice.
 * dev          the device side, as for vpp_chunk_attn_fwd with num_reqs = 1 and total_q = chunk_len: caches and
 *              strides, block_table (device, one row), geometry, softmax_scale, num_kv_splits; q / out / lse are
 *              DEVICE staging buffers of the chunk's size (lse may be NULL iff lse_host is NULL); prefix_len and
 *              chunk_len are ignored (the library writes its own per slice); workspace of at least
 *              vpp_chunk_attn_host_workspace_size bytes; status optional device int32: the first nonzero status of
 *              the call's launches in launch order, 0 if none.  The caches are WRITTEN (the chunk's rows) and read.
 * k_new_dev, v_new_dev    device staging for the chunk's key / value rows, sizes as k_new_host / v_new_host
 *              (v_new_dev may be NULL under MLA aliasing).
 * Calls on one device are enqueued one at a time (a process-wide lock) and share two copy streams and their events,
 * created on the first call on that device (not a stream operation: make that first call outside any capture).
 * After that the call can be captured in a CUDA graph like any fork-join of streams; a replay reads the host buffers anew.
 * On return everything is enqueued and `stream` waits for the last device -> host copy.  Errors: as
 * vpp_chunk_attn_fwd and vpp_kv_append (vpp_host_last_error() has the detail); VPP_ERR_CUDA if a copy or an event
 * operation fails -- earlier slices may have been enqueued by then.
 */
#define VPP_HOST_MAX_SLICES 16
typedef struct {
    const void *q_host;
    const void *k_new_host;
    const void *v_new_host;
    void *out_host;
    float *lse_host;
    int32_t prefix_len;
    int32_t chunk_len;
    const int32_t *slice_rows;
    int32_t num_slices;
    vpp_chunk_attn_args dev;
    void *k_new_dev;
    void *v_new_dev;
} vpp_chunk_attn_host_args;

size_t vpp_chunk_attn_host_workspace_size(const vpp_chunk_attn_host_args *args);
/* Writes the slice lengths the call would use (at most VPP_HOST_MAX_SLICES) and returns their number; 0 if invalid. */
int32_t vpp_chunk_attn_host_plan(const vpp_chunk_attn_host_args *args, int32_t *slice_rows_out);
vpp_status vpp_chunk_attn_host_fwd(const vpp_chunk_attn_host_args *args, vpp_stream_t stream);
/* Thread-local detail of the last failure of the three functions above on this host thread. */
const char *vpp_host_last_error(void);

/*
 * Index-selected (sparse) chunk attention over the absorbed-MLA latent cache: the attention of the paper's third
 * model ("MLA + DSA sparse attention", evaluation set-up; its "Impact of Sparse Attention" paragraph is about the
 * flat cost curve this has).  The selection itself (a learned top-k indexer) is an input: for every query token a
 * list of key positions of its own request, shared by all q-heads.  Eq. 1 is evaluated over the listed keys:
 *   entry e of token t (position pos = prefix_len[r] + i) takes part iff 0 <= e <= pos; any other value is skipped;
 *   a position listed twice counts twice; out = softmax(scale q.k_e) v_e over the entries that take part, lse = log
 *   of the sum of their exp(scale q.k_e); a token with no entry that takes part gets out = 0 and lse = -inf.
 *
 * q            bf16 [total_q, num_q_heads, 576], dense, packed request-major. 16-byte aligned. num_q_heads <= 128.
 * kv_cache     bf16 latent cache, one kv-head of 576 features per position; values are features 0..511 of the same
 *              row.  Position pos of request r is row block_table[r][pos / block_size] * block_size + pos % block_size
 *              (block_table NULL: r * max_seq_len + pos, so the cache must hold num_reqs * max_seq_len rows); rows are
 *              kv_row_stride elements apart (a multiple of 8,
 *              >= 576), so a paged cache must have block stride = block_size * row stride.  16-byte aligned.  The
 *              cache must hold the chunk's own positions (every token's own row is read).
 * indices      int32 [total_q, topk], topk >= 1.
 * block_table, prefix_len, chunk_len, num_reqs (<= 8192), max_blocks_per_req, block_size (power of two), num_blocks,
 * total_q, max_seq_len, softmax_scale: as in vpp_chunk_attn_args.
 * out          bf16 [total_q, num_q_heads, 512]; lse float [total_q, num_q_heads] or NULL.
 * workspace    device memory of at least vpp_sparse_attn_workspace_size(total_q) bytes, 16-byte aligned; owned by the
 *              caller, contents irrelevant on entry.
 * status       optional device int32, zeroed by the call; VPP_DEV_BAD_LENGTHS (nothing is written),
 *              VPP_DEV_BAD_BLOCK (a needed block_table entry outside [0, num_blocks): results undefined but no
 *              access leaves the cache) or VPP_DEV_TIMEOUT as in vpp_chunk_attn_fwd.
 * Returns after enqueueing two kernels on `stream`; no allocation, no synchronisation.
 */
typedef struct {
    const void *q;
    const void *kv_cache;
    int64_t kv_row_stride;
    const int32_t *indices;
    int32_t topk;
    const int32_t *block_table;
    const int32_t *prefix_len;
    const int32_t *chunk_len;
    int32_t num_reqs;
    int32_t max_blocks_per_req;
    int32_t block_size;
    int32_t num_blocks;
    int32_t total_q;
    int32_t max_seq_len;
    int32_t num_q_heads;
    float softmax_scale;
    void *out;
    float *lse;
    void *workspace;
    size_t workspace_bytes;
    int32_t *status;
} vpp_sparse_attn_args;

size_t vpp_sparse_attn_workspace_size(int32_t total_q);
vpp_status vpp_sparse_mla_fwd(const vpp_sparse_attn_args *args, vpp_stream_t stream);

/* Static description of a status code. */
const char *vpp_status_string(vpp_status s);

/* Thread-local detail of the last failure on this host thread ("" if none). */
const char *vpp_last_error(void);

/* Number of kernels the last successful vpp_chunk_attn_fwd on this host thread enqueued. */
int32_t vpp_last_launch_count(void);

/*
 * The entry points describe q, the caches and their tiles to the copy engine with encoded tensor maps;
 * encoded maps are kept in a process-wide cache keyed on (base address, extents, strides, tile), so a call
 * that repeats an earlier call's buffers and shapes encodes nothing.  Process-wide totals so far (host
 * pointers; either may be NULL): look-ups and driver encodes.
 */
void vpp_tensor_map_cache_stats(int64_t *lookups, int64_t *encodes);

/*
 * Test hooks (no attention arithmetic; not needed by a user of the library).
 * vpp_test_tensor_map_cache: pure host code -- runs `repeats` identical look-ups plus two different ones
 *   through the cache logic with a stand-in encoder; returns the number of encodes it took (3 when the
 *   cache works) or a negative number on an inconsistency.
 * vpp_test_bounded_wait: enqueues a one-CTA kernel that waits, with the bounded wait every kernel of this
 *   library uses, at most limit_cycles (1 .. 2^31 SM clocks) for an arrival that never comes, then takes
 *   the kernels' teardown: *status (device int32, zeroed by the caller) becomes VPP_DEV_TIMEOUT.  Nothing
 *   is copied or multiplied, so nothing can fault or hang.
 */
int32_t vpp_test_tensor_map_cache(int32_t repeats);
vpp_status vpp_test_bounded_wait(int32_t *status, int64_t limit_cycles, vpp_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* VPP_H_ */
