/*
 * lagkv.h -- C ABI of the B200 (sm_100a) LagKV KV-cache compression library.
 *
 * LagKV (arXiv 2504.04704, Section 2.2) shortens a transformer KV cache without looking
 * at attention weights.  After an attention-sink prefix of S rows the cache is cut into
 * partitions of L rows ("lag size").  Partition p is scored against partition p+1: the
 * per-channel min and max of the next partition (Eq. 7, Eq. 8) normalise the current one
 * (Eq. 9); the standard deviation over head_dim of every normalised token goes through a
 * softmax over the partition's tokens (Eq. 10), once for K and once for V, and the two are
 * added (Eq. 11).  Per head and per partition the k = ceil(r*L) best tokens are kept
 * (last bullet of Section 2.2); the last full partition plus the Mod(Ls-S, L) trailing
 * rows stay as a sliding window.  The resulting length is Eq. 12.
 *
 * Conventions shared by every entry point
 *   - All cache pointers are DEVICE pointers to data in the plan's storage format (bf16 by
 *     default, fp16 or fp8 e4m3 when the plan says so: "bf16" below stands for the plan's
 *     format), 16-byte aligned; scalars and the config struct are host values.  The library allocates no device memory and
 *     never synchronises the stream, except in lagkv_read_status().
 *   - A cache is addressed as  base + b*stride_b + h*stride_h + s*stride_s + d  (strides
 *     in elements, channel stride 1).  A stride given as 0 means "contiguous
 *     [B, H, S, D]" for the S passed to the call.  Strides must be multiples of 16 bytes
 *     (8 elements of a 16-bit format, 16 of fp8).
 *   - "Layers" have no separate dimension: fold them into B (one allocation
 *     [layers*B, H, S, D]) so that one call covers a whole model.
 *   - Every function returning int returns a lagkv_status code (0 = success).
 *     Errors detected on the host leave all buffers untouched.  Errors detected on the
 *     device (a bounded wait that ran out, an append that would overflow idx capacity)
 *     are recorded in the status block at the start of the workspace and reported by
 *     lagkv_read_status(); the kernels never trap or spin forever.  After LAGKV_ETIMEOUT
 *     the outputs of that call are incomplete: a prefill's K_out / V_out / idx_out hold
 *     undefined rows; an append leaves seq_len / static_len of every sequence one of whose
 *     heads gave up as they were before the call, and the rows of such a sequence behind
 *     its static part are undefined (other heads may already have been moved).  The
 *     workspace itself stays usable: the per-sequence counters return to zero.
 *   - The workspace is caller-owned device memory of at least lagkv_workspace_bytes()
 *     bytes, 256-byte aligned, cleared once with lagkv_workspace_init() and then reusable
 *     across calls on the same stream.  Calls sharing a workspace must not overlap.
 */
#ifndef LAGKV_H_
#define LAGKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct lagkv_plan_s *lagkv_plan_t;

enum lagkv_status {
    LAGKV_OK = 0,
    LAGKV_EINVAL = 1,       /* null pointer, misalignment, bad shape / stride / size  */
    LAGKV_EUNSUPPORTED = 2, /* valid request the library has no kernel for            */
    LAGKV_EWORKSPACE = 3,   /* workspace missing or too small                         */
    LAGKV_ECUDA = 4,        /* CUDA runtime error at launch (left sticky, not cleared)*/
    LAGKV_ETIMEOUT = 5,     /* device: a bounded wait on an async copy ran out        */
    LAGKV_ECAPACITY = 6,    /* device: append needed more chunks than max_new_chunks  */
    LAGKV_ENOALLOC_LIMIT = 7 /* request larger than LAGKV_NOALLOC_SCRATCH_BYTES        */
};

enum lagkv_variant {
    LAGKV_VARIANT_LAGKV = 0,   /* Eq. 7-11: statistics from the next partition        */
    LAGKV_VARIANT_LOCALKV = 1, /* Eq. 14, Eq. 15: statistics from the partition itself */
    LAGKV_VARIANT_L2NORM = 2   /* Eq. 16: score = -||K row||_2, no softmax, V is only
                                  gathered.  Section 4.3 leaves the first two layers of
                                  the model uncompressed for this variant: layers have
                                  no dimension here, so the caller keeps those two
                                  layers out of the batch it folds into B               */
};

enum lagkv_dtype {
    LAGKV_DTYPE_BF16 = 0, /* the default (a zeroed field)                                */
    LAGKV_DTYPE_FP16 = 1, /* IEEE binary16 caches                                        */
    LAGKV_DTYPE_FP8_E4M3 = 2 /* one byte per element: 1 sign, 4 exponent (bias 7), 3 fraction
                             bits, no infinities, 0x7f / 0xff are NaN (the "e4m3fn" of the
                             deep-learning frameworks).  The paper names no storage format
                             and no scale; none is needed: whatever positive per-tensor,
                             per-head or per-channel scale the caller's quantiser uses, it
                             cancels in Eq. 9 (the same scale multiplies value, min and max),
                             so the scores are those of the stored bytes and the kept rows
                             are copied byte for byte.                                     */
};

typedef struct {
    int32_t B;          /* sequences (times layers when folded), >= 1                 */
    int32_t H_kv;       /* KV heads per sequence, >= 1; selection is per KV head      */
    int32_t D;          /* head_dim; supported: 64, 96, 128, 256 (128 is tuned)      */
    int32_t sink;       /* S: attention-sink rows kept verbatim, >= 0                 */
    int32_t lag;        /* L: partition size, 2 <= L <= 8192                          */
    double keep_ratio;  /* r in (0, 1]; k = ceil(r*L - 1e-9) clamped to [1, L]        */
    int32_t keep_k;     /* if > 0, k directly (overrides keep_ratio)                  */
    int32_t std_ddof;   /* divisor of the variance is D - std_ddof: 0 or 1            */
    int32_t variant;    /* enum lagkv_variant                                         */
    int64_t stride_b;   /* input-cache strides in elements; 0 = contiguous (see top)  */
    int64_t stride_h;
    int64_t stride_s;
    int32_t device;     /* CUDA device ordinal the plan launches on                   */
    int32_t dtype;      /* enum lagkv_dtype: storage format of every cache of the plan;
                           the paper names none, and the arithmetic after the exact
                           widening to fp32 is the same                               */
} lagkv_config;

/*
 * Build an immutable plan from a config (Section 2.2: S, L, r fix the whole pass).
 * Host work plus one-time CUDA attribute queries on cfg->device; no stream work.
 * On success *out owns host memory freed by lagkv_plan_destroy().
 */
int lagkv_plan(const lagkv_config *cfg, lagkv_plan_t *out);
void lagkv_plan_destroy(lagkv_plan_t plan);

/* k, the rows kept per compressed partition (r*L, text before Eq. 12). */
int32_t lagkv_keep_count(lagkv_plan_t plan);

/*
 * Eq. 12 generalised to a cache whose first static_len rows (sink + already compressed
 * part) are left alone:  static_len + k*(n-1) + L + rem  with n = floor(rest/L),
 * rem = rest mod L, rest = seq_len - static_len;  seq_len itself when rest < 2L (third
 * bullet of Section 2.2).  Pure host arithmetic.  static_len < 0 means "the plan's sink".
 */
int64_t lagkv_compressed_len(lagkv_plan_t plan, int64_t seq_len, int64_t static_len);

/*
 * The two lengths of a sequence after a pass (Section 2.2, bullets 2-4; Eq. 12): what
 * lagkv_compress_append() writes to seq_len[b] and static_len[b] on the device, computed on the
 * host so that a driver loop can mirror them without a read-back.  rest < 2L: both unchanged.
 * static_len < 0 means "the plan's sink".  Returns LAGKV_EINVAL for seq_len < static_len.
 */
int lagkv_lengths_after(lagkv_plan_t plan, int64_t seq_len, int64_t static_len, int64_t *new_seq_len,
                        int64_t *new_static_len);

/*
 * Inverse of Eq. 12 / Eq. 13 as used for the adaptive retention ratio of Section 3.2:
 * the smallest k in [1, L] whose compression ratio C = 1 - L_R/Ls does not exceed
 * target_C for a prompt of Ls rows.  Host arithmetic.  Returns k (L when no compression
 * is possible because Ls < S + 2L).
 */
int32_t lagkv_keep_for_target(int64_t Ls, int32_t sink, int32_t lag, double target_C);

/*
 * Bytes of workspace needed: the status block plus, for lagkv_compress_append(), one counter
 * per sequence (rounded up to 256 bytes) and room for max_new_chunks*k kept indices per
 * (b, h).  Pass 0 for prefill / gather only.
 */
size_t lagkv_workspace_bytes(lagkv_plan_t plan, int32_t max_new_chunks);

/* Clear the status block and the append counters (async memset on the stream).  Call once
 * per workspace; the kernels leave the counters at zero. */
int lagkv_workspace_init(lagkv_plan_t plan, void *workspace, size_t workspace_bytes,
                         void *cuda_stream);

/*
 * One-shot compression of a freshly prefilled cache (first bullet of Section 2.2; Eq. 7-12).
 * Every sequence has S_in rows.  Out of place; K, V are not modified and may not alias
 * the outputs.  With L_R = lagkv_compressed_len(plan, S_in, -1):
 *   K_out, V_out [B, H, L_R, D] bf16 contiguous: sink rows, then for p = 0..n-2 the k kept
 *                rows of partition p in ascending position, then the window rows.
 *                Both NULL = indices only.
 *   idx_out      [B, H, L_R] int32 or NULL: source row of every output row.
 *   scores_out   [B, H, (n-1)*L] fp32 or NULL: final score (Eq. 11) of every token of a
 *                compressed partition.
 * S_in < S + 2L is not an error: the pass is the identity (L_R = S_in).
 * Asynchronous on cuda_stream (a cudaStream_t, NULL = default stream).
 */
int lagkv_compress_prefill(lagkv_plan_t plan, const void *K, const void *V, int64_t S_in,
                           void *K_out, void *V_out, int32_t *idx_out, float *scores_out,
                           void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * lagkv_compress_prefill() for caches that live in HOST memory (the same pass, Section 2.2,
 * Eq. 7-12; the paper has no counterpart for the transfer).  K_host, V_host [B, H, S_in, D]
 * and the outputs K_out_host, V_out_host [B, H, L_R, D], idx_out_host [B, H, L_R] are HOST
 * pointers, contiguous, pinned if the copies are to overlap (pageable memory works, slower);
 * the plan's strides must be 0.  The B sequences are cut into chunks of chunk_B (B % chunk_B
 * == 0); each chunk is copied to the device, compressed and copied back, on three internal
 * streams with two staging slots so that copies in both directions overlap the kernel.
 *   staging    caller-owned DEVICE memory, 256-byte aligned, at least
 *              lagkv_host_staging_bytes(plan, S_in, chunk_B) bytes (0 = bad arguments)
 *   workspace  as for lagkv_compress_prefill()
 * Nothing is allocated on the device; streams and events are created once per plan on the
 * first call and freed by lagkv_plan_destroy().  Ordered after the work already on
 * cuda_stream; cuda_stream waits for the last copy, so a synchronise on it (or
 * lagkv_read_status) makes the host buffers valid.  The host does not block.  Calls on one
 * plan are enqueued one at a time (internal lock) and must use the same cuda_stream if they
 * share staging memory.
 */
size_t lagkv_host_staging_bytes(lagkv_plan_t plan, int64_t S_in, int32_t chunk_B);
int lagkv_compress_prefill_host(lagkv_plan_t plan, const void *K_host, const void *V_host, int64_t S_in,
                                void *K_out_host, void *V_out_host, int32_t *idx_out_host,
                                int32_t chunk_B, void *staging, size_t staging_bytes, void *workspace,
                                size_t workspace_bytes, void *cuda_stream);

/*
 * Incremental (recursive) compression during decode or chunked prefill (Section 2.2,
 * bullets 2-4; Fig. 1).  In place on caches [B, H, S_cap, D] (the plan's strides, 0 =
 * contiguous for S_cap).  seq_len[B] and static_len[B] are DEVICE int32 arrays: rows
 * [0, static_len[b]) are the sink plus everything kept so far, rows up to seq_len[b] are
 * valid.  For every sequence whose rest = seq_len - static_len is at least 2L the n-1
 * oldest partitions are scored against their successors, their k kept rows are packed
 * behind the static part, the window (last full partition + remainder) is moved down
 * behind them, and the call sets static_len += (n-1)*k, seq_len = static_len + L + rem.
 * Other sequences are left untouched (decided on the device: no host sync).  The call is
 * always the same single launch with the same arguments, so it may be captured into a CUDA
 * graph once and replayed after every decoded token.
 *   max_new_chunks  capacity: a sequence with n-1 > max_new_chunks is left untouched and
 *                   LAGKV_ECAPACITY is recorded in the status block.
 *   idx_out     [B, H, max_new_chunks*k] int32 or NULL: pre-call positions of the rows
 *               kept by this call (entries of skipped sequences are not written).
 *   scores_out  [B, H, max_new_chunks*L] fp32 or NULL.
 * The workspace must have been sized with the same max_new_chunks.
 * With max_new_chunks == 1 (decode: at most one partition completes per call) and at most
 * sm_count (b, h) units the launch is a grid of thread-block clusters, one cluster per unit,
 * which keeps the window in shared memory between its two uses; it is still one launch.
 */
int lagkv_compress_append(lagkv_plan_t plan, void *K_cache, void *V_cache, int64_t S_cap,
                          int32_t *seq_len, int32_t *static_len, int32_t max_new_chunks,
                          int32_t *idx_out, float *scores_out, void *workspace,
                          size_t workspace_bytes, void *cuda_stream);

/*
 * Paged caches (block tables).  The method itself (Section 2.2) only speaks of a cache of n
 * rows per head; serving engines store that cache as fixed-size pages drawn from a pool, with a
 * table per sequence saying which page holds which rows.  K_pool / V_pool are DEVICE pointers to
 * pools addressed as
 *     pool + block_table[b*max_blocks + s/page_size]*stride_page + h*stride_h + (s%page_size)*stride_s + d
 * (the same table and strides for K and V).  A stride given as 0 means dense
 * [num_pages, H_kv, page_size, D].  With layers folded into B, sequence b's table row simply
 * names pages of its own layer.  The plan's own strides must be 0.
 */
typedef struct {
    const int32_t *block_table; /* DEVICE int32 [B, max_blocks], 4-byte aligned               */
    int32_t max_blocks;         /* entries per sequence; max_blocks*page_size >= rows addressed */
    int32_t page_size;          /* rows per page: a power of two, >= 16                        */
    int64_t stride_page;        /* elements between pages          (0 = H_kv*stride_h)         */
    int64_t stride_h;           /* elements between heads in a page (0 = page_size*stride_s)   */
    int64_t stride_s;           /* elements between rows in a page  (0 = D); all three strides
                                   multiples of 16 bytes                                       */
} lagkv_paged_layout;

/*
 * lagkv_compress_prefill() reading a paged cache (same pass, Section 2.2, Eq. 7-12): every
 * sequence has S_in rows; the outputs are contiguous as there.  Runs on the kernel family that
 * looks rows up page by page (a tile that straddles a page boundary is fetched in two copies).
 */
int lagkv_compress_prefill_paged(lagkv_plan_t plan, const void *K_pool, const void *V_pool,
                                 const lagkv_paged_layout *layout, int64_t S_in, void *K_out, void *V_out,
                                 int32_t *idx_out, float *scores_out, void *workspace, size_t workspace_bytes,
                                 void *cuda_stream);

/*
 * lagkv_compress_append() in place on a paged cache (Section 2.2, bullets 2-4; Fig. 1): kept rows
 * and the window are moved down inside the sequence's own pages, seq_len / static_len are
 * updated as there.  A sequence may hold at most max_blocks*page_size rows.  Pages that lie wholly
 * behind the new seq_len[b] hold no valid rows any more; giving them back to the pool is the
 * caller's business (the table is not modified).
 */
int lagkv_compress_append_paged(lagkv_plan_t plan, void *K_pool, void *V_pool, const lagkv_paged_layout *layout,
                                int32_t *seq_len, int32_t *static_len, int32_t max_new_chunks, int32_t *idx_out,
                                float *scores_out, void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * lagkv_compress_append() for callers that have no device memory to give as a workspace.
 * (The paper has no counterpart: this is a property of the library, not of the method.)
 *
 * Who needs it: code that runs where allocating is off the table -- a decode loop inside a
 * serving engine whose memory pool is already carved up, a plug-in called from someone
 * else's stream callback or capture region, a host that forbids cudaMalloc after start-up
 * because it would synchronise the device.  Such a caller cannot produce the workspace
 * that lagkv_compress_append() wants, so the library brings its own: a fixed array of
 * LAGKV_NOALLOC_SCRATCH_BYTES bytes inside the library image.  Every GPU that loads the
 * library holds one copy of it until the process exits.
 *
 * Arguments are those of lagkv_compress_append() minus workspace / workspace_bytes, plus
 *   status_out  DEVICE int32[4] or NULL: receives the status block of this call (same
 *               meaning as lagkv_read_status(): [0] first device-side status, [1] detail,
 *               [2] zero-range channel count), written on cuda_stream after the kernels.
 *               With NULL the block stays in the built-in array until the next call on that
 *               device clears it: read it before then with lagkv_read_status(plan, NULL, ...),
 *               or a device-side LAGKV_ECAPACITY / LAGKV_EINVAL / LAGKV_ETIMEOUT of this call
 *               goes unnoticed.
 * The call allocates nothing and frees nothing; it enqueues a small memset (status block and
 * counters), the append kernel and, if asked, a 16-byte device-to-device copy.
 *
 * Limit: 256 + 256*ceil(B/64) + B*H_kv*max_new_chunks*k*4 bytes must not exceed
 * LAGKV_NOALLOC_SCRATCH_BYTES when idx_out is NULL (the kept positions are parked in the
 * scratch); with idx_out given only the first two terms (status block, one counter per
 * sequence) are used.  Beyond the limit the call returns
 * LAGKV_ENOALLOC_LIMIT and touches nothing.
 *
 * First call on a device: the library looks up the device address of its array (once per
 * device, with that device current).  Make that first call outside any stream capture.
 *
 * Sharing: all calls on a device use the same array, and the array keeps whatever the last
 * call left in it.  The status block is cleared at the start of every call; the kept
 * positions are rewritten before they are read.  Two calls that overlap on the GPU (two
 * streams, no dependency between them) race on the array: order them.
 */
#define LAGKV_NOALLOC_SCRATCH_BYTES 1048576
int lagkv_compress_append_noalloc(lagkv_plan_t plan, void *K_cache, void *V_cache, int64_t S_cap,
                                  int32_t *seq_len, int32_t *static_len, int32_t max_new_chunks,
                                  int32_t *idx_out, float *scores_out, int32_t *status_out,
                                  void *cuda_stream);

/*
 * Row gather, the separable part of the compaction (Fig. 1):
 *   K_out[b,h,j,:] = K[b,h,idx[b,h,j],:],  same for V,  j < n_idx.
 * K, V use the plan's strides with S_in rows; outputs are contiguous [B, H, n_idx, D].
 * V / V_out may both be NULL.  idx is a DEVICE int32 array [B, H, n_idx]; every entry
 * must lie in [0, S_in) -- entries outside are skipped and LAGKV_EINVAL is recorded in
 * the status block when a workspace is given (workspace may be NULL).
 */
int lagkv_gather(lagkv_plan_t plan, const void *K, const void *V, int64_t S_in,
                 const int32_t *idx, int64_t n_idx, void *K_out, void *V_out, void *workspace,
                 void *cuda_stream);

/* lagkv_gather() reading a paged cache (see lagkv_paged_layout); outputs contiguous as there. */
int lagkv_gather_paged(lagkv_plan_t plan, const void *K_pool, const void *V_pool, const lagkv_paged_layout *layout,
                       int64_t S_in, const int32_t *idx, int64_t n_idx, void *K_out, void *V_out, void *workspace,
                       void *cuda_stream);

/*
 * Synchronise cuda_stream, copy the status block to the host and clear it.  workspace == NULL
 * names the status block of the library's built-in scratch on the plan's device (the one
 * lagkv_compress_append_noalloc() uses).
 * host_status[0] = first device-side lagkv_status recorded since the last read (0 = none),
 * host_status[1] = detail (block index), host_status[2] = count of zero-range reference
 * channels seen, host_status[3] = reserved.  Returns host_status[0], or LAGKV_ECUDA.
 */
int lagkv_read_status(lagkv_plan_t plan, void *workspace, void *cuda_stream,
                      int32_t host_status[4]);

/*
 * Launch shape the plan uses for a prefill of S_in rows: info[0] = grid, info[1] = block
 * threads, info[2] = dynamic shared memory bytes, info[3] = kernel launches per call,
 * info[4] = kernel family (0 = identity copy, 1 = uniform kernel, 2 = warp-specialised
 * kernel, 3 = pair kernel), info[5] = kernel family lagkv_compress_prefill_paged() uses for
 * the same call (1 or 2; 0 for the identity copy).
 */
int lagkv_launch_info(lagkv_plan_t plan, int64_t S_in, int32_t info[6]);

/*
 * Tuning override of the launch shape: warps per CTA (2, 4 or 8 = the uniform kernel, used
 * for prefill and append alike; 12 = the warp-specialised prefill kernel with 8 streaming,
 * 3 select and 1 copy warp; LAGKV_TUNE_PAIRS = the prefill kernel for partitions of at most
 * 512 rows, four K/V warp pairs with an epilogue warp each, LagKV only; the last two leave
 * the append shape alone), rows per staged tile
 * (16 or 32), ring stages per streaming warp (2..8) and resident CTAs per SM to size the
 * prefill grid for (>= 1; must be 1 with 12 warps).  A value of 0 keeps the current
 * choice.  Returns LAGKV_EUNSUPPORTED for a combination that was not compiled or does not
 * fit shared memory.
 */
#define LAGKV_TUNE_PAIRS 100
/*
 * warps = LAGKV_TUNE_APPEND_CLUSTER (4 warps per CTA) or LAGKV_TUNE_APPEND_CLUSTER8 (8 warps,
 * head_dim 128 only) shapes the kernel of one-partition appends (lagkv_compress_append with
 * max_new_chunks == 1, LagKV scoring) instead: tile_rows = row splits per tensor (1, 2 or 4: a
 * cluster of 2, 4 or 8 CTAs per (b, h) unit), stages = ring stages (2..4), ctas_per_sm = CTAs
 * per SM to leave room for (1..4; fewer resident rows of the window when they do not all fit,
 * which only a split of 1 allows).  The prefill shape is left alone.
 */
#define LAGKV_TUNE_APPEND_CLUSTER 101
#define LAGKV_TUNE_APPEND_CLUSTER8 102
int lagkv_plan_tune(lagkv_plan_t plan, int32_t warps, int32_t tile_rows, int32_t stages,
                    int32_t ctas_per_sm);

/*
 * Self-test of the failure path: launches one warp that waits, with the same bounded wait the
 * compress kernels use, on a barrier nothing will ever complete.  After about limit_ms
 * (1..2000) the wait gives up and LAGKV_ETIMEOUT is recorded in the status block of
 * `workspace` (read it with lagkv_read_status()); the device stays usable.  Asynchronous.
 */
int lagkv_selftest_bounded_wait(lagkv_plan_t plan, void *workspace, int32_t limit_ms, void *cuda_stream);

const char *lagkv_status_string(int status);
const char *lagkv_version(void);

#ifdef __cplusplus
}
#endif
#endif /* LAGKV_H_ */
