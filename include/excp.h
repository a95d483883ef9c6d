/*
 * excp.h -- C ABI of the ExCP checkpoint-compression hot path for NVIDIA B200 (sm_100a).
 *
 * What the library computes (arXiv 2406.11257, "ExCP: Extreme LLM Checkpoint
 * Compression via Weight-Momentum Joint Shrinking"):
 *
 *   compress   Algorithm 1 without its archiver step, per tensor:
 *                dW = W_t - W^_(t-1)                       (Section 3.1, Eq. ckpt_res)
 *                M_w(i) = [ |dW(i)| * sqrt(eas(i)) > alpha * median ]      (Section 3.2, Eq. rw)
 *                M_o(i) = [ |ea(i)| > beta * mean(|ea|) ] and M_w(i)       (Section 3.2, Eq. ro)
 *                joint application of M_w to dW and of M_o to BOTH moments (Algorithm 1, joint_prune)
 *                K-means of the survivors to 2^bits - 1 centres per stream, codes 1..K,
 *                packed `bits` per code (Section 3.3; Section 4.2: bits = 4, two per byte)
 *   decompress Algorithm 2 without its un-archiver step:
 *                dW^ = C_w[I_w], O^ = C_o[I_o], W^_t = W^_(t-1) + dW^
 *
 * Letters: the paper writes v_t for Adam's FIRST moment and m_t for its SECOND.  This header
 * says `ea` (first moment, exp_avg) and `eas` (second moment, exp_avg_sq).
 *
 * Where the paper is silent the library fixes one reading so that the output is unique:
 *   - the median is the lower median (rank floor((n-1)/2)) of |W_t| (EXCP_MEDIAN_ABS_WEIGHT, the
 *     letter of Eq. rw) or of |dW| (EXCP_MEDIAN_ABS_RESIDUAL), per tensor;
 *   - mean(|ea|) is the exact mean rounded once to fp32;
 *   - K-means is Lloyd's algorithm per tensor and per stream (dW, ea, eas): start = the K
 *     equal-mass quantiles of a seeded index-stratified sample of <= 1024 survivors; assignment
 *     = number of mid-points (c_j + c_j+1)/2, taken in fp64, lying strictly below x; update =
 *     fixed-point mean (values scaled by 2^(30-E), E = exponent of the stream's largest
 *     magnitude, rounded half-to-even, summed in int64); empty clusters keep their centre;
 *     centres kept in ascending order, -0 before +0 (they can only meet with pruning switched
 *     off: a kept value is never zero otherwise); `kmeans_iters` iterations, then the final
 *     assignment.
 *
 * Record layout of one tensor (little endian, every section on a 16-byte boundary, padding zero):
 *     0 u32 magic "EXCP"   4 u32 version = 1     8 u64 numel
 *    16 u64 nnz_w         24 u64 nnz_o          32 u32 bits      36 u32 K = 2^bits - 1
 *    40 u32 header bytes  44 u32 record flags   48 u64 record bytes   56 u64 0
 *       (record flags: 0 for the full method; see excp_flags for the ablation variants)
 *    64 f32 centres of dW [K], of ea [K], of eas [K]; header padded to 16 bytes
 *    .. bitmap of M_w, bitmap of M_o: u32 words, bit k of word w = element 32 w + k
 *    .. codes of dW [nnz_w], of ea [nnz_o], of eas [nnz_o]: survivors in index order, `bits`
 *       each, value 1..K, survivor r at bit r * bits of the section (low bits first)
 * A checkpoint blob is the tensors' records back to back.
 *
 * Conventions for every call:
 *   - "device" pointers are CUDA device memory on the handle's device, 16-byte aligned;
 *     "host" pointers are ordinary host memory.  The library never frees or reallocates a
 *     caller's buffer and never writes an input.
 *   - All work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL = the
 *     legacy default stream).  Calls that return sizes or statistics to the host
 *     synchronise that stream once, at their end.
 *   - The handle owns the scratch workspace; it is not thread-safe: one call at a time.
 *   - Errors are return codes; nothing is thrown and nothing aborts.  After a non-OK
 *     return the output buffers hold unspecified bytes.
 */
#ifndef EXCP_H_
#define EXCP_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct excp_handle_s* excp_handle;

typedef enum {
    EXCP_OK = 0,
    EXCP_ERR_INVALID_ARG = -1,      /* null / misaligned pointer, bad parameter, workspace too small for a tensor */
    EXCP_ERR_UNSUPPORTED = -2,      /* a variant the called routine does not handle (dense layout of a record that is
                                       not the 4-bit method's own; raw records through the host-buffer entry point) */
    EXCP_ERR_BUFFER_TOO_SMALL = -3, /* blob_capacity below what the records need */
    EXCP_ERR_CUDA = -4,             /* a CUDA runtime call failed; see excp_last_cuda_error */
    EXCP_ERR_CORRUPT_BLOB = -5,     /* decompress: header, sizes, bitmap population or a code is inconsistent */
    EXCP_ERR_NONFINITE_INPUT = -6,  /* compress: NaN or infinity in an input, or a negative second moment */
    EXCP_ERR_TIMEOUT = -7           /* a bounded wait on an asynchronous copy ran out (no kernel waits on another kernel) */
} excp_status;

typedef enum {
    EXCP_MEDIAN_ABS_WEIGHT = 0,     /* median(|W_t|): Eq. (rw) as printed */
    EXCP_MEDIAN_ABS_RESIDUAL = 1    /* median(|dW_t|): the quantity the mask prunes */
} excp_median_source;

/* Ablation switches: the rows of the paper's two ablation tables as variants of the same path.
 * The ViT table's caption defines the first two ("no check" under M2W: the weights are pruned by a
 * set threshold instead of alpha / sqrt(m_t); under W2M: M_o(i) = [ v_t(i) > r_o ]); the table of
 * Section 4.4 toggles residual, prune and quant.  A record written with a switch says so in its
 * header (offset 44), and excp_decompress_* honour it. */
typedef enum {
    EXCP_FLAG_NO_W2M = 1,           /* M_o(i) = [ |ea(i)| > beta * mean ], without "and M_w(i)"; record flag 1 */
    EXCP_FLAG_NO_M2W = 2,           /* M_w(i) = [ |dW(i)| > alpha ]: alpha itself is the set threshold */
    EXCP_FLAG_NO_RESIDUAL = 4,      /* W_t is compressed instead of dW; w_prev is not read (may be NULL);
                                       decompress writes W^ = decoded value, 0 where pruned; record flag 2 */
    EXCP_FLAG_NO_PRUNE = 8,         /* both masks keep every element */
    EXCP_FLAG_NO_QUANT = 16         /* no K-means: the sections hold the survivors as fp32 (bits = 32, K = 0,
                                       64-byte header without centres); record flag 4 */
} excp_flags;

/* Hyper-parameters.  Section 4.2: alpha = 5e-5, beta = 2.0, bits = 4. */
typedef struct {
    float alpha;                    /* Eq. (rw) */
    float beta;                     /* Eq. (ro) */
    int bits;                       /* code width n: 2, 4 or 8; K = 2^n - 1 centres (Section 4.2 uses 4; the
                                       quantisation-bins table of Section 4.4 also 2 and 8) */
    int kmeans_iters;               /* Lloyd iterations before the final assignment (>= 0) */
    unsigned long long seed;        /* seed of the K-means start sample */
    int median_source;              /* excp_median_source */
    unsigned flags;                 /* excp_flags, OR-ed; 0 = the full method */
} excp_params;

/* Per-tensor result, written to host memory. */
typedef struct {
    unsigned long long numel;
    unsigned long long nnz_w;       /* population of M_w */
    unsigned long long nnz_o;       /* population of M_o */
    unsigned long long blob_bytes;  /* size of this tensor's record */
    float median;                   /* the median entering Eq. (rw) */
    float mean_abs_ea;              /* the mean entering Eq. (ro) */
    float thr_w;                    /* alpha * median */
    float thr_o;                    /* beta * mean */
    /* The K-means objective (Section 3.3) after the final assignment, per stream: the sum over the
     * survivors of (value - its centre)^2.  A diagnostic: squares and sums of up to 16 of them in fp32, those
     * added in fp64 in no fixed order, so it agrees with the plain fp64 sum to about 1e-6 relative and its
     * last bits can differ from run to run.  0 where the sections hold raw fp32 survivors, and 0 unless
     * excp_set_report_sse has switched it on (it costs the packing sweep about a quarter more time). */
    double sse_w;
    double sse_ea;
    double sse_eas;
} excp_tensor_stats;

/* Creates a handle on CUDA device `device` with a scratch workspace for `workspace_numel`
 * elements (about 24.3 bytes each; tensors are processed in groups whose sizes, each rounded
 * up to 4096, sum to at most this), so the largest single tensor must not exceed it.
 * Allocates device and pinned host memory.  Returns EXCP_ERR_CUDA if the device or the
 * memory cannot be had. */
excp_status excp_create(excp_handle* out, int device, size_t workspace_numel);

/* Frees everything the handle owns.  NULL is accepted. */
excp_status excp_destroy(excp_handle h);

/* Size in bytes of a record with the given counts (the layout above).  0 if bits is not 2, 4, 8
 * or 32 (32 = EXCP_FLAG_NO_QUANT's raw fp32 sections). */
size_t excp_record_bytes(size_t numel, size_t nnz_w, size_t nnz_o, int bits);

/* Worst-case record size for a tensor of `numel` elements (every element kept). */
size_t excp_compress_bound(size_t numel, int bits);

/* Static, NUL-terminated description of a status code. */
const char* excp_status_string(excp_status s);

/* The cudaError_t (as int) of the last failed CUDA call on this handle, 0 if none. */
excp_status excp_last_cuda_error(excp_handle h, int* cuda_err);

/* Algorithm 1 (up to the archiver) for one tensor.
 *   w_t, w_prev, ea, eas  device, fp32[numel], read only.  w_prev is the LAST RECONSTRUCTED
 *                         weight tensor W^_(t-1) (Section 3.4).
 *   blob_out              device, blob_capacity bytes; receives the record.
 *   blob_bytes_out        host; receives the record size.
 *   stats_out             host, may be NULL.
 * numel = 0 is legal and gives a header-only record.  The tensor counts as index 0 of a
 * checkpoint for the K-means start.  Synchronises the stream. */
excp_status excp_compress_tensor(excp_handle h, const excp_params* params,
                                 const float* w_t, const float* w_prev, const float* ea, const float* eas,
                                 size_t numel, void* blob_out, size_t blob_capacity,
                                 size_t* blob_bytes_out, excp_tensor_stats* stats_out, void* cuda_stream);

/* Algorithm 1 over a tensor list; tensor i uses i as its index in the K-means start.
 *   w_t, w_prev, ea, eas  host arrays [num_tensors] of device pointers (fp32[numel[i]]).
 *   numel                 host [num_tensors].
 *   blob_out              device, blob_capacity bytes; records back to back.
 *   tensor_offsets_out    host [num_tensors + 1]; record i is [offsets[i], offsets[i+1]).
 *   stats_out             host [num_tensors], may be NULL.
 * All tensors of a group run through each kernel together, so the number of launches does
 * not grow with the tensor count.  Synchronises the stream. */
excp_status excp_compress_checkpoint(excp_handle h, const excp_params* params, size_t num_tensors,
                                     const float* const* w_t, const float* const* w_prev,
                                     const float* const* ea, const float* const* eas,
                                     const size_t* numel, void* blob_out, size_t blob_capacity,
                                     size_t* tensor_offsets_out, excp_tensor_stats* stats_out,
                                     void* cuda_stream);

/* excp_compress_checkpoint for a SHARE of a checkpoint: the tensors of one checkpoint dealt to
 * several processes, one GPU each (Algorithm 1 treats every tensor on its own, so nothing is
 * exchanged between them).  tensor_index (host [num_tensors]) gives, for every tensor of the call,
 * its index in the WHOLE checkpoint, which is what seeds its K-means start sample; the records are
 * then byte for byte the ones a single excp_compress_checkpoint over the whole list writes for
 * those tensors.  Offsets are relative to this call's blob_out.  Everything else as for
 * excp_compress_checkpoint. */
excp_status excp_compress_checkpoint_indexed(excp_handle h, const excp_params* params, size_t num_tensors,
                                             const float* const* w_t, const float* const* w_prev,
                                             const float* const* ea, const float* const* eas,
                                             const size_t* numel, const size_t* tensor_index,
                                             void* blob_out, size_t blob_capacity,
                                             size_t* tensor_offsets_out, excp_tensor_stats* stats_out,
                                             void* cuda_stream);

/* Weights stored in 16 bits (Section 4.3 notes that the PanGu-pi weights are saved in float16).
 * excp_compress_checkpoint with W_t and W^_(t-1) given as IEEE binary16 (EXCP_WEIGHTS_F16) or
 * bfloat16 (EXCP_WEIGHTS_BF16) arrays; the moments stay fp32.  Every weight is widened to fp32,
 * which is exact, and from there the path is the fp32 one: the record is byte for byte the record
 * of the widened tensors, and carries no trace of the storage format.
 *   w_t, w_prev           host arrays [num_tensors] of device pointers to numel[i] 16-bit values,
 *                         16-byte aligned.
 * Everything else as for excp_compress_checkpoint. */
typedef enum {
    EXCP_WEIGHTS_F16 = 1,
    EXCP_WEIGHTS_BF16 = 2
} excp_weight_format;
excp_status excp_compress_checkpoint_w16(excp_handle h, const excp_params* params, size_t num_tensors,
                                         const void* const* w_t, const void* const* w_prev,
                                         const float* const* ea, const float* const* eas,
                                         const size_t* numel, int weight_format, void* blob_out, size_t blob_capacity,
                                         size_t* tensor_offsets_out, excp_tensor_stats* stats_out,
                                         void* cuda_stream);

/* excp_decompress_checkpoint for 16-bit weights: w_prev and w_out hold `weight_format` values.
 * W^_t = W^_(t-1) + dW^ is taken in fp32 and rounded once, to nearest even, to the stored format;
 * a pruned weight keeps the bits of W^_(t-1).  ea_out, eas_out are fp32. */
excp_status excp_decompress_checkpoint_w16(excp_handle h, const void* blob, const size_t* tensor_offsets,
                                           size_t num_tensors, const void* const* w_prev, const size_t* numel,
                                           int weight_format, void* const* w_out, float* const* ea_out,
                                           float* const* eas_out, void* cuda_stream);

/* excp_compress_checkpoint for a checkpoint that lives in HOST memory (the usual case: the
 * compression runs beside training, Section 3.4, on a copy of the states).
 *   w_t, w_prev, ea, eas  host arrays [num_tensors] of HOST pointers (fp32[numel[i]]); page-locked
 *                         memory is needed for the copies to overlap the kernels.
 *   blob_out              HOST, blob_capacity bytes; receives the records back to back.
 * The tensor list is cut into the same groups as in excp_compress_checkpoint; while the kernels
 * of one group run on `cuda_stream`, the inputs of the next are copied to a second device
 * staging slot on a copy stream of the handle and the finished records are copied back on
 * another.  The first call allocates the staging (32 bytes per workspace element plus two record
 * buffers).  Records and offsets are identical to excp_compress_checkpoint's.  Synchronises.
 * All four pointers of a tensor are required whatever the flags; EXCP_FLAG_NO_QUANT is not offered here
 * (EXCP_ERR_UNSUPPORTED: the device-side record staging is sized for coded records; a group whose records
 * outgrow it returns EXCP_ERR_BUFFER_TOO_SMALL). */
excp_status excp_compress_checkpoint_host(excp_handle h, const excp_params* params, size_t num_tensors,
                                          const float* const* w_t, const float* const* w_prev,
                                          const float* const* ea, const float* const* eas,
                                          const size_t* numel, void* blob_out, size_t blob_capacity,
                                          size_t* tensor_offsets_out, excp_tensor_stats* stats_out,
                                          void* cuda_stream);

/* Algorithm 2 (after the un-archiver) for one tensor.
 *   blob                  device, blob_bytes bytes, one record.
 *   w_prev                device fp32[numel]: W^_(t-1).
 *   w_out, ea_out, eas_out device fp32[numel].  w_out may be the same buffer as w_prev
 *                         (in-place update); no other overlap is allowed.
 * Pruned weights keep w_prev bit for bit; pruned moments decode to 0.
 * Synchronises the stream; returns EXCP_ERR_CORRUPT_BLOB if the record is inconsistent
 * (every read stays inside [blob, blob + blob_bytes) even then). */
excp_status excp_decompress_tensor(excp_handle h, const void* blob, size_t blob_bytes,
                                   const float* w_prev, size_t numel,
                                   float* w_out, float* ea_out, float* eas_out, void* cuda_stream);

/* Algorithm 2 over a tensor list (the loop body of Algorithm 3).
 *   blob                  device; tensor_offsets host [num_tensors + 1] as returned by compress.
 *   w_prev, w_out, ea_out, eas_out  host arrays [num_tensors] of device pointers. */
excp_status excp_decompress_checkpoint(excp_handle h, const void* blob, const size_t* tensor_offsets,
                                       size_t num_tensors, const float* const* w_prev, const size_t* numel,
                                       float* const* w_out, float* const* ea_out, float* const* eas_out,
                                       void* cuda_stream);

/* The index layout as the paper prints it (Section 3.3: the pruned entries stay zero and the
 * cluster index I_t is saved; Section 4.2: zero occupies one of the 2^n centres, two int4 per
 * int8): one code per ELEMENT, 0 where the element is pruned, no bitmap.  This is the (I, C) pair
 * Algorithm 1 hands to its archiver.  Container of one tensor (little endian, sections on 16 bytes,
 * padding zero):
 *     the record's 64-byte header with magic "EXCD" and the CONTAINER's size at offset 48,
 *     f32 centres of dW [K], of ea [K], of eas [K]; header padded to 16 bytes
 *     codes of dW [numel], of ea [numel], of eas [numel]: `bits` each, element i at bit i * bits
 * excp_dense_bytes gives its size (0 if bits is not 2, 4 or 8).
 *
 * excp_record_to_dense / excp_checkpoint_to_dense rewrite records (device) as dense containers
 * (device): bitmap rank -> code, per element.  Records of an ablation variant (non-zero record
 * flags) have no dense layout: EXCP_ERR_UNSUPPORTED.
 *   blob, tensor_offsets  as returned by excp_compress_checkpoint.
 *   dense_out             device, dense_capacity bytes; containers back to back.
 *   dense_offsets_out     host [num_tensors + 1] (excp_record_to_dense: dense_bytes_out, host).
 * Return EXCP_ERR_BUFFER_TOO_SMALL before any launch if the containers do not fit, and
 * EXCP_ERR_CORRUPT_BLOB like excp_decompress_checkpoint.  Synchronise the stream. */
size_t excp_dense_bytes(size_t numel, int bits);
excp_status excp_record_to_dense(excp_handle h, const void* record, size_t record_bytes, size_t numel,
                                 void* dense_out, size_t dense_capacity, size_t* dense_bytes_out,
                                 void* cuda_stream);
excp_status excp_checkpoint_to_dense(excp_handle h, const void* blob, const size_t* tensor_offsets,
                                     size_t num_tensors, const size_t* numel, void* dense_out,
                                     size_t dense_capacity, size_t* dense_offsets_out, void* cuda_stream);

/* Algorithm 2 on the dense layout: every element looks its code up; code 0 keeps W^_(t-1) bit for
 * bit and gives 0 in both moments.  Arguments as for excp_decompress_tensor / _checkpoint, with
 * dense containers in place of records.  EXCP_ERR_CORRUPT_BLOB if the header disagrees with the
 * layout, the number of non-zero codes differs from the header's counts, the two moments disagree
 * on what is kept, a moment is kept where the weight is pruned, or a code lies past the last
 * element (every read stays inside the container even then).  Synchronise the stream. */
excp_status excp_decompress_dense_tensor(excp_handle h, const void* dense, size_t dense_bytes,
                                         const float* w_prev, size_t numel,
                                         float* w_out, float* ea_out, float* eas_out, void* cuda_stream);
excp_status excp_decompress_dense_checkpoint(excp_handle h, const void* dense, const size_t* dense_offsets,
                                             size_t num_tensors, const float* const* w_prev, const size_t* numel,
                                             float* const* w_out, float* const* ea_out, float* const* eas_out,
                                             void* cuda_stream);

/* excp_decompress_tensor for callers that cannot allocate memory (the paper has no counterpart:
 * this is a property of the library, not of the method).
 *
 * It takes no handle and calls no allocating routine.  The little scratch memory that decoding
 * needs (survivor counts and offsets per 4096-element tile, the parsed header, an error flag) is
 * a fixed array inside the library's device image, which every GPU that loads the library holds
 * until the process ends (about 68 KB).  It is meant for restore paths that run where memory
 * cannot be requested: on a device that the training framework's own allocator has already
 * reserved in full, so that cudaMalloc fails, or where the device-wide synchronisation that
 * cudaMalloc / cudaFree imply must not happen because other streams are busy.
 *
 *   - Runs on the CURRENT device; all pointers are device memory of that device, 16-byte aligned.
 *     Arguments and results are those of excp_decompress_tensor (w_out may be w_prev).
 *   - numel may not exceed EXCP_NOALLOC_MAX_NUMEL; larger tensors return EXCP_ERR_INVALID_ARG
 *     before anything is launched (use a handle for those).
 *   - The first call on a device looks up the array's device address, and the first launch of each
 *     of its kernels makes the CUDA runtime load that kernel's code, which takes a little device
 *     memory once and may synchronise.  So make one warm-up call per device, with a non-empty
 *     tensor (every kernel then runs), while memory is still to be had and before any stream capture
 *     begins; the calls after it do nothing but launch.
 *   - All calls on a device share the one array, which keeps the previous call's contents; each
 *     call clears what it needs cleared.  Calls that overlap on the GPU (two streams, two
 *     threads) race on it: issue them one after the other.
 *   - Synchronises the stream; returns EXCP_ERR_CORRUPT_BLOB like excp_decompress_tensor. */
#define EXCP_NOALLOC_MAX_NUMEL (1u << 24)
excp_status excp_decompress_tensor_noalloc(const void* blob, size_t blob_bytes, const float* w_prev,
                                           size_t numel, float* w_out, float* ea_out, float* eas_out,
                                           void* cuda_stream);

/* Per-stage timing of the last compress/decompress call (no counterpart in the paper; the
 * stages are this library's kernels).  With timing enabled each call records CUDA events on
 * its stream between stages and, after its final synchronisation, sums the elapsed times per
 * stage.  The launch counter is kept whether or not timing is enabled.
 *   excp_profile_enable       turns event recording on (non-zero) or off; creates the events once.
 *   excp_profile_stage_count  number of stages; excp_profile_stage_name gives each a static name.
 *   excp_profile_read         stage_ms_out: host double[stage_count], milliseconds per stage of the
 *                             last call (may be NULL); launches_out: kernels launched by the last
 *                             call (may be NULL). */
excp_status excp_profile_enable(excp_handle h, int enable);
int excp_profile_stage_count(void);
const char* excp_profile_stage_name(int stage);
excp_status excp_profile_read(excp_handle h, double* stage_ms_out, unsigned long long* launches_out);

/* Switches the K-means objective in excp_tensor_stats (sse_w, sse_ea, sse_eas) on (non-zero) or off (the
 * default) for the handle's later compress calls. */
excp_status excp_set_report_sse(excp_handle h, int enable);

/* The bounded waits (no counterpart in the paper).  The dense sweeps stage their inputs in shared memory with
 * asynchronous bulk copies; a warp waits for a copy at most `nanoseconds` (default 2 s; a healthy copy lands
 * within microseconds).  When a wait runs out the warp raises the call's time-out flag, lets its other
 * copies land and leaves; every later kernel of the call then returns at once and the call returns
 * EXCP_ERR_TIMEOUT with the output buffers unspecified.  The handle stays usable.
 *   excp_set_wait_limit          sets the limit for the handle's later calls.
 *   excp_selftest_wait_timeout   exercises the error path on its own: one warp waits `nanoseconds` (at most
 *                                1e9) on a barrier that nothing will ever complete, so the wait always runs
 *                                out and the call returns EXCP_ERR_TIMEOUT; no copy is in flight at any
 *                                point.  Synchronises the stream. */
excp_status excp_set_wait_limit(excp_handle h, unsigned long long nanoseconds);
excp_status excp_selftest_wait_timeout(excp_handle h, unsigned long long nanoseconds, void* cuda_stream);

/* Tuning knob of the K-means stage (Section 3.3 leaves the implementation of K-means open; the
 * centres do not depend on this value).  The iterations need, per threshold between two centres,
 * the values of one narrow value cell.  The cells that all T iterations will visit are predicted
 * from per-cell counts and sums, and `margin` further cells on either side of every predicted one
 * are copied out as well (default 1).  A stream whose exact thresholds leave the copied cells
 * takes a second, complete round, which costs time but gives the same centres; margin = -1 copies
 * nothing in the first round, so every stream takes the second one.  margin >= -1, else
 * EXCP_ERR_INVALID_ARG.  Applies to the handle's later calls. */
excp_status excp_set_kmeans_margin(excp_handle h, int margin);

#ifdef __cplusplus
}
#endif
#endif /* EXCP_H_ */
