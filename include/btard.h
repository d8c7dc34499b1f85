/*
 * btard.h — C ABI of the batched CenteredClip + verification library for one NVIDIA B200.
 *
 * The library implements the arithmetic core of Byzantine-Tolerant All-Reduce (BTARD,
 * arXiv 2106.11257): the robust aggregation that replaces averaging in ButterflyClip
 * (Alg. 2, the ButterflyClip aggregation of every part) and the metadata of Verifications 1-2 (Alg. 6).  The n peers are rows of
 * one tensor in device memory; the P butterfly partitions are slabs of that tensor.
 *
 * Conventions
 *   - Tensor layout: g is [P][n][row_stride] float32, v is [P][row_stride] float32, both in
 *     device memory, 16-byte aligned, row_stride a multiple of 4.  Row i of slab p is peer i's
 *     part p.  Only the first part_len[p] columns of slab p are data; what lies beyond is ignored
 *     on input and written as 0 in v.
 *   - Every pointer marked "device" is owned by the caller and must stay valid until the work
 *     queued on `stream` has finished.  Pointers marked "host" are read before the call returns.
 *   - Calls that take device buffers are asynchronous on `stream` (a cudaStream_t passed as
 *     void*; NULL is the default stream).  They allocate nothing, on the device or on the host heap,
 *     copy nothing from pageable memory and never wait for the device: the small host arrays
 *     (part_len, tau) travel as arguments of a small kernel.  Scratch memory comes from `workspace`,
 *     sized by the matching *_workspace() query.  What such a call does on the host besides the
 *     launches: argument checks, a few device-attribute queries and, the first time a kernel is
 *     used on a device, setting its shared-memory attribute.
 *   - Return value: BTARD_OK, or a negative error.  Arguments and sizes (workspace included) are
 *     checked before anything is queued, so on INVALID_ARG, BAD_ALIGNMENT, WORKSPACE_TOO_SMALL and
 *     UNSUPPORTED nothing was queued.  BTARD_ERR_CUDA means a launch failed part-way: earlier
 *     launches of the call may already be on the stream and the outputs are undefined.  Conditions
 *     that only the device can see are reported per partition in `status` (BTARD_STATUS_* bits).
 */
#ifndef BTARD_H_
#define BTARD_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define BTARD_API __attribute__((visibility("default")))
#else
#define BTARD_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

#define BTARD_OK 0
#define BTARD_ERR_INVALID_ARG (-1)      /* NULL pointer, size out of range, tau < 0 or NaN ...   */
#define BTARD_ERR_BAD_ALIGNMENT (-2)    /* pointer not 16-byte aligned / row_stride % 4 != 0      */
#define BTARD_ERR_WORKSPACE_TOO_SMALL (-3)
#define BTARD_ERR_CUDA (-4)             /* a CUDA call failed; see btard_last_cuda_error()        */
#define BTARD_ERR_UNSUPPORTED (-5)      /* e.g. n_peers > BTARD_MAX_PEERS                          */

#define BTARD_MAX_PEERS 256
#define BTARD_MAX_Z 64

#define BTARD_SPLIT_PAPER 0     /* first d mod P parts have ceil(d/P) entries, the rest floor(d/P)  */
#define BTARD_SPLIT_CEIL_PAD 1  /* every part ceil(d/P) until d runs out; the tail part is short   */

#define BTARD_INIT_CALLER_V0 0      /* v holds v^0 on entry                                         */
#define BTARD_INIT_ZERO 1
#define BTARD_INIT_MEAN 2
#define BTARD_INIT_COORD_MEDIAN 3   /* coordinate-wise median of the n rows                         */

#define BTARD_ALGO_DIRECT 0         /* one pass over g per update, one kernel launch per update     */
#define BTARD_ALGO_GRAM 1           /* Gram matrix pass + iteration in coefficient space + combine  */
#define BTARD_ALGO_DIRECT_COOPERATIVE 2 /* as DIRECT, but all updates of all partitions inside one
                                       cooperative kernel: no launch per update and nothing runs
                                       after the last partition converged; where the device cannot
                                       launch it: DIRECT                                            */

/* Aggregation rule.  The paper's experiments (Sec. 4.1) compare CenteredClip with plain averaging,
   the coordinate-wise median and the geometric median; they run on the same streaming kernels. */
#define BTARD_RULE_CENTERED_CLIP 0     /* App. D.2 eq. (CenteredClip)                                 */
#define BTARD_RULE_GEOMETRIC_MEDIAN 1  /* Weiszfeld: v <- sum_i x_i/rho_i / sum_i 1/rho_i, rho_i =
                                          max(||x_i - v||, tau[p]): tau is the distance floor, > 0;
                                          same stop rules; DIRECT algorithms only                    */
#define BTARD_RULE_MEAN 2              /* v = (1/n) sum_i x_i, one pass, iters = 0                    */
#define BTARD_RULE_COORD_MEDIAN 3      /* coordinate-wise median, iters = 0                           */

#define BTARD_STOP_FIXED_ITERS 0    /* exactly max_iters updates                                    */
#define BTARD_STOP_EPS 1            /* stop once ||v^{l+1} - v^l||_2 <= eps, at most max_iters       */

#define BTARD_STATUS_NOT_CONVERGED 1u   /* EPS mode: max_iters reached with the last step > eps     */
#define BTARD_STATUS_NONFINITE_ROW 2u   /* a row with non-finite residual norm got weight 0         */
#define BTARD_STATUS_WAIT_EXPIRED 4u    /* a bounded wait inside a kernel ran out: results invalid  */

/*
 * Split(v, n) of App. D.1 ("Basic building blocks"): offsets and lengths of the P parts of a
 * vector of d coordinates, and the padded row length used to store one part.
 * Host only, pure, no CUDA.  part_offset, part_len: host arrays of P entries (out).
 * row_stride (out) = longest part rounded up to a multiple of align_elems (a multiple of 4).
 * Errors: INVALID_ARG for d < 0, P < 1, unknown mode, align_elems < 4 or not a multiple of 4.
 */
BTARD_API int btard_partition_layout(int64_t d, int32_t P, int32_t mode, int32_t align_elems,
                           int64_t* part_offset, int64_t* part_len, int64_t* row_stride);

/*
 * Commitments of Alg. 2 (hash(g_i[j]) and hash(g^_i), broadcast before the parts travel).
 * The paper asks only for "a cryptographic hash"; this library fixes SHA-256 (FIPS 180-4) in a two-level
 * tree so that one part is hashed by many threads:
 *     H(row) = SHA256( SHA256(chunk_0) || SHA256(chunk_1) || ... || LE64(byte length) ),
 * chunks = consecutive 4096-byte pieces of the row's first 4 * part_len bytes (float32 as stored).
 * x: device [P][rows_per_part][row_stride] — pass g with rows_per_part = n for the peers' parts, or v
 * with rows_per_part = 1 for the aggregates.  digests: device [P][rows_per_part][32] bytes out.
 * Workspace from btard_hash_partitions_workspace.  Asynchronous on `stream`.
 */
BTARD_API size_t btard_hash_partitions_workspace(int32_t n_partitions, int32_t rows_per_part, int64_t row_stride);
BTARD_API int btard_hash_partitions(int32_t n_partitions, int32_t rows_per_part, int64_t row_stride,
                                    const int64_t* part_len /* host [P] */, const float* x,
                                    uint8_t* digests, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Split and Merge of App. D.1 as device copies.  btard_split_gradients turns the n gradient vectors
 * grads [n][d] into the slab tensor g [P][n][row_stride] (row i of slab p = part p of peer i, padding
 * columns zero): with all peers on one GPU this is what the all-to-all of Alg. 2 (every peer sends part j to aggregator j) delivers.
 * btard_merge_partitions concatenates the aggregated parts v [P][row_stride] into out [d] (Alg. 2, Merge).
 * part_offset / part_len: host [P], as returned by btard_partition_layout or any P pairs with
 * 0 <= offset, len <= row_stride, offset + len <= d (slab q then holds coordinates offset[q] .. offset[q] +
 * len[q] - 1: a permutation of the parts gives a send buffer ordered by destination); table: device scratch
 * of 16 * P bytes.  All tensors device memory; asynchronous on `stream`.
 */
BTARD_API int btard_split_gradients(int64_t d, int32_t n_peers, int32_t n_partitions, int64_t row_stride,
                                    const int64_t* part_offset, const int64_t* part_len,
                                    const float* grads, float* g, void* table, void* stream);
BTARD_API int btard_merge_partitions(int64_t d, int32_t n_partitions, int64_t row_stride,
                                     const int64_t* part_offset, const int64_t* part_len,
                                     const float* v, float* out, void* table, void* stream);

/*
 * CenteredClip, App. D.2 eq. (CenteredClip), on all P partitions at once:
 *     v^{l+1} = v^l + (1/n) sum_i (x_i - v^l) min{1, tau / ||x_i - v^l||_2},   x_i = g[p][i][:].
 * A row whose residual norm is not finite takes weight 0 and is left out of the sum.
 */
typedef struct {
    int32_t n_peers;             /* n, 1..BTARD_MAX_PEERS                                           */
    int32_t n_partitions;        /* P >= 1                                                          */
    int64_t row_stride;          /* elements, multiple of 4                                         */
    const int64_t* part_len;     /* host [P], 0 <= part_len[p] <= row_stride                        */
    const float* g;              /* device [P][n][row_stride], read only                            */
    const double* tau;           /* host [P], clip radius per partition; >= 0, +inf allowed         */
    int32_t init_mode;           /* BTARD_INIT_*                                                    */
    int32_t algo;                /* BTARD_ALGO_*                                                    */
    int32_t stop_mode;           /* BTARD_STOP_*                                                    */
    int32_t max_iters;           /* >= 1                                                            */
    double eps;                  /* used in EPS mode, >= 0                                          */
    float* v;                    /* device [P][row_stride]; in: v^0 if CALLER_V0; out: result       */
    int32_t* iters;              /* device [P] out: updates applied                                 */
    double* last_step_norm;      /* device [P] out: ||v^{I} - v^{I-1}||_2                           */
    double* resid_norm;          /* device [P][n] out: ||x_i - v||_2 at the returned v              */
    uint32_t* status;            /* device [P] out: BTARD_STATUS_* bits                             */
    void* workspace;             /* device, 256-byte aligned                                        */
    size_t workspace_bytes;
    void* stream;                /* cudaStream_t                                                    */
    int32_t rule;                /* BTARD_RULE_*; 0 = CenteredClip                                  */
    const double* tau_schedule;  /* device [P][max_iters] or NULL: update l of partition p uses the radius
                                    tau_schedule[p][l] (the schedule tau_l of App. D.2) instead of tau[p];
                                    entries must be >= 0 (not checked: they live on the device)         */
    const double* row_scale;     /* device [P][n] or NULL: row i of slab p enters as row_scale[p][i] g[p][i][:],
                                    e.g. the factors of btard_preclip_factors (Alg. 9) - the clipped
                                    gradients are aggregated without rewriting g.  A factor of exactly 0
                                    makes the row read as zeros.  DIRECT and GRAM algorithms              */
} btard_cclip_args;

/* Bytes of workspace btard_centered_clip needs for these arguments (0 on invalid arguments).
   Reads only the sizes and modes, no pointer. */
BTARD_API size_t btard_centered_clip_workspace(const btard_cclip_args* args);
BTARD_API int btard_centered_clip(const btard_cclip_args* args);

/*
 * Verification metadata, Sec. 3.1 eq. (2) and Alg. 6 (norms, clip weights and projections each aggregator broadcasts), for all partitions:
 *     norm_i = ||g_i - v||_2,  w_i = min{1, tau/norm_i},
 *     dot_ik = <g_i - v, z_k>  with z_k = GetRandomVector(seed) restricted to partition p, unnormalised,
 *     s_ik   = w_i dot_ik / ||z_k||_2   (the paper's s_i^j = <z[j], Delta_i^j>),
 *     s_sum_k = sum_i s_ik,  resid_sum = sum_i w_i (g_i - v)   (both ~ 0 at the fixed point, eq. (1)).
 * z_k for partition p is keyed by (seed, partition_base + p, k); see btard_random_vector.
 */
typedef struct {
    int32_t n_peers;
    int32_t n_partitions;
    int64_t row_stride;
    const int64_t* part_len;     /* host [P]                                                        */
    const float* g;              /* device [P][n][row_stride]                                       */
    const float* v;              /* device [P][row_stride]: the aggregate as a peer received it     */
    const double* tau;           /* host [P]                                                        */
    uint64_t seed;               /* shared seed r (output of the multi-party generator)             */
    int32_t n_z;                 /* K, 1..BTARD_MAX_Z random vectors per partition                  */
    int32_t partition_base;      /* global index of slab 0 (0 unless the tensor is a shard)         */
    const double* resid_norm_in; /* device [P][n] norms at v (e.g. from btard_centered_clip) or NULL:
                                    NULL costs one more pass over g                                 */
    double* norm;                /* device [P][n] out                                               */
    double* weight;              /* device [P][n] out                                               */
    double* dot;                 /* device [P][n][K] out                                            */
    double* s;                   /* device [P][n][K] out                                            */
    double* s_sum;               /* device [P][K] out                                               */
    double* znorm2;              /* device [P][K] out: ||z_k||_2^2 over the part_len[p] coordinates */
    double* resid_sum_norm;      /* device [P] out: ||sum_i w_i (g_i - v)||_2                       */
    float* resid_sum;            /* device [P][row_stride] out, or NULL                             */
    uint32_t* status;            /* device [P] out                                                  */
    void* workspace;
    size_t workspace_bytes;
    void* stream;
    const double* row_scale;     /* device [P][n] or NULL: as in btard_cclip_args                   */
} btard_verify_args;

BTARD_API size_t btard_verify_projections_workspace(const btard_verify_args* args);
BTARD_API int btard_verify_projections(const btard_verify_args* args);

/*
 * Aggregation (Alg. 2) and verification metadata (Alg. 6) in one call: the same results as
 * btard_centered_clip(clip) followed by btard_verify_projections(verify) on the aggregate it returned.
 * `verify` supplies the seed, n_z, partition_base, its outputs and its own workspace; its g, v, part_len,
 * tau, row_scale, resid_norm_in and stream are taken from `clip` (what it holds there is ignored), and its n_peers,
 * n_partitions and row_stride must equal clip's.  Both workspaces are sized by the two *_workspace()
 * queries as for the separate calls.
 * What the one call buys: with BTARD_ALGO_GRAM the pass that forms v from the coefficients and the
 * verification pass are one read of g instead of two (the clip weights inside that pass come from the
 * Gram matrix, the reported norms and weights from the pass itself; they agree to rounding).  The other
 * algorithms run the two calls back to back.
 */
BTARD_API int btard_centered_clip_verify(const btard_cclip_args* clip, const btard_verify_args* verify);

/*
 * Per-part gradient clipping of BTARD-Clipped-SGD (Alg. 9 and the paragraph after it):
 *     g~_i(l) = min{1, lambda / ||g_i(l)||_2} g_i(l)
 * Two forms.  btard_preclip_factors reads g once and returns row_norm [P][n] = ||g_i(l)||_2 and
 * factor [P][n] = the multiplier min{1, lambda / ||g_i(l)||} (1 for a row inside the radius; 0 for a row
 * with a non-finite norm, flagged in status); g is not modified.  Handing `factor` to btard_centered_clip /
 * btard_verify_projections as `row_scale` aggregates the clipped gradients: one extra pass over g for a
 * Clipped-SGD aggregation.  btard_preclip does the same and then rescales the clipped rows IN PLACE (a row
 * with a non-finite norm is set to zero): a second pass, for callers that want g~ itself.
 * lambda: host [P] (the paper uses one lambda_k per step; per-part values are allowed), >= 0, +inf = no
 * clipping.
 */
typedef struct {
    int32_t n_peers, n_partitions;
    int64_t row_stride;
    const int64_t* part_len;     /* host [P] */
    const double* lambda;        /* host [P] */
    float* g;                    /* device [P][n][row_stride], modified in place */
    double* row_norm;            /* device [P][n] out */
    double* factor;              /* device [P][n] out */
    uint32_t* status;            /* device [P] out */
    void* workspace;             /* device, 256-byte aligned */
    size_t workspace_bytes;
    void* stream;
} btard_preclip_args;
BTARD_API size_t btard_preclip_workspace(const btard_preclip_args* args);
BTARD_API int btard_preclip(const btard_preclip_args* args);
BTARD_API int btard_preclip_factors(const btard_preclip_args* args);   /* same arguments and workspace; g is read only */

/*
 * The predicates of Verifications 1-3 (Alg. 6) on the scalars peers broadcast.  For
 * partition p (aggregated by peer p) and peer i:
 *   Verification 1: norm_mismatch[p][i] = reported norm_ip differs from ||g_i(p) - v(p)||;
 *   Verification 2: s_mismatch[p][i][k] = reported s_i^p differs from <z_k[p], Delta_i^p>;
 *                   sum_violation[p][k] = sum_i (reported s_i^p) != 0   ("v(p) is wrong");
 *   Verification 3: check[p][i] = ||g_i(p) - v(p)|| > Delta_max[p];  votes[p] = sum_i check[p][i];
 *                   check_averaging[p] = votes[p] > n/2  (then CheckAveraging(p) is due).
 * The paper compares exactly; here "differs" means |a - b| > rel_tol max(|a|, |b|) + abs_tol (NaN always
 * differs) and the sum test is |sum_i s| > sum_tol sum_i |s|, so that all-zero tolerances give the
 * paper's tests.  The library only evaluates the predicates; accusing and banning are the caller's.
 * `norm` and `s` are what btard_verify_projections computed; `norm_reported` / `s_reported` are what
 * the peers sent (either may be NULL: that test is skipped and, for the sum, the computed s is used).
 * All arrays are device memory; outputs are one byte per flag.  One small kernel on `stream`;
 * no workspace.
 */
typedef struct {
    int32_t n_peers, n_partitions, n_z;
    const double* norm;           /* device [P][n]    computed */
    const double* norm_reported;  /* device [P][n]    or NULL  */
    const double* s;              /* device [P][n][K] computed */
    const double* s_reported;     /* device [P][n][K] or NULL  */
    const double* delta_max;      /* device [P] (+inf or NaN: Verification 3 never fires) */
    double rel_tol, abs_tol, sum_tol;
    uint8_t* norm_mismatch;       /* device [P][n]    out */
    uint8_t* s_mismatch;          /* device [P][n][K] out */
    uint8_t* sum_violation;       /* device [P][K]    out */
    uint8_t* check;               /* device [P][n]    out */
    int32_t* votes;               /* device [P]       out */
    uint8_t* check_averaging;     /* device [P]       out */
    void* stream;
} btard_checks_args;
BTARD_API int btard_verification_checks(const btard_checks_args* args);

/*
 * btard_verify_projections without caller-supplied scratch.  The paper has no counterpart: this is
 * a packaging variant of the call above, same arguments, same kernels, same outputs.
 *
 * It is for callers that cannot give the library a workspace because they cannot allocate device
 * memory: a plug-in running inside a process whose framework has already claimed the whole GPU for
 * its own memory pool (cudaMalloc would fail), or a latency-critical loop that must never call
 * cudaMalloc / cudaFree because those may synchronise the device.  The caller still passes inputs
 * and outputs; `workspace` and `workspace_bytes` in the arguments are ignored.
 *
 * The scratch is a fixed array of BTARD_STATIC_SCRATCH_BYTES inside the library's device image; every
 * GPU that loads the library holds it until the process exits.  Problems whose scratch need exceeds
 * it (many partitions, very long rows, many z vectors) are refused with
 * BTARD_ERR_WORKSPACE_TOO_SMALL and nothing is queued; use btard_verify_projections for those.
 * The call allocates nothing, on the device or on the host heap.
 *
 * The first call on each device looks up the array's device address (one driver query, with that
 * device current; the result is kept per device ordinal for the life of the process, so it is stale
 * after a cudaDeviceReset).  Because that first call does this set-up, make it before any stream
 * capture is begun on that device.  All calls on one GPU share the array: calls that may overlap on the GPU
 * (other streams or threads) race on it and must be serialised by the caller.  Nothing needs to
 * persist in it between calls; what must start at zero is cleared on `stream` by each call.
 */
#define BTARD_STATIC_SCRATCH_BYTES (8 * 1024 * 1024)
BTARD_API int btard_verify_projections_static(const btard_verify_args* args);

/*
 * GetRandomVector (Alg. 6) made visible: writes the unnormalised float32 coordinates
 * z_k[0 .. part_len) of partition p to device memory (z_out, 16-byte aligned, room for
 * part_len rounded up to a multiple of 4).  Coordinates 4q..4q+3 are the Box-Muller images of the
 * four words of Philox4x32-10 with counter (q, p, k, 0x42544152) and key (seed low, seed high).
 * Bit-exact against the CPU oracle.  Asynchronous on `stream`.
 */
BTARD_API int btard_random_vector(uint64_t seed, int32_t p, int32_t k, int64_t part_len, float* z_out,
                        void* stream);

/*
 * The same aggregation + verification with HOST buffers: copies g to the device, runs
 * btard_centered_clip_verify with the algorithm in `algo`, copies the results back and waits for
 * `stream` (and for copy_stream, which only carries copies this call queued).  All device memory
 * comes from device_scratch (sized by btard_aggregate_host_scratch for the same n_peers, n_partitions,
 * row_stride, n_z and algo).  With BTARD_ALGO_DIRECT in EPS mode the updates run in the cooperative
 * kernel, so that nothing is launched after convergence (except with a coordinate-median start at 32
 * or 64 peers, where the launch-per-update path saves a pass over the rows and stays).
 * Host output pointers may be NULL to skip that copy, except v.  Pinned host memory makes the
 * copies asynchronous and fast; pageable memory works too.
 */
typedef struct {
    int32_t n_peers;
    int32_t n_partitions;
    int64_t row_stride;
    const int64_t* part_len;     /* host [P] */
    const double* tau;           /* host [P] */
    const float* g;              /* HOST [P][n][row_stride] */
    int32_t init_mode;           /* CALLER_V0: v holds v^0 on entry */
    int32_t stop_mode;
    int32_t max_iters;
    double eps;
    uint64_t seed;
    int32_t n_z;
    float* v;                    /* HOST [P][row_stride] out (in for CALLER_V0) */
    int32_t* iters;              /* HOST [P] out */
    double* last_step_norm;      /* HOST [P] out */
    double* norm;                /* HOST [P][n] out */
    double* weight;              /* HOST [P][n] out */
    double* dot;                 /* HOST [P][n][K] out */
    double* s;                   /* HOST [P][n][K] out */
    double* s_sum;               /* HOST [P][K] out */
    double* znorm2;              /* HOST [P][K] out */
    double* resid_sum_norm;      /* HOST [P] out */
    uint32_t* status;            /* HOST [P] out: OR of the two calls' status words */
    void* device_scratch;        /* device, 256-byte aligned */
    size_t device_scratch_bytes;
    void* stream;
    void* copy_stream;           /* optional second cudaStream_t (NULL: none).  When given and different
                                    from `stream`, the rows are copied in up to four chunks of partitions
                                    on it while the kernels of the previous chunk run on `stream`; g must
                                    then be pinned host memory for the overlap to happen.  The chunks
                                    change no result: partitions are independent.                      */
    int32_t algo;                /* BTARD_ALGO_DIRECT (0), BTARD_ALGO_GRAM or BTARD_ALGO_DIRECT_COOPERATIVE */
} btard_host_args;

BTARD_API size_t btard_aggregate_host_scratch(const btard_host_args* args);
BTARD_API int btard_aggregate_host(const btard_host_args* args);

/* The cudaError_t (as int) of the last failed CUDA call made by this thread inside the library. */
BTARD_API int btard_last_cuda_error(void);

/*
 * Optional per-kernel timing for benchmarks (no counterpart in the paper).  While enabled, every
 * streaming kernel the library launches is bracketed by CUDA events on the caller's stream.
 * btard_profile_collect waits for the recorded events, adds up elapsed milliseconds and launch counts
 * per kernel kind into total_ms[kind] / launches[kind] (host arrays of n_kinds >= 8 entries:
 * 0 median start, 1 init pass, 2 CenteredClip iteration pass, 3 verification pass, 4 other,
 * 5 Gram pass, 6 coefficient iteration, 7 combine pass) and
 * forgets them.  Process-wide state; not meant for concurrent use from several threads.
 */
BTARD_API void btard_profile_enable(int on);
BTARD_API int btard_profile_collect(double* total_ms, int64_t* launches, int32_t n_kinds);

/* Number of kernels the library has launched from this process so far (for accounting). */
BTARD_API int64_t btard_kernel_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* BTARD_H_ */
