// Shared declarations of the library's translation units (not part of the public ABI).
#pragma once
#include <cuda_runtime.h>
#include <atomic>
#include <cstddef>
#include <cstdint>

#include "../../include/btard.h"

namespace btard {

// Per-partition constants the kernels read from the workspace.
struct PartEntry {
    long long len;   // number of real columns
    double tau;      // clip radius
};

// How one streaming pass is cut into CTAs.  A CTA is RG row groups x CL column lanes; a thread
// owns R consecutive rows of its group and 4 consecutive columns of every tile it visits.
struct Geometry {
    int R;        // rows per thread (compile-time choice, one of the instantiated values)
    int RG;       // row groups = ceil(n / R)
    int CL;       // column lanes (multiple of 32)
    int threads;  // RG * CL
    int cpp;      // CTAs per partition
    int slots;    // CTAs resident on the whole GPU at once
};

constexpr int kMaxTilesPerCta = 64;   // bounds the length of every fp32 running sum (256 terms)
// CenteredClip passes add one term per tile and row to a thread's fp32 running sums (the term is the
// sum of 4 squares), so twice as many tiles keep the sums as short.
constexpr int kMaxTilesPerPass = 128;

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Error bookkeeping (thread local).
void set_cuda_error(cudaError_t e);
void count_launch(int n = 1);

// Optional per-kernel timing (off by default): CUDA events around every launch of a kind.
enum KernelKind { KIND_MEDIAN = 0, KIND_INIT = 1, KIND_ITER = 2, KIND_VERIFY = 3, KIND_OTHER = 4,
                  KIND_GRAM = 5, KIND_COEF = 6, KIND_COMBINE = 7, KIND_COUNT = 8 };
void prof_begin(int kind, cudaStream_t st);
void prof_end(int kind, cudaStream_t st);
int sm_count();
// One bit per device ordinal: true until mark_device_done() has been called for the current device.
// Used to set kernel attributes once per device instead of on every call (setting them twice is
// harmless, so two threads racing here only repeat the work).
bool device_needs_setup(const std::atomic<unsigned long long>& seen);
void mark_device_done(std::atomic<unsigned long long>& seen);
// Writes {part_len[p], tau[p]} (tau == nullptr: 0) for p < P to a device table, as kernel arguments.
int upload_table(PartEntry* dev, int P, const int64_t* part_len, const double* tau, cudaStream_t st);

#define BTARD_CUDA_TRY(expr)                         \
    do {                                             \
        cudaError_t e__ = (expr);                    \
        if (e__ != cudaSuccess) {                    \
            ::btard::set_cuda_error(e__);            \
            return BTARD_ERR_CUDA;                   \
        }                                            \
    } while (0)

// ---- CenteredClip passes (btard_cclip.cu) -------------------------------------------------------
enum PassMode { PASS_INIT = 0, PASS_ITER = 1, PASS_NORMS = 2, PASS_COMBINE = 3 };

struct CclipLaunch {
    const float* g;
    float* v;                 // PASS_NORMS never writes it
    unsigned short* v_lo;     // device [P][stride] bf16 low-order part of v, or nullptr (plain fp32 v)
    const PartEntry* table;   // device [P]
    double* slots;            // device [P][cpp][n+1] per-CTA partial sums of the running pass
    const double* tot_in;     // device [P][n+1] totals of the previous pass
    double* tot_out;          // device [P][n+1] totals of this pass
    unsigned int* ticket;     // device [P] CTAs of the partition that have finished (0 between passes)
    const double* coef;       // device [P][n] combination coefficients (PASS_COMBINE)
    int* done;                // device [P]
    int32_t* iters;
    double* last_step;
    double* resid_norm;
    uint32_t* status;
    long long stride;
    int n, P;
    int l;                    // index of the update this pass applies (PASS_ITER)
    int stop_mode, max_iters;
    double eps2;
    int init_mode;            // PASS_INIT
    int rule;                 // BTARD_RULE_*: how the row weights follow from the norms
    int v_fits_l2;            // v (and its bf16 part) of all partitions takes at most 60 % of the L2
    const double* tau_sched;  // device [P][max_iters] radius of update l, or nullptr (the table's tau)
    const double* row_scale;  // device [P][n] factor applied to row i on load, or nullptr
};

// x scaled by a row factor; a factor of exactly 0 drops the row whatever it holds.  A NaN keeps its own
// bits: its sign decides at which end of a column's order it sits (coordinate median).
__device__ __forceinline__ float scale_value(float x, float f) { return (x == x) ? x * f : x; }
__device__ __forceinline__ float4 scale_row(float4 x, float f)
{
    if (f == 0.0f) return make_float4(0.f, 0.f, 0.f, 0.f);
    return make_float4(scale_value(x.x, f), scale_value(x.y, f), scale_value(x.z, f), scale_value(x.w, f));
}

Geometry cclip_geometry(int n, int P, long long stride);
int choose_ctas_per_partition(int P, long long quads, int CL, int slots, int max_tiles = kMaxTilesPerCta);
int launch_cclip_pass(const CclipLaunch& a, const Geometry& geo, int mode, cudaStream_t st);
int launch_cclip_finalize(const CclipLaunch& a, const Geometry& geo, cudaStream_t st);
// Median start and the start pass of the direct algorithm in one kernel (32 or 64 rows, no row factors).
bool median_norms_supported(int n, long long stride, const double* row_scale);
int launch_median_norms(const CclipLaunch& a, const Geometry& geo, cudaStream_t st);
// One cooperative launch that runs the start pass and every update of all partitions (work items =
// the CTAs of launch_cclip_pass, dealt round-robin to one wave of resident CTAs).  streaming != 0:
// the tensor does not fit L2 (evict-first loads, alternating sweep direction).
constexpr int kCoopMaxGrid = 148 * 8;
constexpr long long kCoopMaxItems = 1LL << 20;
int cooperative_launch_supported();
int launch_cclip_cooperative(const CclipLaunch& a, const Geometry& geo, int streaming, double* rslots,
                             unsigned long long* barrier, unsigned int* error, cudaStream_t st);
int launch_median_init(const float* g, float* v, const PartEntry* table, const double* row_scale,
                       long long stride, int n, int P, cudaStream_t st);
// squared-norm totals -> norms, used when verification is asked to compute the norms itself.
int launch_totals_to_norms(const double* tot, double* norm, int n, int P, cudaStream_t st);

// ---- Gram-matrix variant (btard_gram.cu) --------------------------------------------------------
struct GramGeometry {
    int NB;        // 8-row blocks = ceil(n / 8)
    int nblk;      // upper-triangular 8x8 blocks = NB (NB + 1) / 2
    int KG;        // column groups per CTA = 256 / nblk
    int NP;        // padded row count in shared memory (8 NB + 4)
    int TK;        // columns per tile
    int cpp;       // CTAs per partition
    int entries;   // doubles per Gram slot = 64 nblk
    size_t smem;   // dynamic shared memory of the Gram kernel
    int umma;      // 17 <= n <= 64 and the rows can be described by a tensor map: tcgen05 kernel
};
struct GramLaunch {
    const float* g;
    const float* v0;            // device [P][stride] centre of the Gram matrix
    float* v0_out;              // fuse_median: the same buffer, written by the Gram pass
    int fuse_median;            // n <= 16: the Gram pass takes the coordinate-wise median itself (v0 is an output)
    const PartEntry* table;
    double* slots;              // device [P][cpp][entries]
    double* gram;               // device [P][entries] summed blocks
    unsigned int* ticket;       // device [P]
    unsigned int* error;        // device: set when a bounded wait in the Gram kernel expired
    double* coef;               // device [P][n] out of the coefficient iteration
    int32_t* iters;
    double* last_step;
    uint32_t* status;
    long long stride;
    int n, P;
    int stop_mode, max_iters;
    double eps2;
    const double* tau_sched;    // device [P][max_iters] or nullptr
    const double* row_scale;    // device [P][n] or nullptr
};
GramGeometry gram_geometry(int n, int P, long long stride);
int launch_gram(const GramLaunch& a, const GramGeometry& geo, cudaStream_t st);
int launch_gram_iterate(const GramLaunch& a, const GramGeometry& geo, cudaStream_t st);
// resid_norm from the totals of the combine pass
int launch_gram_finalize(const double* tot, double* resid_norm, uint32_t* status, int n, int P,
                         const unsigned int* error, cudaStream_t st);

// ---- per-part gradient clipping (btard_preclip.cu) ----------------------------------------------
int preclip_chunks(int n, int P, long long stride);
// rewrite = false: norms and factors only, g untouched
int launch_preclip(float* g, const PartEntry* table, double* slots, double* row_norm, double* factor,
                   uint32_t* status, long long stride, int n, int P, int chunks, bool rewrite, cudaStream_t st);

// ---- Split / Merge copies (btard_pack.cu); table_dev: device {offset, len}[P] as two int64 each ---
int launch_split(const float* grads, float* g, const void* table_dev, long long d, long long stride,
                 int n, int P, cudaStream_t st);
int launch_merge(const float* v, float* out, const void* table_dev, long long stride, int P, cudaStream_t st);

// ---- commitments (btard_hash.cu): tree SHA-256 of every row of a [rows][stride] tensor ----------
int hash_max_leaves(long long stride);
int launch_hash_rows(const float* x, const PartEntry* table, uint32_t* leaves, unsigned char* out,
                     long long stride, int rows_per_part, int rows, cudaStream_t st);

// ---- verification (btard_verify.cu) -------------------------------------------------------------
struct VerifyLaunch {
    const float* g;
    const float* v;
    const PartEntry* table;
    const double* norm_in;    // device [P][n]
    double* part_out;         // device [P][cpp][slots]
    float* resid_sum;         // device [P][stride] or nullptr
    double *norm, *weight, *dot, *s, *s_sum, *znorm2, *resid_sum_norm;
    uint32_t* status;
    long long stride;
    int n, P, K, k0, kc;      // this launch covers z indices k0 .. k0+kc-1
    int p_base;
    uint32_t seed_lo, seed_hi;
    // Fused with the combine pass of the Gram variant: v holds v0 on entry and
    // receives v = v0 + sum_j coef_j (x_j - v0); the norms come out of this pass (norm_in is not read).
    int combine;
    float* v_out;                 // == v
    const double* coef;           // device [P][n]
    const double* gram;           // device [P][gram_entries] blocks of G = (g - v0)(g - v0)^T
    int gram_entries, gram_nb;
    double* resid_norm_out;       // device [P][n]: the aggregation's resid_norm output
    uint32_t* cclip_status;       // device [P]: the aggregation's status word (bits are OR-ed in)
    const unsigned int* gram_error;   // device: a bounded wait of the Gram kernel expired
    const double* row_scale;          // device [P][n] factor applied to row i on load, or nullptr
};

// Where entry (i, j) of a partition's Gram matrix sits: upper-triangular 8 x 8 blocks, NB = ceil(n / 8)
// blocks per side, a diagonal block stored whole.
__host__ __device__ inline int gram_entry_index(int NB, int i, int j)
{
    const int i0 = i < j ? i : j, j0 = i < j ? j : i;
    const int bi = i0 >> 3, bj = j0 >> 3;
    int blk = bj - bi;
    for (int q = 0; q < bi; ++q) blk += NB - q;
    return blk * 64 + (i0 & 7) * 8 + (j0 & 7);
}

struct VerifyGeometry {
    Geometry g;
    int KT;      // z vectors per launch (compile-time choice)
    int slots;   // doubles per CTA in part_out
    int own_z;   // n <= 16: each thread draws the z of its own columns (verify_rows_kernel)
};

// fused: the pass also carries the combine step of the Gram variant (its kernel may hold fewer CTAs per SM)
VerifyGeometry verify_geometry(int n, int P, long long stride, int K, bool fused = false);
int launch_verify(const VerifyLaunch& a, const VerifyGeometry& vg, cudaStream_t st);
int launch_checks(const btard_checks_args& a, cudaStream_t st);
int launch_random_vector(uint64_t seed, int p, int k, long long len, float* z, cudaStream_t st);

}  // namespace btard
