// C ABI entry points: argument validation, workspace carving and the sequence of launches.
#include <atomic>
#include <cmath>
#include <cstring>
#include <mutex>
#include <vector>   // per-kernel timing records only (off by default)

#include "btard_common.h"

namespace btard {

static thread_local int g_last_cuda_error = 0;
static std::atomic<long long> g_launches{0};

void set_cuda_error(cudaError_t e) { g_last_cuda_error = (int)e; }
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

// ---- optional kernel timing ---------------------------------------------------------------------
// Size of the L2 cache of the current device in bytes (B200's when no device can be asked).
static long long l2_bytes()
{
    int dev = 0, l2 = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, dev) != cudaSuccess || l2 <= 0) {
        (void)cudaGetLastError();
        return 126LL << 20;
    }
    return l2;
}

namespace {
struct ProfRecord { int kind; cudaEvent_t a, b; };
std::mutex g_prof_mu;
bool g_prof_on = false;
std::vector<ProfRecord> g_prof_records;
std::vector<cudaEvent_t> g_prof_pool;
cudaEvent_t g_prof_open = nullptr;

cudaEvent_t prof_event()
{
    if (!g_prof_pool.empty()) { cudaEvent_t e = g_prof_pool.back(); g_prof_pool.pop_back(); return e; }
    cudaEvent_t e = nullptr;
    if (cudaEventCreate(&e) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
    return e;
}
}  // namespace

void prof_begin(int kind, cudaStream_t st)
{
    std::lock_guard<std::mutex> lk(g_prof_mu);
    if (!g_prof_on) return;
    g_prof_open = prof_event();
    if (g_prof_open) cudaEventRecord(g_prof_open, st);
}

void prof_end(int kind, cudaStream_t st)
{
    std::lock_guard<std::mutex> lk(g_prof_mu);
    if (!g_prof_on || !g_prof_open) return;
    cudaEvent_t b = prof_event();
    if (!b) { g_prof_pool.push_back(g_prof_open); g_prof_open = nullptr; return; }
    cudaEventRecord(b, st);
    g_prof_records.push_back(ProfRecord{kind, g_prof_open, b});
    g_prof_open = nullptr;
}

int sm_count()
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) {
        (void)cudaGetLastError();
        return 148;   // B200
    }
    return sms;
}

static unsigned long long device_bit()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { (void)cudaGetLastError(); return 0; }
    return 1ull << dev;
}
bool device_needs_setup(const std::atomic<unsigned long long>& seen)
{
    const unsigned long long bit = device_bit();
    return bit == 0 || !(seen.load(std::memory_order_acquire) & bit);
}
void mark_device_done(std::atomic<unsigned long long>& seen)
{
    seen.fetch_or(device_bit(), std::memory_order_release);
}

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_common(int n, int P, long long stride, const int64_t* part_len, const double* tau)
{
    if (n < 1 || P < 1 || P > 65535 || stride < 4 || !part_len || !tau) return BTARD_ERR_INVALID_ARG;
    if (n > BTARD_MAX_PEERS) return BTARD_ERR_UNSUPPORTED;
    if (stride % 4 != 0) return BTARD_ERR_BAD_ALIGNMENT;
    if (stride > (1LL << 33)) return BTARD_ERR_UNSUPPORTED;   // 32-bit Philox block index
    for (int p = 0; p < P; ++p) {
        if (part_len[p] < 0 || part_len[p] > stride) return BTARD_ERR_INVALID_ARG;
        if (!(tau[p] >= 0.0)) return BTARD_ERR_INVALID_ARG;   // rejects NaN too
    }
    return BTARD_OK;
}

struct CclipWorkspace {
    size_t table, slots, tot[2], flags, flags_bytes, v_lo, v_lo_bytes, total;
    size_t gslots, gram, coef;      // Gram variant only
    size_t rslots, rflags, rflags_bytes;   // cooperative variant only
};

constexpr int kMaxGramPeers = 128;

// EPS mode carries v as fp32 + a bf16 correction so that the stop test sees steps far below the
// rounding of v; FIXED mode needs no such thing.
CclipWorkspace cclip_ws_layout(int n, int P, long long stride, int stop_mode, int algo,
                               const Geometry& geo)
{
    CclipWorkspace w{};
    size_t off = 0;
    w.table = off; off = align_up(off + sizeof(PartEntry) * P, 256);
    const bool gram = (algo == BTARD_ALGO_GRAM);
    const bool comp = (stop_mode == BTARD_STOP_EPS && !gram);
    const int cpp = geo.cpp;
    w.slots = off; off = align_up(off + sizeof(double) * (size_t)P * cpp * (n + 1), 256);
    w.tot[0] = off; off = align_up(off + sizeof(double) * (size_t)P * (n + 1), 256);
    w.tot[1] = off; off = align_up(off + sizeof(double) * (size_t)P * (n + 1), 256);
    w.flags_bytes = sizeof(int) * (3 * (size_t)P + 1);        // done[P], ticket[P], Gram ticket[P], error
    w.flags = off; off = align_up(off + w.flags_bytes, 256);
    w.v_lo_bytes = comp ? sizeof(unsigned short) * (size_t)P * stride : 0;
    w.v_lo = off; off = align_up(off + w.v_lo_bytes, 256);
    if (gram && n <= kMaxGramPeers) {
        const GramGeometry gg = gram_geometry(n, P, stride);
        w.gslots = off; off = align_up(off + sizeof(double) * (size_t)P * gg.cpp * gg.entries, 256);
        w.gram = off; off = align_up(off + sizeof(double) * (size_t)P * gg.entries, 256);
        w.coef = off; off = align_up(off + sizeof(double) * (size_t)P * n, 256);
    }
    if (algo == BTARD_ALGO_DIRECT_COOPERATIVE) {
        w.rslots = off; off = align_up(off + sizeof(double) * 2 * (size_t)P * geo.cpp * (n + 1), 256);
        w.rflags_bytes = sizeof(unsigned long long) * 2;             // barrier word, error flag
        w.rflags = off; off = align_up(off + w.rflags_bytes, 256);
    }
    w.total = off;
    return w;
}

struct VerifyWorkspace {
    size_t table, part, norms, cslots, ctot, cticket, total;
};

// One layout serves the plain pass and the pass fused with the combine step: their CTA counts may
// differ, so the per-CTA slots are sized for the larger of the two.
VerifyWorkspace verify_ws_layout(int n, int P, long long stride, int K, const Geometry& cg)
{
    const VerifyGeometry plain = verify_geometry(n, P, stride, K, false), fused = verify_geometry(n, P, stride, K, true);
    const size_t ctas = (size_t)(plain.g.cpp > fused.g.cpp ? plain.g.cpp : fused.g.cpp);
    const size_t slots = (size_t)(plain.slots > fused.slots ? plain.slots : fused.slots);
    VerifyWorkspace w;
    size_t off = 0;
    w.table = off; off = align_up(off + sizeof(PartEntry) * P, 256);
    w.part = off; off = align_up(off + sizeof(double) * (size_t)P * ctas * slots, 256);
    w.norms = off; off = align_up(off + sizeof(double) * (size_t)P * n, 256);
    w.cslots = off; off = align_up(off + sizeof(double) * (size_t)P * cg.cpp * (n + 1), 256);
    w.ctot = off; off = align_up(off + sizeof(double) * (size_t)P * (n + 1), 256);
    w.cticket = off; off = align_up(off + sizeof(unsigned int) * (size_t)P, 256);
    w.total = off;
    return w;
}

// Small host tables (two 64-bit words per partition) reach the device as kernel arguments, a batch
// per launch: nothing is staged through pageable memory, nothing is allocated, and the launches are
// ordinary stream work.
constexpr int kPairBatch = 128;
struct PairBatch {
    unsigned long long w[2 * kPairBatch];
    int count;
};
__global__ void fill_pairs_kernel(unsigned long long* dst, const PairBatch b)
{
    const int i = threadIdx.x;
    if (i < 2 * b.count) dst[i] = b.w[i];
}

__global__ void or_status_kernel(uint32_t* dst, const uint32_t* other, int P)
{
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p < P) dst[p] |= other[p];
}

template <class Fill>   // fill(p, &w0, &w1)
int upload_pairs(void* dev, int P, cudaStream_t st, Fill fill)
{
    PairBatch b;
    for (int p0 = 0; p0 < P; p0 += kPairBatch) {
        b.count = (P - p0 < kPairBatch) ? P - p0 : kPairBatch;
        for (int q = 0; q < b.count; ++q) fill(p0 + q, &b.w[2 * q], &b.w[2 * q + 1]);
        fill_pairs_kernel<<<1, 2 * kPairBatch, 0, st>>>((unsigned long long*)dev + 2 * (size_t)p0, b);
        BTARD_CUDA_TRY(cudaGetLastError());
        count_launch();
    }
    return BTARD_OK;
}

}  // namespace

int upload_table(PartEntry* dev, int P, const int64_t* part_len, const double* tau, cudaStream_t st)
{
    static_assert(sizeof(PartEntry) == 16, "two 64-bit words per partition");
    return upload_pairs(dev, P, st, [&](int p, unsigned long long* w0, unsigned long long* w1) {
        const long long len = part_len[p];
        const double t = tau ? tau[p] : 0.0;
        std::memcpy(w0, &len, 8);
        std::memcpy(w1, &t, 8);
    });
}

}  // namespace btard

using namespace btard;

extern "C" {

int btard_last_cuda_error(void) { return g_last_cuda_error; }
int64_t btard_kernel_launch_count(void) { return (int64_t)g_launches.load(); }

void btard_profile_enable(int on)
{
    std::lock_guard<std::mutex> lk(g_prof_mu);
    g_prof_on = (on != 0);
}

int btard_profile_collect(double* total_ms, int64_t* launches, int32_t n_kinds)
{
    std::lock_guard<std::mutex> lk(g_prof_mu);
    if (!total_ms || !launches || n_kinds < KIND_COUNT) return BTARD_ERR_INVALID_ARG;
    for (int i = 0; i < n_kinds; ++i) { total_ms[i] = 0.0; launches[i] = 0; }
    int rc = BTARD_OK;
    for (const ProfRecord& r : g_prof_records) {
        float ms = 0.f;
        cudaError_t e = cudaEventSynchronize(r.b);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, r.a, r.b);
        if (e != cudaSuccess) { set_cuda_error(e); rc = BTARD_ERR_CUDA; }
        else { total_ms[r.kind] += ms; launches[r.kind] += 1; }
        g_prof_pool.push_back(r.a);
        g_prof_pool.push_back(r.b);
    }
    g_prof_records.clear();
    return rc;
}

int btard_partition_layout(int64_t d, int32_t P, int32_t mode, int32_t align_elems,
                           int64_t* part_offset, int64_t* part_len, int64_t* row_stride)
{
    if (d < 0 || P < 1 || align_elems < 4 || align_elems % 4 != 0) return BTARD_ERR_INVALID_ARG;
    if (!part_offset || !part_len || !row_stride) return BTARD_ERR_INVALID_ARG;
    if (mode != BTARD_SPLIT_PAPER && mode != BTARD_SPLIT_CEIL_PAD) return BTARD_ERR_INVALID_ARG;
    const int64_t base = d / P, extra = d % P, big = base + (extra != 0);
    int64_t at = 0, longest = 0;
    for (int32_t j = 0; j < P; ++j) {
        int64_t len;
        if (mode == BTARD_SPLIT_PAPER) len = base + (j < extra ? 1 : 0);
        else len = (d - at < big) ? d - at : big;
        part_offset[j] = at;
        part_len[j] = len;
        at += len;
        if (len > longest) longest = len;
    }
    if (longest == 0) longest = 1;
    *row_stride = (longest + align_elems - 1) / align_elems * align_elems;
    return BTARD_OK;
}

size_t btard_centered_clip_workspace(const btard_cclip_args* a)
{
    if (!a || a->n_peers < 1 || a->n_peers > BTARD_MAX_PEERS || a->n_partitions < 1 ||
        a->row_stride < 4)
        return 0;
    const Geometry geo = cclip_geometry(a->n_peers, a->n_partitions, a->row_stride);
    return cclip_ws_layout(a->n_peers, a->n_partitions, a->row_stride, a->stop_mode, a->algo, geo).total;
}

// The verification arguments of a fused call are usable, and the shape is one the fused pass covers.
static int check_verify_args(const btard_verify_args* a);
static bool fusable(const btard_cclip_args* c, const btard_verify_args* v)
{
    (void)v;
    return c->algo == BTARD_ALGO_GRAM && c->rule == BTARD_RULE_CENTERED_CLIP;
}
static int launch_fused_verify(const btard_cclip_args* c, const btard_verify_args* v, const PartEntry* table,
                               const double* coef, const double* gram, const GramGeometry& gg,
                               const unsigned int* gram_error, cudaStream_t st);

// fv != nullptr: the Gram variant ends after the coefficient iteration and the fused
// combine + verification pass follows (the caller has checked fusable()).
static int cclip_run(const btard_cclip_args* a, const btard_verify_args* fv)
{
    if (!a) return BTARD_ERR_INVALID_ARG;
    int rc = check_common(a->n_peers, a->n_partitions, a->row_stride, a->part_len, a->tau);
    if (rc != BTARD_OK) return rc;
    if (!a->g || !a->v || !a->iters || !a->last_step_norm || !a->resid_norm || !a->status ||
        !a->workspace)
        return BTARD_ERR_INVALID_ARG;
    if (a->max_iters < 1 || !(a->eps >= 0.0)) return BTARD_ERR_INVALID_ARG;
    if (a->init_mode < BTARD_INIT_CALLER_V0 || a->init_mode > BTARD_INIT_COORD_MEDIAN)
        return BTARD_ERR_INVALID_ARG;
    if (a->stop_mode != BTARD_STOP_FIXED_ITERS && a->stop_mode != BTARD_STOP_EPS)
        return BTARD_ERR_INVALID_ARG;
    if (a->algo != BTARD_ALGO_DIRECT && a->algo != BTARD_ALGO_GRAM && a->algo != BTARD_ALGO_DIRECT_COOPERATIVE)
        return BTARD_ERR_INVALID_ARG;
    if (a->algo == BTARD_ALGO_GRAM && a->n_peers > kMaxGramPeers) return BTARD_ERR_UNSUPPORTED;
    if (a->rule < BTARD_RULE_CENTERED_CLIP || a->rule > BTARD_RULE_COORD_MEDIAN) return BTARD_ERR_INVALID_ARG;
    if (a->rule != BTARD_RULE_CENTERED_CLIP && a->algo == BTARD_ALGO_GRAM) return BTARD_ERR_UNSUPPORTED;
    if (a->row_scale && a->algo == BTARD_ALGO_DIRECT_COOPERATIVE) return BTARD_ERR_UNSUPPORTED;
    if (a->rule == BTARD_RULE_GEOMETRIC_MEDIAN)
        for (int p = 0; p < a->n_partitions; ++p)
            if (!(a->tau[p] > 0.0) || std::isinf(a->tau[p])) return BTARD_ERR_INVALID_ARG;
    if (!aligned16(a->g) || !aligned16(a->v) || (reinterpret_cast<uintptr_t>(a->workspace) & 255u))
        return BTARD_ERR_BAD_ALIGNMENT;

    const int n = a->n_peers, P = a->n_partitions;
    const Geometry geo = cclip_geometry(n, P, a->row_stride);
    const CclipWorkspace ws = cclip_ws_layout(n, P, a->row_stride, a->stop_mode, a->algo, geo);
    if (a->workspace_bytes < ws.total) return BTARD_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)a->stream;
    char* base = (char*)a->workspace;

    CclipLaunch L{};
    L.g = a->g; L.v = a->v;
    L.table = (const PartEntry*)(base + ws.table);
    L.done = (int*)(base + ws.flags);
    L.ticket = (unsigned int*)(base + ws.flags) + P;
    L.slots = (double*)(base + ws.slots);
    L.iters = a->iters; L.last_step = a->last_step_norm; L.resid_norm = a->resid_norm;
    L.status = a->status;
    L.stride = a->row_stride; L.n = n; L.P = P;
    L.stop_mode = a->stop_mode; L.max_iters = a->max_iters; L.eps2 = a->eps * a->eps;
    L.rule = a->rule;
    L.tau_sched = a->tau_schedule; L.row_scale = a->row_scale;
    double* tot[2] = {(double*)(base + ws.tot[0]), (double*)(base + ws.tot[1])};

    rc = upload_table((PartEntry*)(base + ws.table), P, a->part_len, a->tau, st);
    if (rc != BTARD_OK) return rc;
    BTARD_CUDA_TRY(cudaMemsetAsync(base + ws.flags, 0, ws.flags_bytes, st));
    if (ws.v_lo_bytes) {
        L.v_lo = (unsigned short*)(base + ws.v_lo);
        BTARD_CUDA_TRY(cudaMemsetAsync(L.v_lo, 0, ws.v_lo_bytes, st));
    }
    L.v_fits_l2 = (double)P * (double)a->row_stride * (L.v_lo ? 6.0 : 4.0) <= 0.6 * (double)l2_bytes();

    // Init pass: v^0 and the residual norms at v^0 (slot buffer 0).
    if (a->rule == BTARD_RULE_MEAN || a->rule == BTARD_RULE_COORD_MEDIAN) {
        L.init_mode = BTARD_INIT_MEAN;
        if (a->rule == BTARD_RULE_COORD_MEDIAN) {
            rc = launch_median_init(a->g, a->v, L.table, a->row_scale, a->row_stride, n, P, st);
            if (rc != BTARD_OK) return rc;
            L.init_mode = BTARD_INIT_CALLER_V0;
        }
        L.tot_in = nullptr; L.tot_out = tot[0]; L.l = 0;
        rc = launch_cclip_pass(L, geo, PASS_INIT, st);          // v and the residual norms at v
        if (rc != BTARD_OK) return rc;
        L.tot_in = tot[0]; L.max_iters = 0; L.stop_mode = BTARD_STOP_FIXED_ITERS;
        return launch_cclip_finalize(L, geo, st);
    }

    // How the updates are driven: one cooperative kernel over everything, or one launch per update.
    const bool whole = (a->algo == BTARD_ALGO_DIRECT_COOPERATIVE) && cooperative_launch_supported();
    L.init_mode = a->init_mode;
    // up to 16 peers the Gram pass takes the median start itself (every row of a column sits in one thread)
    const bool gram_takes_median = (a->algo == BTARD_ALGO_GRAM && a->init_mode == BTARD_INIT_COORD_MEDIAN && n <= 16);
    // 32 or 64 peers, launch-per-update path: the median start and the start pass are one kernel
    const bool fused_start = (a->algo == BTARD_ALGO_DIRECT && a->init_mode == BTARD_INIT_COORD_MEDIAN &&
                              median_norms_supported(n, a->row_stride, a->row_scale));
    if (a->init_mode == BTARD_INIT_COORD_MEDIAN && !gram_takes_median && !fused_start) {
        rc = launch_median_init(a->g, a->v, L.table, a->row_scale, a->row_stride, n, P, st);
        if (rc != BTARD_OK) return rc;
        L.init_mode = BTARD_INIT_CALLER_V0;
    }
    L.tot_in = nullptr; L.tot_out = tot[0]; L.l = 0;
    if (a->algo == BTARD_ALGO_GRAM) {
        // v <- v0 (a median start is already in v), G = (g - v0)(g - v0)^T, iterate on coefficients,
        // then one pass forms v and the residual norms at v.
        if (a->init_mode != BTARD_INIT_COORD_MEDIAN && a->init_mode != BTARD_INIT_CALLER_V0) {
            rc = launch_cclip_pass(L, geo, PASS_INIT, st);
            if (rc != BTARD_OK) return rc;
        }
        const GramGeometry gg = gram_geometry(n, P, a->row_stride);
        GramLaunch G{};
        G.g = a->g; G.v0 = a->v; G.v0_out = a->v; G.fuse_median = gram_takes_median ? 1 : 0; G.table = L.table;
        G.slots = (double*)(base + ws.gslots); G.gram = (double*)(base + ws.gram);
        G.ticket = (unsigned int*)(base + ws.flags) + 2 * P;
        G.error = (unsigned int*)(base + ws.flags) + 3 * P;
        G.coef = (double*)(base + ws.coef);
        G.iters = a->iters; G.last_step = a->last_step_norm; G.status = a->status;
        G.stride = a->row_stride; G.n = n; G.P = P;
        G.stop_mode = a->stop_mode; G.max_iters = a->max_iters; G.eps2 = a->eps * a->eps;
        G.tau_sched = a->tau_schedule; G.row_scale = a->row_scale;
        rc = launch_gram(G, gg, st);
        if (rc != BTARD_OK) return rc;
        rc = launch_gram_iterate(G, gg, st);
        if (rc != BTARD_OK) return rc;
        if (fv) return launch_fused_verify(a, fv, L.table, G.coef, G.gram, gg, G.error, st);
        L.coef = G.coef;
        rc = launch_cclip_pass(L, geo, PASS_COMBINE, st);
        if (rc != BTARD_OK) return rc;
        return launch_gram_finalize(L.tot_out, a->resid_norm, a->status, n, P, G.error, st);
    }
    if (whole) {
        BTARD_CUDA_TRY(cudaMemsetAsync(base + ws.rflags, 0, ws.rflags_bytes, st));
        unsigned long long* bar = (unsigned long long*)(base + ws.rflags);
        unsigned int* err = (unsigned int*)(bar + 1);
        // rows + v (fp32 and bf16) of all partitions against three quarters of the L2
        const bool fits = (double)P * (double)a->row_stride * (4.0 * n + 6.0) <= 0.75 * (double)l2_bytes();
        rc = launch_cclip_cooperative(L, geo, fits ? 0 : 1, (double*)(base + ws.rslots), bar, err, st);
        if (rc == BTARD_OK) return BTARD_OK;
        // the cooperative launch was refused: nothing ran, take the launch-per-update path
    }

    rc = fused_start ? launch_median_norms(L, geo, st) : launch_cclip_pass(L, geo, PASS_INIT, st);
    if (rc != BTARD_OK) return rc;

    // Update l reads the totals in buffer l % 2 and writes buffer (l + 1) % 2.
    for (int l = 0; l < a->max_iters; ++l) {
        L.l = l; L.tot_in = tot[l & 1]; L.tot_out = tot[(l + 1) & 1];
        rc = launch_cclip_pass(L, geo, PASS_ITER, st);
        if (rc != BTARD_OK) return rc;
    }
    L.tot_in = tot[a->max_iters & 1];
    return launch_cclip_finalize(L, geo, st);
}

int btard_centered_clip(const btard_cclip_args* a) { return cclip_run(a, nullptr); }

size_t btard_verify_projections_workspace(const btard_verify_args* a)
{
    if (!a || a->n_peers < 1 || a->n_peers > BTARD_MAX_PEERS || a->n_partitions < 1 ||
        a->row_stride < 4 || a->n_z < 1)
        return 0;
    const Geometry cg = cclip_geometry(a->n_peers, a->n_partitions, a->row_stride);
    return verify_ws_layout(a->n_peers, a->n_partitions, a->row_stride, a->n_z, cg).total;
}

static int check_verify_args(const btard_verify_args* a)
{
    if (!a) return BTARD_ERR_INVALID_ARG;
    int rc = check_common(a->n_peers, a->n_partitions, a->row_stride, a->part_len, a->tau);
    if (rc != BTARD_OK) return rc;
    if (!a->g || !a->v || !a->norm || !a->weight || !a->dot || !a->s || !a->s_sum || !a->znorm2 ||
        !a->resid_sum_norm || !a->status || !a->workspace)
        return BTARD_ERR_INVALID_ARG;
    if (a->n_z < 1 || a->n_z > BTARD_MAX_Z || a->partition_base < 0) return BTARD_ERR_INVALID_ARG;
    if (!aligned16(a->g) || !aligned16(a->v) || (a->resid_sum && !aligned16(a->resid_sum)) ||
        (reinterpret_cast<uintptr_t>(a->workspace) & 255u))
        return BTARD_ERR_BAD_ALIGNMENT;
    return BTARD_OK;
}

// The combine pass of the Gram variant and the verification pass as one kernel over the rows.
static int launch_fused_verify(const btard_cclip_args* c, const btard_verify_args* a, const PartEntry* table,
                               const double* coef, const double* gram, const GramGeometry& gg,
                               const unsigned int* gram_error, cudaStream_t st)
{
    const int n = c->n_peers, P = c->n_partitions, K = a->n_z;
    const VerifyGeometry vg = verify_geometry(n, P, c->row_stride, K, true);
    const Geometry cg = cclip_geometry(n, P, c->row_stride);
    const VerifyWorkspace ws = verify_ws_layout(n, P, c->row_stride, K, cg);
    if (a->workspace_bytes < ws.total) return BTARD_ERR_WORKSPACE_TOO_SMALL;
    char* base = (char*)a->workspace;
    VerifyLaunch V{};
    V.g = c->g; V.v = c->v; V.v_out = c->v; V.table = table; V.norm_in = nullptr;
    V.part_out = (double*)(base + ws.part);
    V.resid_sum = a->resid_sum;
    V.norm = a->norm; V.weight = a->weight; V.dot = a->dot; V.s = a->s; V.s_sum = a->s_sum;
    V.znorm2 = a->znorm2; V.resid_sum_norm = a->resid_sum_norm; V.status = a->status;
    V.stride = c->row_stride; V.n = n; V.P = P; V.K = K; V.p_base = a->partition_base;
    V.seed_lo = (uint32_t)a->seed; V.seed_hi = (uint32_t)(a->seed >> 32);
    V.coef = coef; V.gram = gram; V.gram_entries = gg.entries; V.gram_nb = gg.NB;
    V.resid_norm_out = c->resid_norm; V.cclip_status = c->status; V.gram_error = gram_error;
    V.row_scale = c->row_scale;
    // The first group of directions carries the combine; further groups (K beyond what one launch
    // holds) are plain verification launches on the v and the norms the first one left.
    for (int k0 = 0; k0 < K; k0 += vg.KT) {
        V.k0 = k0;
        V.kc = (K - k0 < vg.KT) ? K - k0 : vg.KT;
        V.combine = (k0 == 0) ? 1 : 0;
        V.norm_in = (k0 == 0) ? nullptr : c->resid_norm;
        const int rc = launch_verify(V, vg, st);
        if (rc != BTARD_OK) return rc;
    }
    return BTARD_OK;
}

int btard_centered_clip_verify(const btard_cclip_args* c, const btard_verify_args* v)
{
    if (!c || !v) return BTARD_ERR_INVALID_ARG;
    if (v->n_peers != c->n_peers || v->n_partitions != c->n_partitions || v->row_stride != c->row_stride)
        return BTARD_ERR_INVALID_ARG;
    // the verification reads what the aggregation produced, on the same stream
    btard_verify_args vv = *v;
    vv.g = c->g; vv.v = c->v; vv.part_len = c->part_len; vv.tau = c->tau; vv.row_scale = c->row_scale;
    vv.resid_norm_in = c->resid_norm; vv.stream = c->stream;
    int rc = check_verify_args(&vv);
    if (rc != BTARD_OK) return rc;
    if (fusable(c, &vv)) {
        const Geometry cg = cclip_geometry(c->n_peers, c->n_partitions, c->row_stride);
        if (vv.workspace_bytes < verify_ws_layout(c->n_peers, c->n_partitions, c->row_stride, vv.n_z, cg).total)
            return BTARD_ERR_WORKSPACE_TOO_SMALL;   // before anything is queued
        return cclip_run(c, &vv);
    }
    rc = cclip_run(c, nullptr);
    if (rc != BTARD_OK) return rc;
    return btard_verify_projections(&vv);
}

int btard_verify_projections(const btard_verify_args* a)
{
    int rc = check_verify_args(a);
    if (rc != BTARD_OK) return rc;

    const int n = a->n_peers, P = a->n_partitions, K = a->n_z;
    const VerifyGeometry vg = verify_geometry(n, P, a->row_stride, K);
    const Geometry cg = cclip_geometry(n, P, a->row_stride);
    const VerifyWorkspace ws = verify_ws_layout(n, P, a->row_stride, K, cg);
    if (a->workspace_bytes < ws.total) return BTARD_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)a->stream;
    char* base = (char*)a->workspace;
    PartEntry* table = (PartEntry*)(base + ws.table);
    rc = upload_table(table, P, a->part_len, a->tau, st);
    if (rc != BTARD_OK) return rc;

    const double* norms = a->resid_norm_in;
    if (!norms) {   // one more pass: residual norms at v
        CclipLaunch L{};
        L.g = a->g; L.v = const_cast<float*>(a->v); L.table = table;
        L.slots = (double*)(base + ws.cslots);
        L.tot_out = (double*)(base + ws.ctot);
        L.ticket = (unsigned int*)(base + ws.cticket);
        BTARD_CUDA_TRY(cudaMemsetAsync(L.ticket, 0, sizeof(unsigned int) * (size_t)P, st));
        L.stride = a->row_stride; L.n = n; L.P = P; L.row_scale = a->row_scale;
        rc = launch_cclip_pass(L, cg, PASS_NORMS, st);
        if (rc != BTARD_OK) return rc;
        rc = launch_totals_to_norms(L.tot_out, (double*)(base + ws.norms), n, P, st);
        if (rc != BTARD_OK) return rc;
        norms = (const double*)(base + ws.norms);
    }

    VerifyLaunch V{};
    V.g = a->g; V.v = a->v; V.table = table; V.norm_in = norms;
    V.part_out = (double*)(base + ws.part);
    V.resid_sum = a->resid_sum;
    V.norm = a->norm; V.weight = a->weight; V.dot = a->dot; V.s = a->s; V.s_sum = a->s_sum;
    V.znorm2 = a->znorm2; V.resid_sum_norm = a->resid_sum_norm; V.status = a->status;
    V.stride = a->row_stride; V.n = n; V.P = P; V.K = K; V.p_base = a->partition_base;
    V.seed_lo = (uint32_t)a->seed; V.seed_hi = (uint32_t)(a->seed >> 32);
    V.row_scale = a->row_scale;
    for (int k0 = 0; k0 < K; k0 += vg.KT) {
        V.k0 = k0;
        V.kc = (K - k0 < vg.KT) ? K - k0 : vg.KT;
        rc = launch_verify(V, vg, st);
        if (rc != BTARD_OK) return rc;
    }
    return BTARD_OK;
}

namespace {
int upload_pack_table(void* table, int P, int64_t d, int64_t stride, const int64_t* off, const int64_t* len,
                      cudaStream_t st)
{
    if (P < 1 || P > 65535 || !off || !len || !table || d < 0 || stride < 1) return BTARD_ERR_INVALID_ARG;
    for (int p = 0; p < P; ++p)
        if (off[p] < 0 || len[p] < 0 || len[p] > stride || off[p] + len[p] > d) return BTARD_ERR_INVALID_ARG;
    return upload_pairs(table, P, st, [&](int p, unsigned long long* w0, unsigned long long* w1) {
        const long long o = off[p], l = len[p];
        std::memcpy(w0, &o, 8);
        std::memcpy(w1, &l, 8);
    });
}
}  // namespace

int btard_split_gradients(int64_t d, int32_t n, int32_t P, int64_t stride, const int64_t* off,
                          const int64_t* len, const float* grads, float* g, void* table, void* stream)
{
    if (n < 1 || !grads || !g) return BTARD_ERR_INVALID_ARG;
    int rc = upload_pack_table(table, P, d, stride, off, len, (cudaStream_t)stream);
    if (rc != BTARD_OK) return rc;
    return launch_split(grads, g, table, d, stride, n, P, (cudaStream_t)stream);
}

int btard_merge_partitions(int64_t d, int32_t P, int64_t stride, const int64_t* off, const int64_t* len,
                           const float* v, float* out, void* table, void* stream)
{
    if (!v || !out) return BTARD_ERR_INVALID_ARG;
    int rc = upload_pack_table(table, P, d, stride, off, len, (cudaStream_t)stream);
    if (rc != BTARD_OK) return rc;
    return launch_merge(v, out, table, stride, P, (cudaStream_t)stream);
}

size_t btard_hash_partitions_workspace(int32_t P, int32_t rows_per_part, int64_t stride)
{
    if (P < 1 || rows_per_part < 1 || stride < 1) return 0;
    return align_up(sizeof(PartEntry) * (size_t)P, 256) +
           align_up(sizeof(uint32_t) * 8 * (size_t)P * rows_per_part * hash_max_leaves(stride), 256);
}

int btard_hash_partitions(int32_t P, int32_t rows_per_part, int64_t stride, const int64_t* part_len,
                          const float* x, uint8_t* digests, void* workspace, size_t workspace_bytes,
                          void* stream)
{
    if (P < 1 || rows_per_part < 1 || stride < 1 || !part_len || !x || !digests || !workspace)
        return BTARD_ERR_INVALID_ARG;
    if ((long long)P * rows_per_part > 0x7fffffffLL / 2) return BTARD_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return BTARD_ERR_BAD_ALIGNMENT;
    if (workspace_bytes < btard_hash_partitions_workspace(P, rows_per_part, stride)) return BTARD_ERR_WORKSPACE_TOO_SMALL;
    for (int p = 0; p < P; ++p)
        if (part_len[p] < 0 || part_len[p] > stride) return BTARD_ERR_INVALID_ARG;
    char* base = (char*)workspace;
    int rc = upload_table((PartEntry*)base, P, part_len, nullptr, (cudaStream_t)stream);
    if (rc != BTARD_OK) return rc;
    uint32_t* leaves = (uint32_t*)(base + align_up(sizeof(PartEntry) * (size_t)P, 256));
    return launch_hash_rows(x, (const PartEntry*)base, leaves, digests, stride, rows_per_part,
                            P * rows_per_part, (cudaStream_t)stream);
}

size_t btard_preclip_workspace(const btard_preclip_args* a)
{
    if (!a || a->n_peers < 1 || a->n_peers > BTARD_MAX_PEERS || a->n_partitions < 1 || a->row_stride < 4)
        return 0;
    const int chunks = preclip_chunks(a->n_peers, a->n_partitions, a->row_stride);
    return align_up(sizeof(PartEntry) * (size_t)a->n_partitions, 256) +
           align_up(sizeof(double) * (size_t)a->n_peers * a->n_partitions * chunks, 256);
}

static int preclip_run(const btard_preclip_args* a, bool rewrite)
{
    if (!a) return BTARD_ERR_INVALID_ARG;
    int rc = check_common(a->n_peers, a->n_partitions, a->row_stride, a->part_len, a->lambda);
    if (rc != BTARD_OK) return rc;
    if (!a->g || !a->row_norm || !a->factor || !a->status || !a->workspace) return BTARD_ERR_INVALID_ARG;
    if (!aligned16(a->g) || (reinterpret_cast<uintptr_t>(a->workspace) & 255u)) return BTARD_ERR_BAD_ALIGNMENT;
    if (a->workspace_bytes < btard_preclip_workspace(a)) return BTARD_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)a->stream;
    char* base = (char*)a->workspace;
    PartEntry* table = (PartEntry*)base;
    rc = upload_table(table, a->n_partitions, a->part_len, a->lambda, st);    // lambda rides in the tau field
    if (rc != BTARD_OK) return rc;
    double* slots = (double*)(base + align_up(sizeof(PartEntry) * (size_t)a->n_partitions, 256));
    const int chunks = preclip_chunks(a->n_peers, a->n_partitions, a->row_stride);
    return launch_preclip(a->g, table, slots, a->row_norm, a->factor, a->status, a->row_stride,
                          a->n_peers, a->n_partitions, chunks, rewrite, st);
}

int btard_preclip(const btard_preclip_args* a) { return preclip_run(a, true); }
int btard_preclip_factors(const btard_preclip_args* a) { return preclip_run(a, false); }

int btard_verification_checks(const btard_checks_args* a)
{
    if (!a || a->n_peers < 1 || a->n_partitions < 1 || a->n_partitions > 65535 || a->n_z < 1)
        return BTARD_ERR_INVALID_ARG;
    if (a->n_peers > BTARD_MAX_PEERS || a->n_z > BTARD_MAX_Z) return BTARD_ERR_UNSUPPORTED;
    if (!a->norm || !a->s || !a->delta_max || !a->norm_mismatch || !a->s_mismatch || !a->sum_violation ||
        !a->check || !a->votes || !a->check_averaging)
        return BTARD_ERR_INVALID_ARG;
    if (!(a->rel_tol >= 0.0) || !(a->abs_tol >= 0.0) || !(a->sum_tol >= 0.0)) return BTARD_ERR_INVALID_ARG;
    return launch_checks(*a, (cudaStream_t)a->stream);
}

int btard_random_vector(uint64_t seed, int32_t p, int32_t k, int64_t part_len, float* z_out,
                        void* stream)
{
    if (p < 0 || k < 0 || part_len < 0 || (part_len > 0 && !z_out)) return BTARD_ERR_INVALID_ARG;
    if (part_len > (1LL << 33)) return BTARD_ERR_UNSUPPORTED;
    if (!aligned16(z_out)) return BTARD_ERR_BAD_ALIGNMENT;
    return launch_random_vector(seed, p, k, part_len, z_out, (cudaStream_t)stream);
}

// ---- host-buffer path ---------------------------------------------------------------------------
namespace {
// With a second stream the partitions go through in up to kMaxHostChunks chunks: the copy of the
// next chunk's rows runs on copy_stream while the kernels of the current chunk run on stream, so
// the call takes about the longer of (copy of everything) and (all kernels) plus one chunk of the other.
// Every chunk pays the fixed cost of its updates (a launch or a grid barrier each) again: measured on
// 16 partitions of 16 x 698 400 with 100 updates, 4 chunks take 19.6 ms and 8 chunks 23.1 ms.
constexpr size_t kMaxHostChunks = 4;

struct HostScratch {
    size_t g, v, iters, last_step, resid_norm, status_c, status_v, norm, weight, dot, s, s_sum,
        znorm2, rsn, ws_c, ws_v, total;
    size_t ws_c_bytes, ws_v_bytes;
};

bool host_piped(const btard_host_args* a)
{
    return a->copy_stream != nullptr && a->copy_stream != a->stream && a->n_partitions > 1;
}
size_t host_chunks(const btard_host_args* a)
{
    const size_t P = (size_t)a->n_partitions;
    return host_piped(a) ? (P < kMaxHostChunks ? P : kMaxHostChunks) : 1;
}
// The algorithm a chunk runs: in eps mode the launch-per-update path would keep launching after the
// chunk has converged, so DIRECT becomes the cooperative kernel there, unless the launch-per-update path
// saves a whole pass with its fused median start (32 or 64 peers: 10.0 against 11.3 ms on 64 x 64 x 276 320).
int host_algo(const btard_host_args* a)
{
    if (a->algo == BTARD_ALGO_DIRECT && a->stop_mode == BTARD_STOP_EPS &&
        !(a->init_mode == BTARD_INIT_COORD_MEDIAN && median_norms_supported(a->n_peers, a->row_stride, nullptr)))
        return BTARD_ALGO_DIRECT_COOPERATIVE;
    return a->algo;
}

HostScratch host_layout(const btard_host_args* a)
{
    HostScratch h{};
    const size_t n = a->n_peers, P = a->n_partitions, S = (size_t)a->row_stride, K = a->n_z;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off = align_up(off + bytes, 256); return at; };
    h.g = take(sizeof(float) * P * n * S);
    h.v = take(sizeof(float) * P * S);
    h.iters = take(sizeof(int32_t) * P);
    h.last_step = take(sizeof(double) * P);
    h.resid_norm = take(sizeof(double) * P * n);
    h.status_c = take(sizeof(uint32_t) * P);
    h.status_v = take(sizeof(uint32_t) * P);
    h.norm = take(sizeof(double) * P * n);
    h.weight = take(sizeof(double) * P * n);
    h.dot = take(sizeof(double) * P * n * K);
    h.s = take(sizeof(double) * P * n * K);
    h.s_sum = take(sizeof(double) * P * K);
    h.znorm2 = take(sizeof(double) * P * K);
    h.rsn = take(sizeof(double) * P);
    // The workspaces serve every chunk in turn.  Their layouts are not monotone in the number of
    // partitions (fewer partitions get more CTAs each), so the size is the largest need over every
    // chunk size this call may use, with or without a copy stream.
    btard_cclip_args ca{};
    ca.n_peers = a->n_peers; ca.row_stride = a->row_stride;
    ca.stop_mode = BTARD_STOP_EPS;   // the larger of the two layouts
    ca.algo = (a->algo == BTARD_ALGO_GRAM) ? BTARD_ALGO_GRAM : BTARD_ALGO_DIRECT_COOPERATIVE;
    btard_verify_args va{};
    va.n_peers = a->n_peers; va.row_stride = a->row_stride; va.n_z = a->n_z;
    auto cover = [&](size_t parts) {
        ca.n_partitions = va.n_partitions = (int32_t)parts;
        const size_t c = btard_centered_clip_workspace(&ca), v = btard_verify_projections_workspace(&va);
        if (c > h.ws_c_bytes) h.ws_c_bytes = c;
        if (v > h.ws_v_bytes) h.ws_v_bytes = v;
    };
    cover(P);
    const size_t nchunks = P < kMaxHostChunks ? P : kMaxHostChunks;
    for (size_t c = 0; c < nchunks; ++c) cover(P * (c + 1) / nchunks - P * c / nchunks);
    h.ws_c = take(h.ws_c_bytes);
    h.ws_v = take(h.ws_v_bytes);
    h.total = off;
    return h;
}

bool host_sizes_ok(const btard_host_args* a)
{
    return a && a->n_peers >= 1 && a->n_peers <= BTARD_MAX_PEERS && a->n_partitions >= 1 &&
           a->row_stride >= 4 && a->n_z >= 1 && a->n_z <= BTARD_MAX_Z &&
           (a->algo == BTARD_ALGO_DIRECT || a->algo == BTARD_ALGO_GRAM || a->algo == BTARD_ALGO_DIRECT_COOPERATIVE);
}

// Events of one call; destroyed on every way out.
struct ChunkEvents {
    cudaEvent_t ready[kMaxHostChunks] = {};
    ~ChunkEvents()
    {
        for (size_t c = 0; c < kMaxHostChunks; ++c)
            if (ready[c]) cudaEventDestroy(ready[c]);
    }
};
}  // namespace

size_t btard_aggregate_host_scratch(const btard_host_args* a)
{
    if (!host_sizes_ok(a)) return 0;
    return host_layout(a).total;
}

int btard_aggregate_host(const btard_host_args* a)
{
    if (!host_sizes_ok(a) || !a->g || !a->v || !a->device_scratch) return BTARD_ERR_INVALID_ARG;
    int rc = check_common(a->n_peers, a->n_partitions, a->row_stride, a->part_len, a->tau);
    if (rc != BTARD_OK) return rc;
    if (a->algo == BTARD_ALGO_GRAM && a->n_peers > kMaxGramPeers) return BTARD_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(a->device_scratch) & 255u) return BTARD_ERR_BAD_ALIGNMENT;
    const HostScratch h = host_layout(a);
    if (a->device_scratch_bytes < h.total) return BTARD_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)a->stream;
    char* base = (char*)a->device_scratch;
    const size_t n = a->n_peers, P = a->n_partitions, S = (size_t)a->row_stride, K = a->n_z;

    cudaStream_t cs = (cudaStream_t)a->copy_stream;
    const bool piped = host_piped(a);
    const size_t nchunks = host_chunks(a);
    const int algo = host_algo(a);
    ChunkEvents ev;
    if (a->init_mode == BTARD_INIT_CALLER_V0)
        BTARD_CUDA_TRY(cudaMemcpyAsync(base + h.v, a->v, sizeof(float) * P * S, cudaMemcpyHostToDevice, st));
    if (piped) {
        for (size_t c = 0; c < nchunks; ++c) {
            const size_t p0 = P * c / nchunks, p1 = P * (c + 1) / nchunks;
            BTARD_CUDA_TRY(cudaEventCreateWithFlags(&ev.ready[c], cudaEventDisableTiming));
            BTARD_CUDA_TRY(cudaMemcpyAsync(base + h.g + sizeof(float) * p0 * n * S, a->g + p0 * n * S,
                                           sizeof(float) * (p1 - p0) * n * S, cudaMemcpyHostToDevice, cs));
            BTARD_CUDA_TRY(cudaEventRecord(ev.ready[c], cs));
        }
    } else {
        BTARD_CUDA_TRY(cudaMemcpyAsync(base + h.g, a->g, sizeof(float) * P * n * S, cudaMemcpyHostToDevice, st));
    }

    for (size_t c = 0; c < nchunks; ++c) {
        const size_t p0 = P * c / nchunks, p1 = P * (c + 1) / nchunks;
        if (piped) BTARD_CUDA_TRY(cudaStreamWaitEvent(st, ev.ready[c], 0));
        btard_cclip_args ca{};
        ca.n_peers = a->n_peers; ca.n_partitions = (int32_t)(p1 - p0); ca.row_stride = a->row_stride;
        ca.part_len = a->part_len + p0; ca.g = (const float*)(base + h.g) + p0 * n * S; ca.tau = a->tau + p0;
        ca.init_mode = a->init_mode; ca.stop_mode = a->stop_mode; ca.algo = algo;
        ca.max_iters = a->max_iters; ca.eps = a->eps; ca.v = (float*)(base + h.v) + p0 * S;
        ca.iters = (int32_t*)(base + h.iters) + p0; ca.last_step_norm = (double*)(base + h.last_step) + p0;
        ca.resid_norm = (double*)(base + h.resid_norm) + p0 * n; ca.status = (uint32_t*)(base + h.status_c) + p0;
        ca.workspace = base + h.ws_c; ca.workspace_bytes = h.ws_c_bytes; ca.stream = a->stream;

        btard_verify_args va{};
        va.n_peers = a->n_peers; va.n_partitions = ca.n_partitions; va.row_stride = a->row_stride;
        va.seed = a->seed; va.n_z = a->n_z; va.partition_base = (int32_t)p0;
        va.norm = (double*)(base + h.norm) + p0 * n; va.weight = (double*)(base + h.weight) + p0 * n;
        va.dot = (double*)(base + h.dot) + p0 * n * K; va.s = (double*)(base + h.s) + p0 * n * K;
        va.s_sum = (double*)(base + h.s_sum) + p0 * K; va.znorm2 = (double*)(base + h.znorm2) + p0 * K;
        va.resid_sum_norm = (double*)(base + h.rsn) + p0; va.resid_sum = nullptr;
        va.status = (uint32_t*)(base + h.status_v) + p0;
        va.workspace = base + h.ws_v; va.workspace_bytes = h.ws_v_bytes;
        // one call: with the Gram variant the combine pass and the verification pass are one read of g
        rc = btard_centered_clip_verify(&ca, &va);
        if (rc != BTARD_OK) return rc;
    }

    auto back = [&](void* dst, size_t off, size_t bytes) -> cudaError_t {
        if (!dst) return cudaSuccess;
        return cudaMemcpyAsync(dst, base + off, bytes, cudaMemcpyDeviceToHost, st);
    };
    if (a->status) {
        or_status_kernel<<<(unsigned)((P + 127) / 128), 128, 0, st>>>((uint32_t*)(base + h.status_c),
                                                                      (const uint32_t*)(base + h.status_v), (int)P);
        BTARD_CUDA_TRY(cudaGetLastError());
        count_launch();
    }
    BTARD_CUDA_TRY(back(a->v, h.v, sizeof(float) * P * S));
    BTARD_CUDA_TRY(back(a->iters, h.iters, sizeof(int32_t) * P));
    BTARD_CUDA_TRY(back(a->last_step_norm, h.last_step, sizeof(double) * P));
    BTARD_CUDA_TRY(back(a->norm, h.norm, sizeof(double) * P * n));
    BTARD_CUDA_TRY(back(a->weight, h.weight, sizeof(double) * P * n));
    BTARD_CUDA_TRY(back(a->dot, h.dot, sizeof(double) * P * n * K));
    BTARD_CUDA_TRY(back(a->s, h.s, sizeof(double) * P * n * K));
    BTARD_CUDA_TRY(back(a->s_sum, h.s_sum, sizeof(double) * P * K));
    BTARD_CUDA_TRY(back(a->znorm2, h.znorm2, sizeof(double) * P * K));
    BTARD_CUDA_TRY(back(a->resid_sum_norm, h.rsn, sizeof(double) * P));
    BTARD_CUDA_TRY(back(a->status, h.status_c, sizeof(uint32_t) * P));
    BTARD_CUDA_TRY(cudaStreamSynchronize(st));
    return BTARD_OK;
}

}  // extern "C"
