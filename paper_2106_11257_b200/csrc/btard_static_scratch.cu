// btard_verify_projections_static: the verification pass for callers that cannot hand the library
// any scratch memory of their own.
//
// Who needs this: code that runs inside a process where something else already owns every byte of
// device memory (a serving or training framework that reserves the whole GPU for its own pool at
// start-up, so a later cudaMalloc fails), and code on a latency-critical path that must not call
// cudaMalloc / cudaFree at all because those calls may synchronise the whole device.  Such a caller
// still passes its inputs and outputs; only the scratch comes from here.
//
// The scratch is one fixed array in this library's device image.  It exists once per GPU that loads
// the library, from load until the process exits, whether or not this entry point is ever called.
// Every call on a GPU uses the same array, so two calls that overlap on that GPU (different streams,
// different threads) would overwrite each other's partial sums: callers must serialise them.  Nothing
// in the array is expected to survive from one call to the next; the counters that must start at zero
// are cleared on the stream at the start of every call.
#include <mutex>

#include "btard_common.h"

namespace btard {
namespace {

// File-scope device array.  In host code this name is only a handle: the device address has to be
// asked for with cudaGetSymbolAddress, per device.
static __device__ __align__(256) unsigned char g_static_scratch[BTARD_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
constexpr int kMaxStaticPartitions = 1024;     // more partitions than this never fit the array
std::mutex g_addr_mu;
void* g_scratch_addr[kMaxDevices] = {};

// Device address of the scratch array on the current device; looked up once per device.
int static_scratch_address(void** out)
{
    int dev = -1;
    BTARD_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return BTARD_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lk(g_addr_mu);
    if (!g_scratch_addr[dev]) {
        void* ptr = nullptr;
        BTARD_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch));
        if (!ptr) return BTARD_ERR_CUDA;
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return BTARD_OK;
}

bool is_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace
}  // namespace btard

using namespace btard;

extern "C" int btard_verify_projections_static(const btard_verify_args* a)
{
    if (!a) return BTARD_ERR_INVALID_ARG;
    const int n = a->n_peers, P = a->n_partitions, K = a->n_z;
    const long long stride = a->row_stride;
    if (n < 1 || P < 1 || stride < 4 || !a->part_len || !a->tau) return BTARD_ERR_INVALID_ARG;
    if (n > BTARD_MAX_PEERS || stride > (1LL << 33)) return BTARD_ERR_UNSUPPORTED;
    if (stride % 4 != 0) return BTARD_ERR_BAD_ALIGNMENT;
    if (K < 1 || K > BTARD_MAX_Z || a->partition_base < 0) return BTARD_ERR_INVALID_ARG;
    if (!a->g || !a->v || !a->norm || !a->weight || !a->dot || !a->s || !a->s_sum || !a->znorm2 ||
        !a->resid_sum_norm || !a->status)
        return BTARD_ERR_INVALID_ARG;
    if (!is_aligned16(a->g) || !is_aligned16(a->v) || (a->resid_sum && !is_aligned16(a->resid_sum)))
        return BTARD_ERR_BAD_ALIGNMENT;
    // Beyond this many partitions the problem does not fit the built-in scratch anyway.
    if (P > kMaxStaticPartitions) return BTARD_ERR_WORKSPACE_TOO_SMALL;
    for (int p = 0; p < P; ++p)
        if (a->part_len[p] < 0 || a->part_len[p] > stride || !(a->tau[p] >= 0.0))
            return BTARD_ERR_INVALID_ARG;

    // Carve the fixed array; refuse problems that need more than it holds.
    const VerifyGeometry vg = verify_geometry(n, P, stride, K);
    const Geometry cg = cclip_geometry(n, P, stride);
    size_t off = 0;
    auto take = [&](size_t bytes) { const size_t at = off; off = align_up(off + bytes, 256); return at; };
    const size_t o_table = take(sizeof(PartEntry) * (size_t)P);
    const size_t o_part = take(sizeof(double) * (size_t)P * vg.g.cpp * vg.slots);
    const size_t o_norms = take(sizeof(double) * (size_t)P * n);
    const size_t o_cslots = take(sizeof(double) * (size_t)P * cg.cpp * (n + 1));
    const size_t o_ctot = take(sizeof(double) * (size_t)P * (n + 1));
    const size_t o_ticket = take(sizeof(unsigned int) * (size_t)P);
    if (off > (size_t)BTARD_STATIC_SCRATCH_BYTES) return BTARD_ERR_WORKSPACE_TOO_SMALL;

    void* scratch = nullptr;
    int rc = static_scratch_address(&scratch);
    if (rc != BTARD_OK) return rc;
    char* base = (char*)scratch;
    cudaStream_t st = (cudaStream_t)a->stream;

    PartEntry* table = (PartEntry*)(base + o_table);
    rc = upload_table(table, P, a->part_len, a->tau, st);     // as kernel arguments: no host-memory copy
    if (rc != BTARD_OK) return rc;

    const double* norms = a->resid_norm_in;
    if (!norms) {   // one more pass over g: residual norms at v
        CclipLaunch L{};
        L.g = a->g; L.v = const_cast<float*>(a->v); L.table = table;
        L.slots = (double*)(base + o_cslots);
        L.tot_out = (double*)(base + o_ctot);
        L.ticket = (unsigned int*)(base + o_ticket);
        // The array keeps whatever the previous call left: the finish counters must start at zero.
        BTARD_CUDA_TRY(cudaMemsetAsync(L.ticket, 0, sizeof(unsigned int) * (size_t)P, st));
        L.stride = stride; L.n = n; L.P = P; L.row_scale = a->row_scale;
        rc = launch_cclip_pass(L, cg, PASS_NORMS, st);
        if (rc != BTARD_OK) return rc;
        rc = launch_totals_to_norms(L.tot_out, (double*)(base + o_norms), n, P, st);
        if (rc != BTARD_OK) return rc;
        norms = (const double*)(base + o_norms);
    }

    VerifyLaunch V{};
    V.g = a->g; V.v = a->v; V.table = table; V.norm_in = norms;
    V.part_out = (double*)(base + o_part);
    V.resid_sum = a->resid_sum;
    V.norm = a->norm; V.weight = a->weight; V.dot = a->dot; V.s = a->s; V.s_sum = a->s_sum;
    V.znorm2 = a->znorm2; V.resid_sum_norm = a->resid_sum_norm; V.status = a->status;
    V.stride = stride; V.n = n; V.P = P; V.K = K; V.p_base = a->partition_base;
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
