// C ABI of the verification library: argument checks, workspace layout, kernel launches.
// See include/fsd_verify.h for the contract of every entry point.
#include <climits>
#include <cstdint>
#include <cuda_runtime.h>
#include <atomic>
#include <mutex>

#include "fsd_verify.h"
#include "fsd_device.cuh"
#include "fsd_finish.cuh"
#include "fsd_pair_generic.cuh"
#include "fsd_pair_stream.cuh"
#include "fsd_tuning.cuh"

namespace {

using namespace fsd;

constexpr size_t kAlign = 256;
constexpr int kMaxVirtualCtas = 512;                                   // two per SM
constexpr size_t kExchangeBytes = 2 * kMaxVirtualCtas * sizeof(GroupMsg);
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }
inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

struct Workspace {
    int32_t* item_bits;
    int32_t* item_status;
    int* flags;                // [0] = a bounded device-side wait ran out
    GroupMsg* exchange;        // the streaming kernel's statistics exchange (directly after the flags: one memset clears both)
    PairRecord* records;       // per-pair totals of the streaming kernel
    size_t bytes;
};

Workspace carve(void* base, int B, int G) {
    Workspace w;
    const size_t items = static_cast<size_t>(B) * G;
    char* p = static_cast<char*>(base);
    w.item_bits = reinterpret_cast<int32_t*>(p);
    p += align_up(items * sizeof(int32_t));
    w.item_status = reinterpret_cast<int32_t*>(p);
    p += align_up(items * sizeof(int32_t));
    w.flags = reinterpret_cast<int*>(p);
    p += kAlign;
    w.exchange = reinterpret_cast<GroupMsg*>(p);
    p += kExchangeBytes;
    w.records = reinterpret_cast<PairRecord*>(p);
    p += align_up(items * sizeof(PairRecord));
    w.bytes = static_cast<size_t>(p - static_cast<char*>(base));
    return w;
}

int check_opts(const fsd_opts* o) {
    if (o == nullptr) return FSD_ERR_NULL;
    if (o->struct_size != sizeof(fsd_opts)) return FSD_ERR_ENUM;
    if (o->divergence < FSD_DIV_JS || o->divergence > FSD_DIV_TV) return FSD_ERR_ENUM;
    if (o->mode < FSD_MODE_FSD || o->mode > FSD_MODE_RFSD) return FSD_ERR_ENUM;
    if (o->compare < FSD_CMP_LT || o->compare > FSD_CMP_LE) return FSD_ERR_ENUM;
    if (o->sample < FSD_SAMPLE_INVCDF || o->sample > FSD_SAMPLE_GREEDY) return FSD_ERR_ENUM;
    if (o->logit_dtype < FSD_F32 || o->logit_dtype > FSD_BF16) return FSD_ERR_ENUM;
    if (o->threshold != o->threshold) return FSD_ERR_ENUM;   // NaN threshold
    return FSD_OK;
}

int check_shape(int B, int G, int V) {
    if (B < 1 || G < 1 || V < 1) return FSD_ERR_SHAPE;
    if (static_cast<long long>(B) * (static_cast<long long>(G) + 1) > INT_MAX) return FSD_ERR_SHAPE;
    return FSD_OK;
}

int finish_cluster_size(int B, int V) {
    // about 32 vocabulary entries per thread, at most the portable cluster size, and no more CTAs
    // than one wave of two per SM (148 SMs) when the batch is large
    int cs = 1;
    while (cs < kMaxClusterSize && static_cast<long long>(cs) * kFinishThreads * 32 < V &&
           static_cast<long long>(B) * cs * 2 <= 2 * 148)
        cs <<= 1;
    return cs;
}

std::atomic<void*> g_stage_event{nullptr};   // see fsd_set_stage_event
std::atomic<int> g_mark_timeout{0};          // see fsd_set_timeout_injection
std::atomic<int> g_group_size{0};            // see fsd_set_group_size

// ---- streaming kernel launch -----------------------------------------------------------
constexpr int kMaxDev = 64;

// One CTA of two virtual CTAs per SM, all resident (cooperative launch).  Puts nothing on a stream.
template <int DT, int DIV>
int prepare_stream(int dev) {
    static bool ready[kMaxDev] = {};
    static std::mutex mu;
    auto kernel = fsd_pair_stream_kernel<DT, DIV>;
    if (dev < 0 || dev >= kMaxDev) return FSD_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (!ready[dev]) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(kStreamSmemBytes)) != cudaSuccess)
            return FSD_ERR_CUDA;
        int per = 0;                                 // one CTA must fit an SM, or the cooperative launch is refused
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per, kernel, kStreamCtaThreads, kStreamSmemBytes) != cudaSuccess || per < 1)
            return FSD_ERR_CUDA;
        ready[dev] = true;
    }
    return FSD_OK;
}

template <int DT, int DIV>
int launch_stream(const StreamParams& gp, int nsm, cudaStream_t s) {
    // as many CTAs as give every pair a group, at most one per SM and what the exchange buffer holds
    long long want = (static_cast<long long>(gp.n_items) * gp.C + kStreamHalves - 1) / kStreamHalves;
    int grid = nsm;
    if (grid > kMaxVirtualCtas / kStreamHalves) grid = kMaxVirtualCtas / kStreamHalves;
    if (want < grid) grid = static_cast<int>(want);
    if (grid * kStreamHalves < gp.C) return FSD_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid), 1, 1);
    cfg.blockDim = dim3(kStreamCtaThreads, 1, 1);
    cfg.dynamicSmemBytes = kStreamSmemBytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;     // the groups' virtual CTAs wait for one another: all must be resident
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, fsd_pair_stream_kernel<DT, DIV>, gp) != cudaSuccess) return FSD_ERR_CUDA;
    return FSD_OK;
}

// Virtual CTAs per pair for the streaming kernel; 0 if the shape is not eligible (the generic
// kernel takes it).  Between the fewest whose slice fits on chip and kMaxGroupSize it is the size
// with the lowest estimated time -- rounds * (fixed cost of a round +
// cost of a ring stage * stages per slice), the two costs (3.4 and 1.07 us) measured on a B200.
// Few pairs are spread over many virtual CTAs (short rounds); many pairs over few (fewer rounds).
int group_size(int nvec_row, bool vec, int items, int nsm) {
    if (!vec || nvec_row < 64) return 0;
    const int cmin = (nvec_row + kMaxVecPerCta - 1) / kMaxVecPerCta;
    const int forced = g_group_size.load();
    if (forced >= cmin && forced <= kMaxGroupSize && cmin <= kMaxGroupSize) return forced;
    int vctas = kStreamHalves * nsm;
    if (vctas > kMaxVirtualCtas) vctas = kMaxVirtualCtas;
    int best = 0;
    double best_cost = 0.0;
    for (int C = cmin; C <= kMaxGroupSize && C <= vctas; ++C) {
        const int groups = vctas / C;
        const int rounds = (items + groups - 1) / groups;
        const int slice = (nvec_row + C - 1) / C;
        const int stages = (slice + kStageVecs - 1) / kStageVecs;
        const double cost = rounds * (3.4 + 1.07 * stages);
        if (best == 0 || cost < best_cost) { best = C; best_cost = cost; }
    }
    return best;
}

template <int DT>
int launch_all(const PairParams& pp, FinishParams fp, bool vec, int* flags, GroupMsg* exchange, PairRecord* records, cudaStream_t s) {
    const int items = pp.B * pp.G;
    const int nvec_row = pp.V / Logit<DT>::kPerVec;
    int dev = 0, nsm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&nsm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || nsm < 1)
        return FSD_ERR_CUDA;
    const int C = group_size(nvec_row, vec, items, nsm);
    if (C > 0) {
        StreamParams sp;
        sp.target = pp.target; sp.draft = pp.draft; sp.parent = pp.parent; sp.B = pp.B; sp.G = pp.G;
        sp.nvec_row = nvec_row; sp.n_items = items; sp.records = records; sp.timeout_flag = flags; sp.next_pair = flags + 1;
        sp.C = C; sp.exchange = exchange;
        // test aid: one virtual CTA keeps its first message to itself, so that its group's exchange
        // runs out (after a shorter limit: about a tenth of a second) and the kernel's own give-up path runs
        const bool silent = g_mark_timeout.load() == 2;
        sp.poll_limit = silent ? (1u << 17) : kSpinLimit;
        sp.silent_rank = silent ? C - 1 : -1;
        // everything that can fail without a launch (attributes, the occupancy query) comes before
        // the first thing put on the stream
        int rc;
        if (pp.div == FSD_DIV_JS)      rc = prepare_stream<DT, FSD_DIV_JS>(dev);
        else if (pp.div == FSD_DIV_KL) rc = prepare_stream<DT, FSD_DIV_KL>(dev);
        else                           rc = prepare_stream<DT, FSD_DIV_TV>(dev);
        if (rc != FSD_OK) return rc;
        // the flag block and the exchange buffer start every call at zero: flags [0] timeout, [1] pairs handed out
        if (cudaMemsetAsync(flags, 0, kAlign + kExchangeBytes, s) != cudaSuccess) return FSD_ERR_CUDA;
        if (pp.div == FSD_DIV_JS)      rc = launch_stream<DT, FSD_DIV_JS>(sp, nsm, s);
        else if (pp.div == FSD_DIV_KL) rc = launch_stream<DT, FSD_DIV_KL>(sp, nsm, s);
        else                           rc = launch_stream<DT, FSD_DIV_TV>(sp, nsm, s);
        if (rc != FSD_OK) return rc;
        // test aid: behave as if a bounded wait of the streaming kernel had run out
        if (g_mark_timeout.load() == 1 && cudaMemsetAsync(flags, 1, sizeof(int), s) != cudaSuccess) return FSD_ERR_CUDA;
        fp.timeout_flag = flags;
        fp.records = records;
    } else {
#ifdef FSD_DEBUG_CHECKS
        if (cudaMemsetAsync(flags, 0, kAlign, s) != cudaSuccess) return FSD_ERR_CUDA;   // the debug word starts at zero here too
#endif
        if (vec) fsd_pair_generic_kernel<DT, true><<<items, 512, 0, s>>>(pp);
        else     fsd_pair_generic_kernel<DT, false><<<items, 512, 0, s>>>(pp);
        if (cudaGetLastError() != cudaSuccess) return FSD_ERR_CUDA;
        fp.timeout_flag = nullptr;
        fp.records = nullptr;
    }

    if (void* ev = g_stage_event.load()) {
        if (cudaEventRecord(static_cast<cudaEvent_t>(ev), s) != cudaSuccess) return FSD_ERR_CUDA;
    }
    const int cs = finish_cluster_size(fp.B, fp.V);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(fp.B) * cs, 1, 1);
    cfg.blockDim = dim3(kFinishThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cs;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // The finish kernel may be set up while the pair kernel drains: its CTAs take the SMs the
    // pair kernel's CTAs leave, build their tables, and wait (griddepcontrol.wait) for the pair
    // kernel to complete before they read anything it wrote.
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (cudaLaunchKernelEx(&cfg, fsd_finish_kernel<DT>, fp) != cudaSuccess) return FSD_ERR_CUDA;
    return FSD_OK;
}

int verify_common(const void* target, const void* draft, const int32_t* tokens, const float* u_accept,
                  const float* u_sample, const int32_t* parent, int B, int G, int V, int max_depth,
                  const fsd_opts* o, int32_t* accept_len, int32_t* path, int32_t* next_token,
                  float* divergence, int32_t* row_status, void* workspace, size_t workspace_bytes,
                  void* stream) {
    const size_t es = o->logit_dtype == FSD_BF16 ? 2 : 4;
    if (!aligned(target, es) || !aligned(draft, es) || !aligned(u_sample, 4) || !aligned(accept_len, 4) ||
        !aligned(next_token, 4) || !aligned(divergence, 4) || !aligned(row_status, 4) ||
        !aligned(tokens, 4) || !aligned(u_accept, 4) || !aligned(parent, 4) || !aligned(path, 4) ||
        !aligned(workspace, kAlign))
        return FSD_ERR_ALIGN;
    Workspace ws = carve(workspace, B, G);
    if (workspace_bytes < ws.bytes) return FSD_ERR_WORKSPACE;

    PairParams pp;
    pp.target = target; pp.draft = draft; pp.tokens = tokens; pp.u_accept = u_accept; pp.parent = parent;
    pp.B = B; pp.G = G; pp.V = V;
    pp.div = o->divergence; pp.mode = o->mode; pp.cmp = o->compare; pp.T = o->threshold;
    pp.divergence = divergence; pp.item_bits = ws.item_bits; pp.item_status = ws.item_status;
    pp.debug_word = ws.flags + 2;

    FinishParams fp;
    fp.target = target; fp.draft = draft; fp.parent = parent; fp.u_sample = u_sample;
    fp.B = B; fp.G = G; fp.V = V;
    fp.tokens = tokens; fp.u_accept = u_accept;
    fp.div = o->divergence; fp.mode = o->mode; fp.cmp = o->compare; fp.sample = o->sample; fp.max_depth = max_depth;
    fp.T = o->threshold; fp.records = nullptr; fp.divergence = divergence;
    fp.item_bits = ws.item_bits; fp.item_status = ws.item_status; fp.timeout_flag = nullptr;
    fp.accept_len = accept_len; fp.path = path; fp.next_token = next_token; fp.row_status = row_status;
    fp.debug_word = ws.flags + 2;

    const bool vec = (static_cast<size_t>(V) * es) % 16 == 0 && aligned(target, 16) && aligned(draft, 16);
    fp.vec = vec ? 1 : 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return o->logit_dtype == FSD_BF16 ? launch_all<FSD_BF16>(pp, fp, vec, ws.flags, ws.exchange, ws.records, s)
                                       : launch_all<FSD_F32>(pp, fp, vec, ws.flags, ws.exchange, ws.records, s);
}

struct HostStaging {
    char *target, *draft, *tokens, *u_accept, *u_sample, *accept_len, *next_token, *divergence, *row_status, *ws;
    size_t n_target, n_draft, n_items4, n_rows4, n_ws, bytes;
};

HostStaging carve_staging(void* base, int B, int G, int V, size_t es) {
    HostStaging h;
    h.n_target = static_cast<size_t>(B) * (G + 1) * V * es;
    h.n_draft = static_cast<size_t>(B) * G * V * es;
    h.n_items4 = static_cast<size_t>(B) * G * 4;
    h.n_rows4 = static_cast<size_t>(B) * 4;
    h.n_ws = carve(nullptr, B, G).bytes;
    char* p = static_cast<char*>(base);
    auto take = [&](size_t n) { char* q = p; p += align_up(n); return q; };
    h.target = take(h.n_target); h.draft = take(h.n_draft);
    h.tokens = take(h.n_items4); h.u_accept = take(h.n_items4); h.u_sample = take(h.n_rows4);
    h.accept_len = take(h.n_rows4); h.next_token = take(h.n_rows4);
    h.divergence = take(h.n_items4); h.row_status = take(h.n_rows4);
    h.ws = take(h.n_ws);
    h.bytes = static_cast<size_t>(p - static_cast<char*>(base));
    return h;
}

// Built-in scratch of fsd_verify_chain_static.  In host code this name is only a handle for
// cudaGetSymbolAddress; the kernels get the device address that call returns.
static __device__ __align__(256) unsigned char g_static_scratch[FSD_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void* g_static_ptr[kMaxDevices] = {};

// Device address of g_static_scratch on the current device (looked up once per device).
int static_scratch(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return FSD_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (g_static_ptr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return FSD_ERR_CUDA;
        g_static_ptr[dev] = p;
    }
    *out = g_static_ptr[dev];
    return FSD_OK;
}

}  // namespace

extern "C" {

void fsd_default_opts(fsd_opts* opts) {
    if (opts == nullptr) return;
    opts->struct_size = sizeof(fsd_opts);
    opts->divergence = FSD_DIV_JS;
    opts->mode = FSD_MODE_FSD;
    opts->compare = FSD_CMP_LT;
    opts->sample = FSD_SAMPLE_INVCDF;
    opts->logit_dtype = FSD_BF16;
    opts->threshold = 0.0f;
}

int fsd_workspace_bytes(int B, int positions, int V, const fsd_opts* opts, size_t* bytes_out) {
    if (bytes_out == nullptr) return FSD_ERR_NULL;
    int rc = check_opts(opts);
    if (rc != FSD_OK) return rc;
    rc = check_shape(B, positions, V);
    if (rc != FSD_OK) return rc;
    *bytes_out = carve(nullptr, B, positions).bytes;
    return FSD_OK;
}

int fsd_verify_chain(const void* target_logits, const void* draft_logits, const int32_t* draft_tokens,
                     const float* u_accept, const float* u_sample, int B, int gamma, int V,
                     const fsd_opts* opts, int32_t* accept_len, int32_t* next_token, float* divergence,
                     int32_t* row_status, void* workspace, size_t workspace_bytes, void* stream) {
    int rc = check_opts(opts);
    if (rc != FSD_OK) return rc;
    if (!target_logits || !draft_logits || !u_sample || !accept_len || !next_token || !divergence ||
        !row_status || !workspace)
        return FSD_ERR_NULL;
    if (opts->mode != FSD_MODE_FSD && (!draft_tokens || !u_accept)) return FSD_ERR_NULL;
    rc = check_shape(B, gamma, V);
    if (rc != FSD_OK) return rc;
    return verify_common(target_logits, draft_logits, draft_tokens, u_accept, u_sample, nullptr, B, gamma, V, 0,
                         opts, accept_len, nullptr, next_token, divergence, row_status, workspace,
                         workspace_bytes, stream);
}

int fsd_verify_tree(const void* target_logits, const void* draft_logits, const int32_t* parent,
                    const float* u_sample, int B, int N, int V, int max_depth, const fsd_opts* opts,
                    int32_t* accept_len, int32_t* path, int32_t* next_token, float* divergence,
                    int32_t* row_status, void* workspace, size_t workspace_bytes, void* stream) {
    int rc = check_opts(opts);
    if (rc != FSD_OK) return rc;
    if (!target_logits || !draft_logits || !parent || !u_sample || !accept_len || !path || !next_token ||
        !divergence || !row_status || !workspace)
        return FSD_ERR_NULL;
    if (opts->mode != FSD_MODE_FSD) return FSD_ERR_UNSUPPORTED;
    rc = check_shape(B, N, V);
    if (rc != FSD_OK) return rc;
    if (max_depth < 1 || N > kMaxTreeNodes) return FSD_ERR_SHAPE;
    return verify_common(target_logits, draft_logits, nullptr, nullptr, u_sample, parent, B, N, V, max_depth,
                         opts, accept_len, path, next_token, divergence, row_status, workspace,
                         workspace_bytes, stream);
}

int fsd_host_staging_bytes(int B, int gamma, int V, const fsd_opts* opts, size_t* bytes_out) {
    if (bytes_out == nullptr) return FSD_ERR_NULL;
    int rc = check_opts(opts);
    if (rc != FSD_OK) return rc;
    rc = check_shape(B, gamma, V);
    if (rc != FSD_OK) return rc;
    *bytes_out = carve_staging(nullptr, B, gamma, V, opts->logit_dtype == FSD_BF16 ? 2 : 4).bytes;
    return FSD_OK;
}

int fsd_verify_chain_host(const void* h_target_logits, const void* h_draft_logits, const int32_t* h_draft_tokens,
                          const float* h_u_accept, const float* h_u_sample, int B, int gamma, int V,
                          const fsd_opts* opts, int32_t* h_accept_len, int32_t* h_next_token,
                          float* h_divergence, int32_t* h_row_status, void* staging, size_t staging_bytes,
                          void* stream) {
    int rc = check_opts(opts);
    if (rc != FSD_OK) return rc;
    if (!h_target_logits || !h_draft_logits || !h_u_sample || !h_accept_len || !h_next_token || !h_divergence ||
        !h_row_status || !staging)
        return FSD_ERR_NULL;
    if (opts->mode != FSD_MODE_FSD && (!h_draft_tokens || !h_u_accept)) return FSD_ERR_NULL;
    rc = check_shape(B, gamma, V);
    if (rc != FSD_OK) return rc;
    if (!aligned(staging, kAlign)) return FSD_ERR_ALIGN;
    HostStaging h = carve_staging(staging, B, gamma, V, opts->logit_dtype == FSD_BF16 ? 2 : 4);
    if (staging_bytes < h.bytes) return FSD_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    bool ok = true;
    ok = ok && cudaMemcpyAsync(h.target, h_target_logits, h.n_target, cudaMemcpyHostToDevice, s) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(h.draft, h_draft_logits, h.n_draft, cudaMemcpyHostToDevice, s) == cudaSuccess;
    if (h_draft_tokens) ok = ok && cudaMemcpyAsync(h.tokens, h_draft_tokens, h.n_items4, cudaMemcpyHostToDevice, s) == cudaSuccess;
    if (h_u_accept) ok = ok && cudaMemcpyAsync(h.u_accept, h_u_accept, h.n_items4, cudaMemcpyHostToDevice, s) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(h.u_sample, h_u_sample, h.n_rows4, cudaMemcpyHostToDevice, s) == cudaSuccess;
    if (!ok) return FSD_ERR_CUDA;
    rc = fsd_verify_chain(h.target, h.draft, h_draft_tokens ? reinterpret_cast<int32_t*>(h.tokens) : nullptr,
                          h_u_accept ? reinterpret_cast<float*>(h.u_accept) : nullptr,
                          reinterpret_cast<float*>(h.u_sample), B, gamma, V, opts,
                          reinterpret_cast<int32_t*>(h.accept_len), reinterpret_cast<int32_t*>(h.next_token),
                          reinterpret_cast<float*>(h.divergence), reinterpret_cast<int32_t*>(h.row_status),
                          h.ws, h.n_ws, stream);
    if (rc != FSD_OK) return rc;
    ok = ok && cudaMemcpyAsync(h_accept_len, h.accept_len, h.n_rows4, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(h_next_token, h.next_token, h.n_rows4, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(h_divergence, h.divergence, h.n_items4, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(h_row_status, h.row_status, h.n_rows4, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    ok = ok && cudaStreamSynchronize(s) == cudaSuccess;
    return ok ? FSD_OK : FSD_ERR_CUDA;
}

int fsd_verify_chain_static(const void* target_logits, const void* draft_logits, const int32_t* draft_tokens,
                            const float* u_accept, const float* u_sample, int B, int gamma, int V,
                            const fsd_opts* opts, int32_t* accept_len, int32_t* next_token, float* divergence,
                            int32_t* row_status, void* stream) {
    int rc = check_opts(opts);
    if (rc != FSD_OK) return rc;
    if (!target_logits || !draft_logits || !u_sample || !accept_len || !next_token || !divergence || !row_status)
        return FSD_ERR_NULL;
    if (opts->mode != FSD_MODE_FSD && (!draft_tokens || !u_accept)) return FSD_ERR_NULL;
    rc = check_shape(B, gamma, V);
    if (rc != FSD_OK) return rc;
    if (static_cast<long long>(B) * gamma > FSD_STATIC_MAX_POSITIONS ||
        carve(nullptr, B, gamma).bytes > FSD_STATIC_SCRATCH_BYTES)
        return FSD_ERR_TOO_LARGE;
    void* scratch = nullptr;
    rc = static_scratch(&scratch);
    if (rc != FSD_OK) return rc;
    return verify_common(target_logits, draft_logits, draft_tokens, u_accept, u_sample, nullptr, B, gamma, V, 0,
                         opts, accept_len, nullptr, next_token, divergence, row_status, scratch,
                         FSD_STATIC_SCRATCH_BYTES, stream);
}

const char* fsd_status_string(int status) {
    switch (status) {
        case FSD_OK: return "FSD_OK";
        case FSD_ERR_NULL: return "FSD_ERR_NULL: a required pointer is NULL";
        case FSD_ERR_SHAPE: return "FSD_ERR_SHAPE: a dimension is out of range";
        case FSD_ERR_ALIGN: return "FSD_ERR_ALIGN: a pointer is misaligned";
        case FSD_ERR_ENUM: return "FSD_ERR_ENUM: an option is out of range";
        case FSD_ERR_WORKSPACE: return "FSD_ERR_WORKSPACE: workspace too small";
        case FSD_ERR_UNSUPPORTED: return "FSD_ERR_UNSUPPORTED: combination not defined";
        case FSD_ERR_CUDA: return "FSD_ERR_CUDA: the CUDA runtime refused a launch";
        case FSD_ERR_TOO_LARGE: return "FSD_ERR_TOO_LARGE: B * gamma exceeds FSD_STATIC_MAX_POSITIONS";
        default: return "unknown fsd status";
    }
}

int fsd_version(void) { return 100; }

int fsd_set_stage_event(void* event) {
    g_stage_event.store(event);
    return FSD_OK;
}

int fsd_debug_checks(int B, int positions, size_t* word_offset) {
    if (word_offset != nullptr && B >= 1 && positions >= 1) {
        const Workspace w = carve(nullptr, B, positions);
        *word_offset = static_cast<size_t>(reinterpret_cast<char*>(w.flags + 2) - static_cast<char*>(nullptr));
    }
#ifdef FSD_DEBUG_CHECKS
    return 1;
#else
    return 0;
#endif
}

int fsd_set_timeout_injection(int mode) {
    if (mode < 0 || mode > 2) return FSD_ERR_ENUM;
    g_mark_timeout.store(mode);
    return FSD_OK;
}

int fsd_set_group_size(int group_size) {
    if (group_size < 0 || group_size > kMaxGroupSize) return FSD_ERR_SHAPE;
    g_group_size.store(group_size);
    return FSD_OK;
}

int fsd_threshold_sweep(const float* divergence, int B, int positions, const float* thresholds, int n_thresholds,
                        int compare, float* mean_accept_len, float* accept_fraction, void* stream) {
    if (divergence == nullptr || thresholds == nullptr || mean_accept_len == nullptr || accept_fraction == nullptr)
        return FSD_ERR_NULL;
    if (B < 1 || positions < 1 || n_thresholds < 1) return FSD_ERR_SHAPE;
    if (static_cast<long long>(B) * positions > INT_MAX) return FSD_ERR_SHAPE;      // the kernels count in 32 bits
    if (compare != FSD_CMP_LT && compare != FSD_CMP_LE) return FSD_ERR_ENUM;
    fsd_threshold_sweep_kernel<<<n_thresholds, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        divergence, B, positions, thresholds, compare, mean_accept_len, accept_fraction);
    return cudaGetLastError() == cudaSuccess ? FSD_OK : FSD_ERR_CUDA;
}

int fsd_calibrate_threshold(const float* divergence, int B, int positions, float target_mean_accept_len, int compare,
                            float* threshold_out, float* achieved_out, void* stream) {
    if (divergence == nullptr || threshold_out == nullptr || achieved_out == nullptr) return FSD_ERR_NULL;
    if (B < 1 || positions < 1 || !(target_mean_accept_len >= 0.f)) return FSD_ERR_SHAPE;   // NaN target included
    if (static_cast<long long>(B) * positions > INT_MAX) return FSD_ERR_SHAPE;      // the kernels count in 32 bits
    if (compare != FSD_CMP_LT && compare != FSD_CMP_LE) return FSD_ERR_ENUM;
    fsd_calibrate_kernel<<<1, kTuneThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        divergence, B, positions, target_mean_accept_len, compare, threshold_out, achieved_out);
    return cudaGetLastError() == cudaSuccess ? FSD_OK : FSD_ERR_CUDA;
}

int fsd_accept_labels(const float* divergence, int B, int positions, float threshold, int compare, uint8_t* labels,
                      void* stream) {
    if (divergence == nullptr || labels == nullptr) return FSD_ERR_NULL;
    if (B < 1 || positions < 1) return FSD_ERR_SHAPE;
    if (compare != FSD_CMP_LT && compare != FSD_CMP_LE) return FSD_ERR_ENUM;
    const size_t n = static_cast<size_t>(B) * positions;
    const unsigned blocks = static_cast<unsigned>(n / 256 + 1 < 1184 ? n / 256 + 1 : 1184);
    fsd_accept_labels_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(divergence, n, threshold, compare, labels);
    return cudaGetLastError() == cudaSuccess ? FSD_OK : FSD_ERR_CUDA;
}

}  // extern "C"
