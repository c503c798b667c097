// Streaming per-(row, position) kernel: every logit is read from HBM once.
//
// A (row, position) pair is split along the vocabulary over a group of G CTAs (one CTA per SM,
// G chosen on the host so that a CTA's slice fits on chip with room to run ahead).  Groups are
// persistent and take pairs round-robin.  Inside a CTA the work is a pipeline of specialised
// warps that never meet on a CTA-wide barrier:
//   producer warp   one lane keeps a ring of shared-memory stages full with bulk asynchronous
//                   copies (cp.async.bulk + mbarrier, no multicast) of the CTA's slices of the
//                   target and the draft row;
//   first-sweep     eight warps (two per tensor-memory lane quarter) take each stage as it lands:
//   warps           e = 2^(logit * log2e - k) with one MUFU ex2 per logit, the sums Z = sum e and
//                   S = sum e*y (or the KL sum), a bitwise "rows differ" flag, and park the e
//                   values in a ring of tensor-memory chunks.  k is an integer reference in the
//                   log2 domain that a warp takes from the first vectors in which it meets a
//                   finite logit; it never moves afterwards.  A pair whose sums leave the range in
//                   which that is accurate (a later logit more than 2^62 above the reference, a
//                   NaN, +inf) is marked and recomputed by the finish kernel with exact maxima;
//   exchange        the last first-sweep warp to finish a pair folds the warps' statistics and
//                   publishes the CTA's part in the pair's record in global memory, then counts
//                   the CTA in with a release; nobody waits for this;
//   second-sweep    four warps (one per lane quarter) run one pair behind: they wait for all G
//   warps           parts of the pair (acquire poll of the counter, bounded), fold the
//                   normalisers, and sweep the parked values chunk by chunk: p = e_a/Z_a,
//                   q = e_b/Z_b; JS needs sum (p+q) log2(p+q) (one MUFU lg2 per vocabulary
//                   entry), TV needs sum |p - q|, KL nothing.  A chunk returns to the first-sweep
//                   warps as soon as its values are in registers.
// Because the tensor-memory ring holds more than one pair's slice, the first sweep of the next
// pair proceeds while the group's statistics travel, so the exchange latency is hidden, and
// the special-function pipe sees first-sweep and second-sweep work at the same time.
// The finish kernel folds the record's parts in double precision; no double-precision
// arithmetic runs here.  HBM traffic is the algorithmic minimum.
#pragma once

#include <type_traits>

#include "fsd_device.cuh"

namespace fsd {

constexpr int kS1PerQuarter = 2;                           // first-sweep warps per tensor-memory lane quarter
constexpr int kS1Warps = 4 * kS1PerQuarter;
constexpr int kS2Warps = 4;
constexpr int kPipeWarps = kS1Warps + kS2Warps + 1;        // + producer
constexpr int kPipeThreads = 32 * kPipeWarps;
constexpr int kProducerWarp = kS1Warps + kS2Warps;
constexpr int kVecPerThread = 2;                           // 16-byte vectors per first-sweep thread, row and stage
constexpr int kStageVecs = kS1Warps * 32 * kVecPerThread;  // vectors per row and stage
constexpr int kStageRowBytes = kStageVecs * 16;
constexpr int kStageBytes = 2 * kStageRowBytes;
constexpr int kRing = 8;                                   // stages in the shared-memory ring
constexpr int kTmemCols = 512;                             // the whole tensor memory of the SM
constexpr int kMaxChunks = 16;                             // tensor-memory chunks (fp32 logits; bf16: 8)
constexpr int kPairDepth = 4;                              // pairs the first sweep may run ahead of the second
constexpr int kMaxGroup = 16;                              // CTAs per pair at most (parts in a record)
constexpr int kMaxClusterSize = 8;                         // finish kernel (portable cluster size)
constexpr uint32_t kSpinLimit = 1u << 24;                  // polls before a shared-memory wait gives up
constexpr uint32_t kPollLimit = 1u << 22;                  // polls of the group counter (each an L2 round trip)
constexpr float kRangeLimit = 4.611686018427388e18f;       // 2^62: sums above this (or NaN) mark the pair for recomputation

// Partial statistics of one (target row, draft row) pair: of a warp, of a CTA, or -- in a
// pair's record -- of each CTA of the group that streamed the pair.
//   z = sum 2^y, s = sum 2^y * y with y = logit*log2e - k and k the integer reference (log2
//   domain) the sums are relative to.  s0 is the target row's s for JS and the KL sum
//   sum 2^ya (ya - yb) for KL.
struct alignas(16) Stats {
    float ka, kb;              // references; -inf: no finite logit seen
    float za, zb;
    float s0, sb;
    float x;                   // unused (kept for the record layout)
    uint32_t diff;             // bit 0: the two rows differ somewhere; bit 1: sums out of range, recompute
};
static_assert(sizeof(Stats) == 32, "Stats is written as two 16-byte stores");
constexpr uint32_t kDiffRows = 1, kDiffRedo = 2;

// What the streaming kernel leaves per pair for the finish kernel, which folds the parts in
// double precision (second-sweep sums: JS sum s log2 s, TV sum |p - q|).
struct alignas(16) PairRecord {
    Stats part[kMaxGroup];
    float x[kMaxGroup];        // each CTA's second-sweep sum of this pair
    uint32_t ncta;             // parts in use
    uint32_t state;            // kRecordStats | kRecordBadTree
    uint32_t pad[2];
};
static_assert(sizeof(PairRecord) == 592, "PairRecord layout");
constexpr uint32_t kRecordStats = 1, kRecordBadTree = 2;

struct PipeParams {
    const void* target;        // [B, G+1, V]
    const void* draft;         // [B, G,   V]
    const int32_t* parent;     // [B, G] (tree) or null (chain)
    int B, G;
    int nvec_row;              // 16-byte vectors per logit row
    int n_items;               // B * G
    int group;                 // CTAs per pair
    PairRecord* records;       // [B * G]
    int* arrived;              // [B * G] CTAs that have published their part; zero at launch
    int* timeout_flag;         // set to 1 if a bounded wait ran out; zero at launch
    uint32_t poll_limit;       // polls of a pair's counter before the second sweep gives up
};

// ---- PTX wrappers -----------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: returns false (and raises the flag) if the phase never completes.  Once a
// wait of this thread has run out (`dead`), later waits return at once: the results are
// already marked invalid and the kernel only has to reach its end.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, int* timeout_flag, bool& dead) {
    if (dead) return false;
#pragma unroll 1
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        // somebody else has given up already: nothing this thread waits for is certain to come
        if ((i & 1023u) == 1023u && *reinterpret_cast<volatile int*>(timeout_flag) != 0) break;
    }
    atomicExch(timeout_flag, 1);
    dead = true;
    return false;
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

template <int N> __device__ __forceinline__ void tmem_st(uint32_t taddr, const float (&r)[N]);
template <> __device__ __forceinline__ void tmem_st<16>(uint32_t taddr, const float (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "f"(r[0]), "f"(r[1]), "f"(r[2]), "f"(r[3]), "f"(r[4]), "f"(r[5]), "f"(r[6]), "f"(r[7]),
        "f"(r[8]), "f"(r[9]), "f"(r[10]), "f"(r[11]), "f"(r[12]), "f"(r[13]), "f"(r[14]), "f"(r[15]) : "memory");
}
template <> __device__ __forceinline__ void tmem_st<8>(uint32_t taddr, const float (&r)[8]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 ::"r"(taddr), "f"(r[0]), "f"(r[1]), "f"(r[2]), "f"(r[3]), "f"(r[4]), "f"(r[5]), "f"(r[6]), "f"(r[7])
                 : "memory");
}
template <int N> __device__ __forceinline__ void tmem_ld(uint32_t taddr, float (&r)[N]);
template <> __device__ __forceinline__ void tmem_ld<16>(uint32_t taddr, float (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=f"(r[0]), "=f"(r[1]), "=f"(r[2]), "=f"(r[3]), "=f"(r[4]), "=f"(r[5]), "=f"(r[6]), "=f"(r[7]),
          "=f"(r[8]), "=f"(r[9]), "=f"(r[10]), "=f"(r[11]), "=f"(r[12]), "=f"(r[13]), "=f"(r[14]), "=f"(r[15])
        : "r"(taddr) : "memory");
}
template <> __device__ __forceinline__ void tmem_ld<8>(uint32_t taddr, float (&r)[8]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(r[0]), "=f"(r[1]), "=f"(r[2]), "=f"(r[3]), "=f"(r[4]), "=f"(r[5]), "=f"(r[6]), "=f"(r[7])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// NaN-propagating maxima: a NaN logit must reach the sums so that the pair is marked
__device__ __forceinline__ uint32_t bf16x2_max_nan(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ float fmax_nan(float a, float b) {
    float d;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}
__device__ __forceinline__ float warp_max_nan(float v) {
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) v = fmax_nan(v, __shfl_xor_sync(0xffffffffu, v, m));
    return v;
}
// ---- packed pairs of floats (one instruction works on two values) --------------------------
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float sum2(uint64_t v) {
    float lo, hi;
    unpack2(v, lo, hi);
    return lo + hi;
}

// 2^d for an integer-valued d <= 0 (exact); 0 below the normal range and for d = -inf; NaN for NaN
__device__ __forceinline__ float pow2_int(float d) {
    if (d != d) return d;
    return d < -126.f ? 0.f : __int_as_float((static_cast<int>(d) + 127) << 23);
}
// A KL partial sum brought to another reference: +inf (a logit with p > 0 = q) stays +inf even
// when the factor underflows to 0
__device__ __forceinline__ float scale_kl(float f, float v) { return v == INFINITY ? v : f * v; }

// ---- group counter in global memory ------------------------------------------------------
__device__ __forceinline__ void red_release_add(int* p, int v) {
    asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ int ld_acquire(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// ---- shared-memory layout ---------------------------------------------------------------
struct PipeShared {
    uint64_t full[kRing];                  // a ring stage has landed
    uint64_t empty[kRing];                 // every first-sweep warp has its vectors of the stage in registers
    uint64_t tfull[4][kMaxChunks];         // per lane quarter: the chunk's e values are parked
    uint64_t tfree[4][kMaxChunks];         // per lane quarter: the second sweep has the chunk in registers
    uint64_t pdone[kPairDepth];            // the second-sweep warps are done with the pair in this slot
    uint32_t tmem_base;
    int s1_count[kPairDepth];              // first-sweep warps that have left their statistics
    int s2_count[kPairDepth];              // second-sweep warps that have left their sums
    float xs[kPairDepth][kS2Warps];
    Stats ws[kPairDepth][kS1Warps];        // the first-sweep warps' statistics of a pair
};
constexpr size_t kPipeSmemBytes = kRing * kStageBytes + sizeof(PipeShared) + 128;

// Vectors of a logit row that CTA `rank` of a group of `group` takes: [vbeg, vbeg + vcnt)
__host__ __device__ inline void pipe_slice(int nvec_row, int group, int rank, int& vbeg, int& vcnt) {
    const int base = nvec_row / group, rem = nvec_row % group;
    vbeg = rank * base + (rank < rem ? rank : rem);
    vcnt = base + (rank < rem ? 1 : 0);
}

template <int DT, int DIV>
__global__ void __launch_bounds__(kPipeThreads, 1) fsd_pair_pipeline_kernel(PipeParams P) {
    constexpr int EPV = Logit<DT>::kPerVec;          // logits per 16-byte vector
    constexpr int EPT = 2 * EPV;                     // e values per thread and vector position (both rows)
    constexpr int VPT = kVecPerThread;
    constexpr int CPC = kS1PerQuarter * VPT * EPT;   // tensor-memory columns per chunk
    constexpr int NCH = kTmemCols / CPC;             // chunks in the tensor-memory ring
    static_assert(NCH <= kMaxChunks, "chunk barriers");
    constexpr bool kSecondSweep = DIV != FSD_DIV_KL;
    constexpr uint32_t kNegInfVec = DT == FSD_BF16 ? 0xFF80FF80u : 0xFF800000u;

    extern __shared__ unsigned char smem_raw[];
    unsigned char* ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    PipeShared& sh = *reinterpret_cast<PipeShared*>(ring + kRing * kStageBytes);

    const int G = P.group;
    const int group_id = blockIdx.x / G, n_groups = gridDim.x / G, rank = blockIdx.x % G;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    int vbeg, vcnt;
    pipe_slice(P.nvec_row, G, rank, vbeg, vcnt);
    const int ns = (vcnt + kStageVecs - 1) / kStageVecs;             // stages (= chunks) per pair
    const int ns_full = vcnt / kStageVecs;                           // stages with every vector present
    const size_t row_bytes = static_cast<size_t>(P.nvec_row) * 16;

    // ---- set-up: barriers, tensor memory ----
    if (tid == 0) {
        for (int s = 0; s < kRing; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], kS1Warps); }
        for (int q = 0; q < 4; ++q)
            for (int c = 0; c < kMaxChunks; ++c) { mbar_init(&sh.tfull[q][c], kS1PerQuarter); mbar_init(&sh.tfree[q][c], 1); }
        for (int d = 0; d < kPairDepth; ++d) { mbar_init(&sh.pdone[d], kS2Warps); sh.s1_count[d] = 0; sh.s2_count[d] = 0; }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kProducerWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&sh.tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tmem_fence_before();
    __syncthreads();
    tmem_fence_after();
    const int quarter = warp & 3;                    // a warp reaches tensor-memory lanes 32*(warp%4)..+31 only
    const uint32_t tbase = sh.tmem_base + (static_cast<uint32_t>(32 * quarter) << 16);

    bool dead = false;                               // a bounded wait of this thread ran out

    if (warp == kProducerWarp) {
        // ================= producer: one lane streams this CTA's slices, pair after pair =================
        if (lane == 0) {
            uint32_t gg = 0;
            for (int item = group_id; item < P.n_items; item += n_groups) {
                const int b = item / P.G, i = item - b * P.G;
                int trow = i;
                if (P.parent != nullptr) {
                    const int par = __ldg(P.parent + item);
                    trow = (par >= -1 && par < i) ? par + 1 : 0;       // an invalid node still moves (ignored) data
                }
                const char* a_src = static_cast<const char*>(P.target) + (static_cast<size_t>(b) * (P.G + 1) + trow) * row_bytes +
                                    static_cast<size_t>(vbeg) * 16;
                const char* b_src = static_cast<const char*>(P.draft) + (static_cast<size_t>(b) * P.G + i) * row_bytes +
                                    static_cast<size_t>(vbeg) * 16;
                for (int s = 0; s < ns; ++s, ++gg) {
                    const uint32_t slot = gg % kRing;
                    if (gg >= kRing) mbar_wait(&sh.empty[slot], ((gg / kRing) - 1) & 1, P.timeout_flag, dead);
                    if (dead) break;                 // nothing more is copied once a wait has run out
                    const int v0 = s * kStageVecs;
                    const int nv = (vcnt - v0) < kStageVecs ? (vcnt - v0) : kStageVecs;
                    const uint32_t bytes = static_cast<uint32_t>(nv) * 16;
                    unsigned char* dst = ring + slot * kStageBytes;
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // earlier reads of the slot precede the async writes
                    mbar_arrive_expect_tx(&sh.full[slot], 2 * bytes);
                    bulk_g2s(dst, a_src + static_cast<size_t>(v0) * 16, bytes, &sh.full[slot]);
                    bulk_g2s(dst + kStageRowBytes, b_src + static_cast<size_t>(v0) * 16, bytes, &sh.full[slot]);
                }
                if (dead) break;
            }
            // Every copy this lane issued has landed before the CTA may leave (normally the first
            // sweep consumed them long ago and these waits return at once).
            const uint32_t first = gg > kRing ? gg - kRing : 0;
            for (uint32_t k = first; k < gg; ++k) {
#pragma unroll 1
                for (uint32_t t = 0; t < kSpinLimit; ++t)
                    if (mbar_try_wait(&sh.full[k % kRing], (k / kRing) & 1)) break;
            }
        }
        __syncwarp();
    } else if (warp < kS1Warps) {
        // ================= first sweep =================
        const int j = warp >> 2;                     // which of the quarter's first-sweep warps
        const uint64_t l2 = pack2(kLog2e, kLog2e);
        uint32_t gg = 0;
        uint32_t li = 0;
        for (int item = group_id; item < P.n_items; item += n_groups, ++li) {
            const int ps = static_cast<int>(li % kPairDepth);
            float ka = -INFINITY, kb = -INFINITY;    // warp-uniform references; -inf: not taken yet
            uint64_t ca2 = 0, cb2 = 0;               // packed -k (0 while no finite logit has been seen)
            uint64_t za2[VPT], zb2[VPT], sa2[VPT], sb2[VPT];
#pragma unroll
            for (int v = 0; v < VPT; ++v) { za2[v] = 0; zb2[v] = 0; sa2[v] = 0; sb2[v] = 0; }
            float kk = 0.f;
            uint32_t diff = 0;

            auto stage = [&](auto tail_tag, int s) {
                constexpr bool TAIL = decltype(tail_tag)::value;
                const uint32_t slot = gg % kRing, chunk = gg % NCH;
                mbar_wait(&sh.full[slot], (gg / kRing) & 1, P.timeout_flag, dead);
                const unsigned char* st = ring + slot * kStageBytes + (warp * 32 + lane) * 16;
                uint4 va[VPT], vb[VPT];
                bool any[VPT];                       // warp-uniform: some lane of the warp has this vector
#pragma unroll
                for (int v = 0; v < VPT; ++v) {
                    any[v] = true;
                    bool mine = true;
                    if constexpr (TAIL) {
                        const int left = vcnt - (s * kStageVecs + v * (kS1Warps * 32) + warp * 32);
                        any[v] = left > 0;
                        mine = lane < left;
                    }
                    va[v] = make_uint4(kNegInfVec, kNegInfVec, kNegInfVec, kNegInfVec);
                    vb[v] = va[v];
                    if (mine) {
                        va[v] = *reinterpret_cast<const uint4*>(st + v * (kS1Warps * 32 * 16));
                        vb[v] = *reinterpret_cast<const uint4*>(st + kStageRowBytes + v * (kS1Warps * 32 * 16));
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.empty[slot]);     // the slot may be refilled: every lane's vectors are loaded
#pragma unroll
                for (int v = 0; v < VPT; ++v) {
                    diff |= (va[v].x ^ vb[v].x) | (va[v].y ^ vb[v].y) | (va[v].z ^ vb[v].z) | (va[v].w ^ vb[v].w);
                    if constexpr (DT == FSD_BF16) {
                        // -inf logits are read as -1e30: 2^y = 0 and 0 * y = 0 stay finite; NaN passes through
                        constexpr uint32_t kClamp2 = 0xF149F149u;
                        va[v].x = bf16x2_max_nan(va[v].x, kClamp2); va[v].y = bf16x2_max_nan(va[v].y, kClamp2);
                        va[v].z = bf16x2_max_nan(va[v].z, kClamp2); va[v].w = bf16x2_max_nan(va[v].w, kClamp2);
                        if constexpr (DIV != FSD_DIV_KL) {        // KL needs the draft's -inf: q = 0 < p gives +inf
                            vb[v].x = bf16x2_max_nan(vb[v].x, kClamp2); vb[v].y = bf16x2_max_nan(vb[v].y, kClamp2);
                            vb[v].z = bf16x2_max_nan(vb[v].z, kClamp2); vb[v].w = bf16x2_max_nan(vb[v].w, kClamp2);
                        }
                    } else {
                        constexpr float kClamp = -1.0e30f;
                        va[v].x = __float_as_uint(fmax_nan(__uint_as_float(va[v].x), kClamp)); va[v].y = __float_as_uint(fmax_nan(__uint_as_float(va[v].y), kClamp));
                        va[v].z = __float_as_uint(fmax_nan(__uint_as_float(va[v].z), kClamp)); va[v].w = __float_as_uint(fmax_nan(__uint_as_float(va[v].w), kClamp));
                        if constexpr (DIV != FSD_DIV_KL) {
                            vb[v].x = __float_as_uint(fmax_nan(__uint_as_float(vb[v].x), kClamp)); vb[v].y = __float_as_uint(fmax_nan(__uint_as_float(vb[v].y), kClamp));
                            vb[v].z = __float_as_uint(fmax_nan(__uint_as_float(vb[v].z), kClamp)); vb[v].w = __float_as_uint(fmax_nan(__uint_as_float(vb[v].w), kClamp));
                        }
                    }
                }
                if (ka == -INFINITY || kb == -INFINITY) {
                    // The warp has met no finite logit in one of the rows yet (normally: this is the
                    // pair's first stage): take the reference from the largest logit of this stage.
                    float ma = -INFINITY, mb = -INFINITY;
#pragma unroll
                    for (int v = 0; v < VPT; ++v) {
                        if constexpr (DT == FSD_BF16) {
                            const uint32_t pa = bf16x2_max_nan(bf16x2_max_nan(va[v].x, va[v].y), bf16x2_max_nan(va[v].z, va[v].w));
                            const uint32_t pb = bf16x2_max_nan(bf16x2_max_nan(vb[v].x, vb[v].y), bf16x2_max_nan(vb[v].z, vb[v].w));
                            ma = fmax_nan(ma, fmax_nan(bf16_lo(pa), bf16_hi(pa)));
                            mb = fmax_nan(mb, fmax_nan(bf16_lo(pb), bf16_hi(pb)));
                        } else {
                            ma = fmax_nan(ma, fmax_nan(fmax_nan(__uint_as_float(va[v].x), __uint_as_float(va[v].y)),
                                                       fmax_nan(__uint_as_float(va[v].z), __uint_as_float(va[v].w))));
                            mb = fmax_nan(mb, fmax_nan(fmax_nan(__uint_as_float(vb[v].x), __uint_as_float(vb[v].y)),
                                                       fmax_nan(__uint_as_float(vb[v].z), __uint_as_float(vb[v].w))));
                        }
                    }
                    ma = warp_max_nan(ma); mb = warp_max_nan(mb);
                    // a NaN maximum leaves the reference unset; the NaN reaches the sums and marks the pair
                    if (ka == -INFINITY && ma > -1.0e29f) { ka = ceilf(ma * kLog2e); ca2 = pack2(-ka, -ka); }
                    if (kb == -INFINITY && mb > -1.0e29f) { kb = ceilf(mb * kLog2e); cb2 = pack2(-kb, -kb); }
                }
                float e[VPT][EPT];
#pragma unroll
                for (int v = 0; v < VPT; ++v) {
                    if (TAIL && !any[v]) continue;
                    float xa[EPV], xb[EPV];
                    unpack_vec<DT>(va[v], xa);
                    unpack_vec<DT>(vb[v], xb);
#pragma unroll
                    for (int t = 0; t < EPV; t += 2) {
                        const uint64_t ya2 = fma2(pack2(xa[t], xa[t + 1]), l2, ca2), yb2 = fma2(pack2(xb[t], xb[t + 1]), l2, cb2);
                        float ya0, ya1, yb0, yb1;
                        unpack2(ya2, ya0, ya1);
                        unpack2(yb2, yb0, yb1);
                        const float ea0 = ex2(ya0), ea1 = ex2(ya1), eb0 = ex2(yb0), eb1 = ex2(yb1);
                        const uint64_t ea2 = pack2(ea0, ea1), eb2 = pack2(eb0, eb1);
                        za2[v] = add2(za2[v], ea2);
                        zb2[v] = add2(zb2[v], eb2);
                        if constexpr (DIV == FSD_DIV_JS) {
                            sa2[v] = fma2(ea2, ya2, sa2[v]);
                            sb2[v] = fma2(eb2, yb2, sb2[v]);
                        }
                        if constexpr (DIV == FSD_DIV_KL) {
                            if (ea0 > 0.f) kk = fmaf(ea0, ya0 - yb0, kk);
                            if (ea1 > 0.f) kk = fmaf(ea1, ya1 - yb1, kk);
                        }
                        e[v][t] = ea0; e[v][t + 1] = ea1;
                        e[v][EPV + t] = eb0; e[v][EPV + t + 1] = eb1;
                    }
                }
                if constexpr (kSecondSweep) {
                    // the chunk's previous values are in the second sweep's registers (every warp waits,
                    // also one with nothing to park, so that it never runs a phase ahead of the barrier)
                    if (gg >= NCH) mbar_wait(&sh.tfree[quarter][chunk], ((gg / NCH) - 1) & 1, P.timeout_flag, dead);
                    tmem_fence_after();
#pragma unroll
                    for (int v = 0; v < VPT; ++v) {
                        if (TAIL && !any[v]) continue;
                        tmem_st<EPT>(tbase + chunk * CPC + (j * VPT + v) * EPT, e[v]);
                    }
                }
                if constexpr (kSecondSweep) {
                    tmem_wait_st();
                    tmem_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sh.tfull[quarter][chunk]);
                }
                ++gg;
            };

            for (int s = 0; s < ns_full; ++s) stage(std::false_type{}, s);
            if (ns > ns_full) stage(std::true_type{}, ns_full);

            // ---- this warp's statistics (the reference is warp-uniform: plain sums) ----
            float za = 0.f, zb = 0.f, s0 = 0.f, sb = 0.f;
#pragma unroll
            for (int v = 0; v < VPT; ++v) {
                za += sum2(za2[v]); zb += sum2(zb2[v]);
                if constexpr (DIV == FSD_DIV_JS) { s0 += sum2(sa2[v]); sb += sum2(sb2[v]); }
            }
            if constexpr (DIV == FSD_DIV_KL) s0 = kk;
            const bool redo = !(za < kRangeLimit) || !(zb < kRangeLimit);     // NaN included
#pragma unroll
            for (int m = 16; m > 0; m >>= 1) {
                za += __shfl_xor_sync(0xffffffffu, za, m);
                zb += __shfl_xor_sync(0xffffffffu, zb, m);
                if constexpr (DIV != FSD_DIV_TV) s0 += __shfl_xor_sync(0xffffffffu, s0, m);
                if constexpr (DIV == FSD_DIV_JS) sb += __shfl_xor_sync(0xffffffffu, sb, m);
            }
            const uint32_t wdiff = (__reduce_or_sync(0xffffffffu, diff) != 0 ? kDiffRows : 0u) |
                                   (__any_sync(0xffffffffu, redo) ? kDiffRedo : 0u);
            // the slot's previous pair has been consumed by the second sweep (which read ws too)
            if (li >= kPairDepth) mbar_wait(&sh.pdone[ps], ((li / kPairDepth) - 1) & 1, P.timeout_flag, dead);
            int last = 0;
            if (lane == 0) {
                Stats mine;
                mine.ka = ka; mine.kb = kb; mine.za = za; mine.zb = zb; mine.s0 = s0; mine.sb = sb; mine.x = 0.f; mine.diff = wdiff;
                sh.ws[ps][warp] = mine;
                __threadfence_block();
                last = atomicAdd(&sh.s1_count[ps], 1) == kS1Warps - 1;
            }
            last = __shfl_sync(0xffffffffu, last, 0);
            if (last) {
                // ---- the CTA's part: fold the warps' statistics and publish ----
                __threadfence_block();
                Stats w;
                w.ka = -INFINITY; w.kb = -INFINITY; w.za = 0.f; w.zb = 0.f; w.s0 = 0.f; w.sb = 0.f; w.x = 0.f; w.diff = 0;
                if (lane < kS1Warps) w = sh.ws[ps][lane];
                Stats c;
                c.ka = warp_max_nan(w.ka); c.kb = warp_max_nan(w.kb);
                {
                    const float da = w.ka == -INFINITY ? 0.f : w.ka - c.ka, db = w.kb == -INFINITY ? 0.f : w.kb - c.kb;
                    const float fa = w.ka == -INFINITY ? 0.f : pow2_int(da), fb = w.kb == -INFINITY ? 0.f : pow2_int(db);
                    c.za = w.za * fa; c.zb = w.zb * fb;
                    c.s0 = DIV == FSD_DIV_KL ? scale_kl(fa, fmaf(da - db, w.za, w.s0)) : fa * fmaf(da, w.za, w.s0);
                    c.sb = fb * fmaf(db, w.zb, w.sb);
                }
#pragma unroll
                for (int m = 16; m > 0; m >>= 1) {
                    c.za += __shfl_xor_sync(0xffffffffu, c.za, m); c.zb += __shfl_xor_sync(0xffffffffu, c.zb, m);
                    c.s0 += __shfl_xor_sync(0xffffffffu, c.s0, m); c.sb += __shfl_xor_sync(0xffffffffu, c.sb, m);
                }
                c.diff = __reduce_or_sync(0xffffffffu, w.diff);
                if (lane == 0) {
                    sh.s1_count[ps] = 0;
                    PairRecord* r = P.records + item;
                    float4* dst = reinterpret_cast<float4*>(&r->part[rank]);
                    dst[0] = make_float4(c.ka, c.kb, c.za, c.zb);
                    dst[1] = make_float4(c.s0, c.sb, 0.f, __uint_as_float(c.diff));
                    if (rank == 0) {
                        bool bad = false;
                        if (P.parent != nullptr) {
                            const int pr = __ldg(P.parent + item);
                            bad = pr < -1 || pr >= item % P.G;
                        }
                        r->ncta = static_cast<uint32_t>(G);
                        r->state = bad ? kRecordBadTree : kRecordStats;
                    }
                    red_release_add(P.arrived + item, 1);
                }
                __syncwarp();
            }
        }
    } else {
        // ================= second sweep, one pair behind =================
        uint32_t cc = 0;
        uint32_t li = 0;
        for (int item = group_id; item < P.n_items; item += n_groups, ++li) {
            const int ps = static_cast<int>(li % kPairDepth);
            // ---- all G parts of the pair are in its record ----
            if (!dead) {
                bool ok = false;
#pragma unroll 1
                for (uint32_t t = 0; t < P.poll_limit; ++t) {
                    if (ld_acquire(P.arrived + item) >= G) { ok = true; break; }
                    if ((t & 255u) == 255u && *reinterpret_cast<volatile int*>(P.timeout_flag) != 0) break;
                }
                if (!ok) { atomicExch(P.timeout_flag, 1); dead = true; }
            }
            float x = 0.f;
            if constexpr (kSecondSweep) {
                float pka = -INFINITY, pkb = -INFINITY, pza = 0.f, pzb = 0.f;
                if (lane < G) {
                    const float4 p = __ldcg(reinterpret_cast<const float4*>(&P.records[item].part[lane]));
                    pka = p.x; pkb = p.y; pza = p.z; pzb = p.w;
                }
                const float Ka = warp_max_nan(pka), Kb = warp_max_nan(pkb);
                float tza = pka == -INFINITY ? 0.f : pza * pow2_int(pka - Ka);
                float tzb = pkb == -INFINITY ? 0.f : pzb * pow2_int(pkb - Kb);
#pragma unroll
                for (int m = 16; m > 0; m >>= 1) {
                    tza += __shfl_xor_sync(0xffffffffu, tza, m); tzb += __shfl_xor_sync(0xffffffffu, tzb, m);
                }
                const bool ok = tza > 0.f && tzb > 0.f && tza < 3.0e38f && tzb < 3.0e38f;   // false for NaN too
                const float iza = ok ? 1.0f / tza : 0.f, izb = ok ? 1.0f / tzb : 0.f;
                uint64_t ia2[kS1PerQuarter], ib2[kS1PerQuarter];
#pragma unroll
                for (int j = 0; j < kS1PerQuarter; ++j) {
                    const float wka = sh.ws[ps][quarter + 4 * j].ka, wkb = sh.ws[ps][quarter + 4 * j].kb;
                    const float ia = (wka == -INFINITY || !ok) ? 0.f : pow2_int(wka - Ka) * iza;
                    const float ib = (wkb == -INFINITY || !ok) ? 0.f : pow2_int(wkb - Kb) * izb;
                    ia2[j] = pack2(ia, ia); ib2[j] = pack2(ib, ib);
                }
                // s = p + q + 1e-37 keeps lg2 finite where both terms vanish; the shift is below one ulp of any s that matters
                const uint64_t tiny2 = pack2(1e-37f, 1e-37f);
                uint64_t x2[2] = {0, 0};
                float xt = 0.f;
                for (int s = 0; s < ns; ++s, ++cc) {
                    const uint32_t chunk = cc % NCH;
                    mbar_wait(&sh.tfull[quarter][chunk], (cc / NCH) & 1, P.timeout_flag, dead);
                    tmem_fence_after();
                    float e[kS1PerQuarter * VPT][EPT];
                    bool have[kS1PerQuarter * VPT];
#pragma unroll
                    for (int j = 0; j < kS1PerQuarter; ++j) {
#pragma unroll
                        for (int v = 0; v < VPT; ++v) {
                            // the first-sweep warp parked this part iff some lane of it had the vector
                            have[j * VPT + v] = vcnt - (s * kStageVecs + v * (kS1Warps * 32) + (quarter + 4 * j) * 32) > 0;
                            if (have[j * VPT + v]) tmem_ld<EPT>(tbase + chunk * CPC + (j * VPT + v) * EPT, e[j * VPT + v]);
                        }
                    }
                    tmem_wait_ld();
                    tmem_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sh.tfree[quarter][chunk]);   // the chunk's values are in registers
#pragma unroll
                    for (int j = 0; j < kS1PerQuarter; ++j) {
#pragma unroll
                        for (int v = 0; v < VPT; ++v) {
                            if (!have[j * VPT + v]) continue;
                            const float (&ev)[EPT] = e[j * VPT + v];
#pragma unroll
                            for (int t = 0; t < EPV; t += 2) {
                                const uint64_t ea2 = pack2(ev[t], ev[t + 1]), eb2 = pack2(ev[EPV + t], ev[EPV + t + 1]);
                                if constexpr (DIV == FSD_DIV_JS) {
                                    const uint64_t s2 = fma2(eb2, ib2[j], fma2(ea2, ia2[j], tiny2));
                                    float s0, s1;
                                    unpack2(s2, s0, s1);
                                    x2[(t >> 1) & 1] = fma2(s2, pack2(lg2(s0), lg2(s1)), x2[(t >> 1) & 1]);
                                } else {
                                    // separately rounded products: a fused p - q would make TV(p, p) != 0
                                    const uint64_t d2 = fma2(mul2(eb2, ib2[j]), pack2(-1.f, -1.f), mul2(ea2, ia2[j]));
                                    float d0, d1;
                                    unpack2(d2, d0, d1);
                                    xt += fabsf(d0) + fabsf(d1);
                                }
                            }
                        }
                    }
                }
                x = sum2(x2[0]) + sum2(x2[1]) + xt;
#pragma unroll
                for (int m = 16; m > 0; m >>= 1) x += __shfl_xor_sync(0xffffffffu, x, m);
            }
            // ---- the CTA's second-sweep sum: the last warp to finish adds the four in a fixed order ----
            if (lane == 0) {
                sh.xs[ps][quarter] = x;
                __threadfence_block();
                if (atomicAdd(&sh.s2_count[ps], 1) == kS2Warps - 1) {
                    __threadfence_block();
                    sh.s2_count[ps] = 0;
                    P.records[item].x[rank] = (sh.xs[ps][0] + sh.xs[ps][1]) + (sh.xs[ps][2] + sh.xs[ps][3]);
                }
                mbar_arrive(&sh.pdone[ps]);
            }
            __syncwarp();
        }
    }

    // ---- release tensor memory ----
    tmem_fence_before();
    __syncthreads();
    if (warp == kProducerWarp) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(sh.tmem_base), "r"(kTmemCols) : "memory");
    }
}

}  // namespace fsd
