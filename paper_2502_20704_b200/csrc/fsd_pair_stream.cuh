// Streaming per-(row, position) kernel: every logit is read from HBM once.
//
// A (row, position) pair is split along the vocabulary over a GROUP of C virtual CTAs (C <= 16,
// chosen by the host from the slice that fits on chip and the number of pairs).  A CTA of 512
// threads, one per SM, holds two virtual CTAs of 256 threads, each with its own half of the SM's
// tensor memory, its own shared-memory ring and its own named barriers; the two belong to
// different groups, so that one computes while the other waits for its group.  The launch is
// cooperative (all CTAs resident: the virtual CTAs of a group wait for one another) and the groups
// are persistent: they claim pairs from a shared counter.  Per pair, each virtual CTA
//   1. receives its slice of both rows in shared memory through a ring of bulk asynchronous
//      copies (cp.async.bulk + mbarrier).  A warp releases a slot as soon as its vectors are in
//      registers; the slot is refilled one stage later by a rotating duty warp, so the next
//      pair's slices stream in while this pair is finished and nobody waits for a slot to drain;
//   2. sweeps each stage once as it lands: e = 2^(logit * log2e - k) with one MUFU ex2 per
//      logit, the sums Z = sum e and S = sum e*y (or the KL sum), a bitwise "rows differ" flag,
//      and parks the e values in tensor memory (128 per thread) and registers (32).  k is a
//      per-thread integer reference in the log2 domain, taken from the thread's first finite
//      logits and moved -- with an exact power-of-two rescale of what has been summed and parked
//      -- only if a later logit exceeds it by more than 2^30, so no separate maximum pass over
//      the slice is needed and every change of reference is exact;
//   3. combines (k, Z, S) over threads and warps; one combiner warp per virtual CTA (rotating)
//      folds the warps' statistics, leaves them as a tagged message in global memory, fetches the
//      messages of the whole group (they live in L2), folds those and wakes the virtual CTA
//      (named barriers: waiting warps issue nothing);
//   4. sweeps the parked e values: p = e_a/Z_a, q = e_b/Z_b; JS needs sum (p+q) log2(p+q) (one
//      MUFU lg2 per pair), TV needs sum |p - q|; KL needs no second sweep.
// The group's rank-0 virtual CTA leaves all members' statistics in the pair's record; the finish
// kernel folds them in double precision and turns them into divergences and accept bits, so no
// double-precision arithmetic runs here.  HBM traffic is the algorithmic minimum.  The
// special-function pipe (1 ex2 per logit + 1 lg2 per pair) and instruction issue are the
// co-bottlenecks, which is why e values are kept rather than recomputed, and why a thread
// owns two vectors per row and stage (independent work to overlap its own latencies) with 512
// threads of 128 registers per SM.  Groups need no co-scheduling on neighbouring SMs, so every
// SM is used whatever C is.
#pragma once

#include "fsd_device.cuh"

namespace fsd {

constexpr int kStreamThreads = 256;
constexpr int kStreamWarps = kStreamThreads / 32;
constexpr int kRing = 6;                                   // stages in the shared-memory ring
constexpr int kVecPerThread = 2;                           // 16-byte vectors per thread, row and stage
constexpr int kStageVecs = kStreamThreads * kVecPerThread; // vectors per row and stage
constexpr int kStageRowBytes = kStageVecs * 16;
constexpr int kStageBytes = 2 * kStageRowBytes;
constexpr int kMaxStagesPerPair = kRing - 1;               // stages of e values a thread can park (4 in tensor memory, 1 in registers)
constexpr int kTmemCols = 256;                             // per virtual CTA: 8 warps -> 2 per lane quarter x 128 columns
constexpr int kTmemPerThread = 128;
constexpr int kMaxVecPerCta = kMaxStagesPerPair * kStageVecs;
constexpr int kMaxClusterSize = 8;                        // finish kernel (portable size)
constexpr int kMaxGroupSize = 16;                      // most virtual CTAs in a group of the streaming kernel
constexpr uint32_t kSpinLimit = 1u << 24;                  // polls before a wait gives up

// Partial statistics of one (target row, draft row) pair: of a warp, of a virtual CTA, or -- in a
// pair's record -- of each virtual CTA of the group that streamed the pair.
//   z = sum 2^y, s = sum 2^y * y with y = logit*log2e - k and k the integer reference (log2
//   domain) the sums are relative to.  s0 is the target row's s for JS and the KL sum
//   sum 2^ya (ya - yb) for KL.
struct alignas(16) Stats {
    float ka, kb;              // references; -inf: no finite logit seen; NaN: a NaN logit
    float za, zb;
    float s0, sb;
    float x;                   // second-sweep sum of the PREVIOUS pair (in flight only)
    uint32_t diff;             // 0: the two rows are bitwise identical so far (bit 0 once a virtual CTA has folded
                               // it; rank 0's message carries the next claimed pair id in the bits above)
};
static_assert(sizeof(Stats) == 32, "Stats travels as two 16-byte stores");

// What the streaming kernel leaves per pair for the finish kernel, which folds the parts in
// double precision (second-sweep sums: JS sum s log2 s, TV sum |p - q|).
struct alignas(16) PairRecord {
    Stats part[kMaxGroupSize];
    float x[kMaxGroupSize];  // each virtual CTA's second-sweep sum of this pair
    uint32_t ncta;             // parts in use
    uint32_t state;            // kRecordStats | kRecordBadTree
    uint32_t pad[2];
};
static_assert(sizeof(PairRecord) == 592, "PairRecord layout");
constexpr uint32_t kRecordStats = 1, kRecordBadTree = 2;

// One virtual CTA's statistics of a round as they cross global memory: three 16-byte units, each
// stored whole and ending in the round's tag, so that a reader knows a unit is this round's
// without any fence or flag (a unit whose tag is older is fetched again).
struct alignas(16) GroupMsg {
    uint4 u[3];                // {ka, kb, za, tag}, {zb, s0, sb, tag}, {x, diff | next pair id << 1, 0, tag}
    uint4 pad;
};
static_assert(sizeof(GroupMsg) == 64, "GroupMsg layout");

struct StreamParams {
    const void* target;        // [B, G+1, V]
    const void* draft;         // [B, G,   V]
    const int32_t* parent;     // [B, G] (tree) or null (chain)
    int B, G;
    int nvec_row;              // 16-byte vectors per logit row
    int n_items;               // B * G
    PairRecord* records;       // [B * G]
    int* timeout_flag;         // set to 1 if a bounded wait ran out; zero at launch
    int* next_pair;            // pairs handed out beyond each group's fixed first ones; zero at launch
    int C;                     // virtual CTAs per group (<= kMaxGroupSize)
    uint32_t poll_limit;       // fetches of the group's messages before the exchange gives up (kSpinLimit normally)
    int silent_rank;           // test aid: this rank of group 0 keeps its first message to itself (-1: nobody)
    GroupMsg* exchange;        // [groups][2][C], zero at launch
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
        // somebody has given up already: nothing this thread waits for is certain to come
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

// NaN-propagating maxima: a NaN logit must reach the row maximum so that the row is flagged
__device__ __forceinline__ uint32_t bf16x2_max_nan(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t bf16x2_max(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
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

// ---- in-stream references ---------------------------------------------------------------------
// A thread keeps, per row, the largest logit its reference may meet without moving: bf16 rows
// hold it as a packed pair so that one packed maximum tests a whole vector.  -1e30 is what -inf
// logits are read as, so "nothing finite seen yet" is a limit of exactly that.
template <int DT> __device__ __forceinline__ uint32_t unset_limit() {
    return DT == FSD_BF16 ? 0xF149F149u : __float_as_uint(-1.0e30f);
}
// limit for a reference taken from maximum m: m + 30 ln 2, rounded to the row's type (rounding
// can add at most another 30 ln 2 before it snaps back to m itself, so 2^y stays below 2^61)
template <int DT> __device__ __forceinline__ uint32_t reference_limit(float m) {
    const float lim = m + 20.7944f;
    if constexpr (DT == FSD_BF16) {
        uint32_t r;
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(lim), "f"(lim));
        return r;
    } else {
        return __float_as_uint(lim);
    }
}
// Multiplies the e values a warp has parked in tensor memory for stages 0..n-1 by fa (first
// half of each stage: target row) and fb (second half: draft row).  Warp-collective.
template <int EPT>
__device__ __noinline__ void rescale_parked(uint32_t taddr, int n, float fa, float fb) {
    tmem_wait_st();
    for (int t = 0; t < n; ++t) {
        float e[EPT];
        tmem_ld<EPT>(taddr + t * EPT, e);
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < EPT / 2; ++j) { e[j] *= fa; e[EPT / 2 + j] *= fb; }
        tmem_st<EPT>(taddr + t * EPT, e);
    }
    tmem_wait_st();
}

// A KL partial sum brought to another reference: +inf (a logit with p > 0 = q) stays +inf even
// when the factor underflows to 0
__device__ __forceinline__ float scale_kl(float f, float v) { return v == INFINITY ? v : f * v; }

// Named barriers of one virtual CTA: waiting warps issue nothing.  `arrive` counts the warp in
// without waiting; `sync` waits until kStreamThreads threads have arrived or synced.  The second
// virtual CTA of a CTA uses ids two higher.
__device__ __forceinline__ void named_arrive(int id) {
    asm volatile("bar.arrive %0, %1;" ::"r"(id), "n"(kStreamThreads) : "memory");
}
__device__ __forceinline__ void named_sync(int id) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "n"(kStreamThreads) : "memory");
}
constexpr int kBarPosted = 1, kBarTotals = 2;

// One unit is stored and fetched as a single 128-bit access (the .b128 forms: one access, not four
// that happen to be adjacent), so a reader sees a unit either whole or not at all.
__device__ __forceinline__ void st_unit(uint4* p, float a, float b, float c, uint32_t tag) {
    const uint64_t lo = static_cast<uint64_t>(__float_as_uint(a)) | (static_cast<uint64_t>(__float_as_uint(b)) << 32);
    const uint64_t hi = static_cast<uint64_t>(__float_as_uint(c)) | (static_cast<uint64_t>(tag) << 32);
    asm volatile("{ .reg .b128 t; mov.b128 t, {%1, %2}; st.relaxed.gpu.global.b128 [%0], t; }" ::"l"(p), "l"(lo), "l"(hi) : "memory");
}
__device__ __forceinline__ uint4 ld_unit(const uint4* p) {
    uint64_t lo, hi;
    asm volatile("{ .reg .b128 t; ld.relaxed.gpu.global.b128 t, [%2]; mov.b128 {%0, %1}, t; }" : "=l"(lo), "=l"(hi) : "l"(p) : "memory");
    return make_uint4(static_cast<uint32_t>(lo), static_cast<uint32_t>(lo >> 32), static_cast<uint32_t>(hi), static_cast<uint32_t>(hi >> 32));
}

// ---- shared-memory layout ---------------------------------------------------------------
struct StreamShared {
    uint64_t full[kRing];      // a ring stage has landed
    uint64_t empty[kRing];     // every warp has finished reading the slot's current stage
    uint32_t armed[kRing];     // copies started into each ring slot so far (the last one is waited for before leaving)
    int items[8];              // pair ids of this group's rounds, indexed by round & 7
    alignas(16) float tot[4];  // group totals of the current pair: Ka, Kb, Za, Zb
    Stats ws[kStreamWarps];    // the warps' statistics of the current pair
};
constexpr int kStreamHalves = 2;                            // virtual CTAs per CTA
constexpr int kStreamCtaThreads = kStreamHalves * kStreamThreads;
constexpr size_t kStreamHalfBytes = kRing * kStageBytes + ((sizeof(StreamShared) + 127) / 128) * 128;
constexpr size_t kStreamSmemBytes = kStreamHalves * kStreamHalfBytes + 128 + 16;

template <int DT, int DIV>
__global__ void __launch_bounds__(kStreamCtaThreads, 1) fsd_pair_stream_kernel(StreamParams P) {
    constexpr int EPV = Logit<DT>::kPerVec;          // logits per 16-byte vector
    constexpr int EPT = 2 * EPV;                     // e values per thread and vector position (both rows)
    constexpr int VPT = kVecPerThread;
    constexpr int EPS = VPT * EPT;                   // e values per thread and stage
    constexpr int NT = (kTmemPerThread / EPS) < kMaxStagesPerPair ? (kTmemPerThread / EPS) : kMaxStagesPerPair;
    constexpr int NR = kMaxStagesPerPair - NT;       // stages kept in registers
    constexpr bool kSecondSweep = DIV != FSD_DIV_KL;
    constexpr float kClamp = -1.0e30f;               // -inf logits are read as this: 2^y = 0 and 0 * y = 0 stay finite

    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    const int half = threadIdx.x / kStreamThreads;   // which virtual CTA of this CTA
    unsigned char* ring = smem + half * kStreamHalfBytes;
    StreamShared& sh = *reinterpret_cast<StreamShared*>(ring + kRing * kStageBytes);
    uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(smem + kStreamHalves * kStreamHalfBytes);

    const int C = P.C;
    // numbered half by half, so that the two virtual CTAs of an SM belong to different groups: while one
    // waits for its group's statistics the other has the SM to itself
    const int vid = half * static_cast<int>(gridDim.x) + static_cast<int>(blockIdx.x);
    const int n_groups = (kStreamHalves * static_cast<int>(gridDim.x)) / C;     // groups
    const int group_id = vid / C, rank = vid - group_id * C;
    const bool active = group_id < n_groups;     // the virtual CTAs left over form no group
    const int tid = threadIdx.x % kStreamThreads, lane = tid & 31, warp = tid >> 5;
    const int bar_posted = kBarPosted + 2 * half, bar_totals = kBarTotals + 2 * half;

    // this virtual CTA's slice of every row, in vectors
    const int base = P.nvec_row / C, rem = P.nvec_row % C;
    const int vbeg = rank * base + (rank < rem ? rank : rem);
    const int vcnt = base + (rank < rem ? 1 : 0);
    const int ns = (vcnt + kStageVecs - 1) / kStageVecs;             // stages per pair (<= kMaxStagesPerPair)
    const size_t row_bytes = static_cast<size_t>(P.nvec_row) * 16;

    // ---- set-up: barriers, tensor memory ----
    // A group's first `ahead` pairs are fixed (group_id + round * n_groups): that is as far
    // as the ring reads ahead.  Every later pair is the next one nobody has taken yet, claimed
    // `ahead` rounds early by rank 0 and sent round with that round's statistics, so groups
    // that happen to run faster take more pairs and all finish together.
    // (from the smallest slice of the group, so that every member computes the same value
    // whatever its own slice: the members must agree on which pairs are fixed and where a claimed
    // id is kept; a member with one stage more per pair reads ahead less far, so the ids it needs
    // are there even earlier)
    const int ns_min = (base + kStageVecs - 1) / kStageVecs;
    const int ahead = 2 + (kRing - 2) / (ns_min > 0 ? ns_min : 1);
    if (tid == 0) {
        for (int k = 0; k < ahead; ++k) sh.items[k] = group_id + k * n_groups;
        for (int s = 0; s < kRing; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], kStreamWarps); sh.armed[s] = 0; }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x < 32) {                          // one allocation for both virtual CTAs: all of the SM's columns
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_base_slot)), "r"(kStreamHalves * kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    // warp w of a virtual CTA owns tensor-memory lanes 32*(w%4)..+31 and columns kTmemCols*half + kTmemPerThread*(w/4)..
    const uint32_t taddr = *tmem_base_slot + (static_cast<uint32_t>(32 * (warp & 3)) << 16) +
                           static_cast<uint32_t>(kTmemCols * half + kTmemPerThread * (warp >> 2));
    // where this group's virtual CTAs exchange their statistics: [parity][rank] messages
    GroupMsg* const xg = P.exchange + static_cast<size_t>(group_id < n_groups ? group_id : 0) * 2 * C;

    bool dead = false;                               // a bounded wait of this thread ran out

    // ---- producer: stage number -> (pair, slice part); any thread may issue a stage ----
    // Stage gg of this virtual CTA is part gg % ns of the (gg / ns)-th pair of its group (its id is in
    // sh.items).  Stage gg + kRing is issued by the duty warp of stage gg + 1 (see the first sweep), so the
    // copies go out early and the work is spread over the warps.
    auto issue_stage = [&](uint32_t gg) {
        const uint32_t k = gg / static_cast<uint32_t>(ns), s = gg - k * static_cast<uint32_t>(ns);
        const int item = sh.items[k & 7];
        if (item >= P.n_items) return;
        FSD_CHECK(P.timeout_flag + 2, item >= 0, kChkItem);
        const int b = item / P.G, i = item - b * P.G;
        int trow = i;
        if (P.parent != nullptr) {
            const int par = __ldg(P.parent + item);
            trow = (par >= -1 && par < i) ? par + 1 : 0;       // an invalid node still moves (ignored) data
        }
        const char* a_row = static_cast<const char*>(P.target) + (static_cast<size_t>(b) * (P.G + 1) + trow) * row_bytes;
        const char* b_row = static_cast<const char*>(P.draft) + (static_cast<size_t>(b) * P.G + i) * row_bytes;
        const uint32_t slot = gg % kRing;
        const int v0 = static_cast<int>(s) * kStageVecs;
        const int nv = (vcnt - v0) < kStageVecs ? (vcnt - v0) : kStageVecs;
        const uint32_t bytes = static_cast<uint32_t>(nv) * 16;
        FSD_CHECK(P.timeout_flag + 2, nv > 0 && vbeg + v0 + nv <= P.nvec_row && bytes <= kStageRowBytes, kChkSlice);
        FSD_CHECK(P.timeout_flag + 2, s < static_cast<uint32_t>(ns) && ns <= kMaxStagesPerPair && trow >= 0 && trow <= P.G, kChkStage);
        unsigned char* dst = ring + slot * kStageBytes;
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // earlier reads of the slot precede the async writes
        sh.armed[slot] += 1;                         // one thread at a time starts copies into a slot
        mbar_arrive_expect_tx(&sh.full[slot], 2 * bytes);
        bulk_g2s(dst, a_row + (static_cast<size_t>(vbeg) + v0) * 16, bytes, &sh.full[slot]);
        bulk_g2s(dst + kStageRowBytes, b_row + (static_cast<size_t>(vbeg) + v0) * 16, bytes, &sh.full[slot]);
    };
    if (tid == 0 && active) {
        for (uint32_t gg = 0; gg < kRing; ++gg) issue_stage(gg);
    }
    __syncwarp();

    float ereg[(NR > 0 ? NR : 1) * EPS];
    uint32_t g = 0;                                  // first ring stage of the current pair
    uint32_t li = 0;                                 // pairs this group has finished
    float x_carry = 0.f;                             // previous pair's second-sweep sum of this warp
    int prev_item = -1;                              // pair whose second-sweep sum is still to be published
    int item = active ? group_id : P.n_items;
    uint32_t claimed = 0;                            // rank 0, combiner lane 0: the pair id taken this round

    for (;;) {
        const bool live = item < P.n_items;          // one extra round publishes the last pair's second sweep
        if (!live && prev_item < 0) break;
        const int par = static_cast<int>(li & 1);
        const uint32_t tag = li + 1;                 // what this round's messages carry (never 0, the buffer's initial state)
        if (kSecondSweep && rank == 0 && lane == 0 && warp == static_cast<int>(li & (kStreamWarps - 1))) {
            // asked now, needed only when the statistics go out
            const long long id = static_cast<long long>(ahead) * n_groups + atomicAdd(P.next_pair, 1);
            claimed = id < 0x3fffffffLL ? static_cast<uint32_t>(id) : 0x3fffffffu;
        }
        bool bad = false;
        if (live && P.parent != nullptr) {
            const int i = item % P.G;
            const int pr = __ldg(P.parent + item);
            bad = pr < -1 || pr >= i;
        }

        // ---- first sweep: exponentials, sums, park the e values; then this warp's statistics ----
        float ka = -INFINITY, kb = -INFINITY;
        Stats mine;
        mine.ka = -INFINITY; mine.kb = -INFINITY; mine.za = 0.f; mine.zb = 0.f; mine.s0 = 0.f; mine.sb = 0.f;
        mine.diff = 0;
        if (live) {
            float kk = 0.f;
            uint32_t diff = 0;
            uint64_t za2 = 0, zb2 = 0, sa2 = 0, sb2 = 0;     // packed (even, odd) partial sums
            // Integer references in the log2 domain, y = logit*log2e - k.  A thread takes k from the
            // first vector that holds a finite logit and keeps it while no later logit exceeds it by
            // more than about 2^30 (2^60 at most); a larger one moves the reference and rescales what
            // has been summed and parked, by an exact power of two.
            uint32_t lima = unset_limit<DT>(), limb = unset_limit<DT>(); // a vector maximum above this moves the reference
            uint64_t ca2 = 0, cb2 = 0;                       // packed -k (0 while no finite logit has been seen)
            const uint64_t l2 = pack2(kLog2e, kLog2e);
#pragma unroll
            for (int s = 0; s < kMaxStagesPerPair; ++s) {
                if (s < ns) {
                    const uint32_t gs = g + s, slot = gs % kRing;
                    mbar_wait(&sh.full[slot], (gs / kRing) & 1, P.timeout_flag, dead);
                    // this thread's vectors of the stage: v * kStreamThreads + tid, v < VPT
                    uint4 va[VPT], vb[VPT];
                    bool has[VPT];
                    float ma = 0.f, mb = 0.f;                // maxima of this thread's vectors of the stage
                    bool fire_a = false, fire_b = false;
                    {
                        uint32_t pa = unset_limit<DT>(), pb = unset_limit<DT>();   // -1e30: below every clamped logit
#pragma unroll
                        for (int v = 0; v < VPT; ++v) {
                            has[v] = s * kStageVecs + v * kStreamThreads + tid < vcnt;
                            va[v] = make_uint4(0, 0, 0, 0); vb[v] = make_uint4(0, 0, 0, 0);
                            if (has[v]) {
                                const unsigned char* st = ring + slot * kStageBytes + (v * kStreamThreads + tid) * 16;
                                va[v] = *reinterpret_cast<const uint4*>(st);
                                vb[v] = *reinterpret_cast<const uint4*>(st + kStageRowBytes);
                                diff |= (va[v].x ^ vb[v].x) | (va[v].y ^ vb[v].y) | (va[v].z ^ vb[v].z) | (va[v].w ^ vb[v].w);
                                if constexpr (DT == FSD_BF16) {
                                    constexpr uint32_t kClamp2 = 0xF149F149u;     // bf16x2 (-1e30, -1e30); NaN passes through
                                    va[v].x = bf16x2_max_nan(va[v].x, kClamp2); va[v].y = bf16x2_max_nan(va[v].y, kClamp2);
                                    va[v].z = bf16x2_max_nan(va[v].z, kClamp2); va[v].w = bf16x2_max_nan(va[v].w, kClamp2);
                                    if constexpr (DIV != FSD_DIV_KL) {            // KL needs the draft's -inf: q = 0 < p gives +inf
                                        vb[v].x = bf16x2_max_nan(vb[v].x, kClamp2); vb[v].y = bf16x2_max_nan(vb[v].y, kClamp2);
                                        vb[v].z = bf16x2_max_nan(vb[v].z, kClamp2); vb[v].w = bf16x2_max_nan(vb[v].w, kClamp2);
                                    }
                                    pa = bf16x2_max_nan(pa, bf16x2_max_nan(bf16x2_max_nan(va[v].x, va[v].y), bf16x2_max_nan(va[v].z, va[v].w)));
                                    pb = bf16x2_max_nan(pb, bf16x2_max_nan(bf16x2_max_nan(vb[v].x, vb[v].y), bf16x2_max_nan(vb[v].z, vb[v].w)));
                                } else {
                                    const float m1 = fmax_nan(fmax_nan(__uint_as_float(va[v].x), __uint_as_float(va[v].y)),
                                                              fmax_nan(__uint_as_float(va[v].z), __uint_as_float(va[v].w)));
                                    const float m2 = fmax_nan(fmax_nan(__uint_as_float(vb[v].x), __uint_as_float(vb[v].y)),
                                                              fmax_nan(__uint_as_float(vb[v].z), __uint_as_float(vb[v].w)));
                                    pa = __float_as_uint(fmax_nan(__uint_as_float(pa), m1));
                                    pb = __float_as_uint(fmax_nan(__uint_as_float(pb), m2));
                                }
                            }
                        }
                        if constexpr (DT == FSD_BF16) {
                            fire_a = bf16x2_max_nan(pa, lima) != lima;
                            fire_b = bf16x2_max_nan(pb, limb) != limb;
                            if (fire_a) ma = fmax_nan(bf16_lo(pa), bf16_hi(pa));
                            if (fire_b) mb = fmax_nan(bf16_lo(pb), bf16_hi(pb));
                        } else {
                            ma = __uint_as_float(pa); mb = __uint_as_float(pb);
                            fire_a = !(ma <= __uint_as_float(lima));      // NaN moves the reference too
                            fire_b = !(mb <= __uint_as_float(limb));
                        }
                    }
                    __syncwarp();
                    if (__any_sync(0xffffffffu, fire_a || fire_b)) {
                        // rare after a pair's first vector: lanes that did not fire scale by 1
                        const float nka = fire_a ? ceilf(ma * kLog2e) : ka, nkb = fire_b ? ceilf(mb * kLog2e) : kb;
                        const float da = ka == -INFINITY ? 0.f : ka - nka, db = kb == -INFINITY ? 0.f : kb - nkb;
                        const float fa = ka == -INFINITY ? 0.f : pow2_int(da), fb = kb == -INFINITY ? 0.f : pow2_int(db);
                        const uint64_t fa2 = pack2(fa, fa), fb2 = pack2(fb, fb);
                        if constexpr (DIV == FSD_DIV_KL) kk = scale_kl(fa, fmaf(da - db, sum2(za2), kk));
                        sa2 = mul2(fma2(za2, pack2(da, da), sa2), fa2); za2 = mul2(za2, fa2);
                        sb2 = mul2(fma2(zb2, pack2(db, db), sb2), fb2); zb2 = mul2(zb2, fb2);
                        if constexpr (kSecondSweep) {
                            if (s > 0) rescale_parked<EPT>(taddr, (s < NT ? s : NT) * VPT, fa, fb);
#pragma unroll
                            for (int t = NT; t < s; ++t) {
#pragma unroll
                                for (int v = 0; v < VPT; ++v) {
#pragma unroll
                                    for (int j = 0; j < EPV; ++j) {
                                        ereg[(t - NT) * EPS + v * EPT + j] *= fa;
                                        ereg[(t - NT) * EPS + v * EPT + EPV + j] *= fb;
                                    }
                                }
                            }
                        }
                        if (fire_a) lima = reference_limit<DT>(ma);
                        if (fire_b) limb = reference_limit<DT>(mb);
                        ka = nka; kb = nkb;
                        const float ca = ka == -INFINITY ? 0.f : -ka, cb = kb == -INFINITY ? 0.f : -kb;
                        ca2 = pack2(ca, ca); cb2 = pack2(cb, cb);
                    }
                    // This warp is done with the slot: every lane's vectors are in registers (the vote
                    // above consumed them).  Nobody waits for the slot to drain: one stage later, when
                    // every warp has long left it, this stage's duty warp refills it.
                    if (lane == 0) {
                        mbar_arrive(&sh.empty[slot]);
                        if (gs > 0 && warp == static_cast<int>(gs % kStreamWarps)) {
                            const uint32_t ps = gs - 1;
                            mbar_wait(&sh.empty[ps % kRing], (ps / kRing) & 1, P.timeout_flag, dead);
                            if (!dead) issue_stage(ps + kRing);      // after a wait has run out nothing more is copied
                        }
                    }
                    float e[VPT][EPT];
#pragma unroll
                    for (int v = 0; v < VPT; ++v) {
                        if (has[v]) {
                            float xa[EPV], xb[EPV];
                            unpack_vec<DT>(va[v], xa);
                            unpack_vec<DT>(vb[v], xb);
#pragma unroll
                            for (int j = 0; j < EPV; j += 2) {
                                float a0 = xa[j], a1 = xa[j + 1], b0 = xb[j], b1 = xb[j + 1];
                                if constexpr (DT == FSD_F32) {
                                    a0 = fmaxf(a0, kClamp); a1 = fmaxf(a1, kClamp);
                                    if constexpr (DIV != FSD_DIV_KL) { b0 = fmaxf(b0, kClamp); b1 = fmaxf(b1, kClamp); }
                                }
                                const uint64_t ya2 = fma2(pack2(a0, a1), l2, ca2), yb2 = fma2(pack2(b0, b1), l2, cb2);
                                float ya0, ya1, yb0, yb1;
                                unpack2(ya2, ya0, ya1);
                                unpack2(yb2, yb0, yb1);
                                const float ea0 = ex2(ya0), ea1 = ex2(ya1), eb0 = ex2(yb0), eb1 = ex2(yb1);
                                const uint64_t ea2 = pack2(ea0, ea1), eb2 = pack2(eb0, eb1);
                                za2 = add2(za2, ea2);
                                zb2 = add2(zb2, eb2);
                                if constexpr (DIV == FSD_DIV_JS) {
                                    sa2 = fma2(ea2, ya2, sa2);
                                    sb2 = fma2(eb2, yb2, sb2);
                                }
                                if constexpr (DIV == FSD_DIV_KL) {
                                    if (ea0 > 0.f) kk = fmaf(ea0, ya0 - yb0, kk);
                                    if (ea1 > 0.f) kk = fmaf(ea1, ya1 - yb1, kk);
                                }
                                e[v][j] = ea0; e[v][j + 1] = ea1;
                                e[v][EPV + j] = eb0; e[v][EPV + j + 1] = eb1;
                            }
                        } else {
#pragma unroll
                            for (int j = 0; j < EPT; ++j) e[v][j] = 0.f;
                        }
                    }
                    if constexpr (kSecondSweep) {
#pragma unroll
                        for (int v = 0; v < VPT; ++v) {
                            if (s < NT) {
                                FSD_CHECK(P.timeout_flag + 2, (s * VPT + v) * EPT + EPT <= kTmemPerThread, kChkTmem);
                                tmem_st<EPT>(taddr + (s * VPT + v) * EPT, e[v]);
                            } else {
#pragma unroll
                                for (int j = 0; j < EPT; ++j) ereg[(s - NT < 0 ? 0 : s - NT) * EPS + v * EPT + j] = e[v][j];
                            }
                        }
                    }
                }
            }
            if constexpr (kSecondSweep) tmem_wait_st();

            // thread -> warp: bring the sums to the warp's reference (exact power-of-two factors)
            const float za = sum2(za2), zb = sum2(zb2);
            const float wka = warp_max_nan(ka), wkb = warp_max_nan(kb);
            const float da = ka == -INFINITY ? 0.f : ka - wka, db = kb == -INFINITY ? 0.f : kb - wkb;
            const float fa = ka == -INFINITY ? 0.f : pow2_int(da), fb = kb == -INFINITY ? 0.f : pow2_int(db);
            float v_za = za * fa, v_zb = zb * fb;
            float v_s0 = 0.f, v_sb = 0.f;
            if constexpr (DIV == FSD_DIV_JS) { v_s0 = fa * fmaf(da, za, sum2(sa2)); v_sb = fb * fmaf(db, zb, sum2(sb2)); }
            if constexpr (DIV == FSD_DIV_KL) v_s0 = scale_kl(fa, fmaf(da - db, za, kk));
#pragma unroll
            for (int m = 16; m > 0; m >>= 1) {
                v_za += __shfl_xor_sync(0xffffffffu, v_za, m);
                v_zb += __shfl_xor_sync(0xffffffffu, v_zb, m);
                if constexpr (DIV != FSD_DIV_TV) v_s0 += __shfl_xor_sync(0xffffffffu, v_s0, m);
                if constexpr (DIV == FSD_DIV_JS) v_sb += __shfl_xor_sync(0xffffffffu, v_sb, m);
            }
            mine.ka = wka; mine.kb = wkb; mine.za = v_za; mine.zb = v_zb; mine.s0 = v_s0; mine.sb = v_sb;
            mine.diff = __reduce_or_sync(0xffffffffu, diff);
        }
        mine.x = x_carry;

        // ---- exchange.  Every warp leaves its statistics in shared memory and counts itself in
        //      on a named barrier; this round's combiner warp waits there for the others, folds
        //      the warps' statistics, stores the virtual CTA's message, fetches the group's messages
        //      until all carry this round's tag, folds those and leaves the totals for the virtual
        //      CTA.  Only the combiner polls; everyone else sleeps on a barrier. ----
        if (lane == 0) sh.ws[warp] = mine;
        __syncwarp();
        if (warp != static_cast<int>(li & (kStreamWarps - 1))) {
            __threadfence_block();
            named_arrive(bar_posted);
        } else {
            named_sync(bar_posted);
            Stats w;
            w.ka = -INFINITY; w.kb = -INFINITY; w.za = 0.f; w.zb = 0.f; w.s0 = 0.f; w.sb = 0.f; w.x = 0.f; w.diff = 0;
            if (lane < kStreamWarps) w = sh.ws[lane];
            Stats c;
            c.ka = warp_max_nan(w.ka); c.kb = warp_max_nan(w.kb);
            {
                const float da = w.ka == -INFINITY ? 0.f : w.ka - c.ka, db = w.kb == -INFINITY ? 0.f : w.kb - c.kb;
                const float fa = w.ka == -INFINITY ? 0.f : pow2_int(da), fb = w.kb == -INFINITY ? 0.f : pow2_int(db);
                c.za = w.za * fa; c.zb = w.zb * fb;
                c.s0 = DIV == FSD_DIV_KL ? scale_kl(fa, fmaf(da - db, w.za, w.s0)) : fa * fmaf(da, w.za, w.s0);
                c.sb = fb * fmaf(db, w.zb, w.sb);
                c.x = w.x;
            }
#pragma unroll
            for (int m = 8; m > 0; m >>= 1) {
                c.za += __shfl_xor_sync(0xffffffffu, c.za, m); c.zb += __shfl_xor_sync(0xffffffffu, c.zb, m);
                c.s0 += __shfl_xor_sync(0xffffffffu, c.s0, m); c.sb += __shfl_xor_sync(0xffffffffu, c.sb, m);
                c.x += __shfl_xor_sync(0xffffffffu, c.x, m);
            }
            c.diff = __reduce_or_sync(0xffffffffu, w.diff) != 0 ? 1u : 0u;
            if constexpr (!kSecondSweep) {
                // KL has no second sweep, so nobody needs the group's totals: every member leaves its part
                // straight in the pair's record and goes on.  Without messages there is no channel for
                // claimed pair ids either: the group's pairs are group_id + round * n_groups throughout.
                if (live && lane == 0) {
                    FSD_CHECK(P.timeout_flag + 2, item >= 0 && item < P.n_items && rank < kMaxGroupSize, kChkRecord);
                    PairRecord* r = P.records + item;
                    r->part[rank] = c;
                    if (rank == 0) { r->ncta = static_cast<uint32_t>(C); r->state = bad ? kRecordBadTree : kRecordStats; }
                }
                const long long id = static_cast<long long>(group_id) + static_cast<long long>(li + ahead) * n_groups;
                const bool stop = __any_sync(0xffffffffu, dead);
                if (lane == 0) {
                    sh.items[(li + ahead) & 7] = (stop || id >= 0x3fffffffLL) ? 0x3fffffff : static_cast<int>(id);
                    *reinterpret_cast<float4*>(sh.tot) = make_float4(0.f, 0.f, 0.f, 0.f);
                }
                named_sync(bar_totals);
            } else {
            {
                const uint32_t cl = __shfl_sync(0xffffffffu, claimed, 0);   // rank 0's message carries the pair id it took
                if (rank == 0) c.diff |= cl << 1;
            }
            // lanes 0..2 each store one 16-byte unit of this virtual CTA's message; every unit ends in the round's tag
            if (lane < 3 && !(li == 0 && group_id == 0 && rank == P.silent_rank)) {
                const float m0 = lane == 0 ? c.ka : lane == 1 ? c.zb : c.x;
                const float m1 = lane == 0 ? c.kb : lane == 1 ? c.s0 : __uint_as_float(c.diff);
                const float m2 = lane == 0 ? c.za : lane == 1 ? c.sb : 0.f;
                st_unit(&xg[par * C + rank].u[lane], m0, m1, m2, tag);
            }
            // group totals for the second sweep (float is enough there); lane r fetches virtual CTA r's message
            Stats t;
            t.ka = -INFINITY; t.kb = -INFINITY; t.za = 0.f; t.zb = 0.f; t.s0 = 0.f; t.sb = 0.f; t.x = 0.f; t.diff = 0;
            if (!__any_sync(0xffffffffu, dead)) {          // (a lane's own earlier wait may have run out: decide as a warp)
                bool got = false;
#pragma unroll 1
                for (uint32_t i = 0; i < P.poll_limit; ++i) {
                    // with the first fetch and every 256th: has anybody's wait run out?  (then nothing
                    // this warp waits for is certain to come, and the group takes no further pair)
                    const bool look = (i & 255u) == 0;
                    int gave_up = 0;
                    if (look && lane == 0) gave_up = *reinterpret_cast<volatile int*>(P.timeout_flag);
                    bool ok = true;
                    if (lane < C) {
                        const uint4 u0 = ld_unit(&xg[par * C + lane].u[0]), u1 = ld_unit(&xg[par * C + lane].u[1]),
                                    u2 = ld_unit(&xg[par * C + lane].u[2]);
                        ok = u0.w == tag && u1.w == tag && u2.w == tag;
                        t.ka = __uint_as_float(u0.x); t.kb = __uint_as_float(u0.y); t.za = __uint_as_float(u0.z);
                        t.zb = __uint_as_float(u1.x); t.s0 = __uint_as_float(u1.y); t.sb = __uint_as_float(u1.z);
                        t.x = __uint_as_float(u2.x); t.diff = u2.y;
                    }
                    const bool all_ok = __all_sync(0xffffffffu, ok);
                    if (look && __shfl_sync(0xffffffffu, gave_up, 0) != 0) break;
                    if (all_ok) { got = true; break; }
                }
                if (!got) {
                    if (lane == 0) atomicExch(P.timeout_flag, 1);
                    dead = true;
                    t.ka = __int_as_float(0x7fc00000);   // the totals of a round that never completed are invalid
                }
            }
            {
                // after a wait that ran out this group takes no further pair: every member reads the same
                // "none" and leaves together once the pairs already in its ring are through
                const uint32_t sent = __shfl_sync(0xffffffffu, t.diff, 0) >> 1;
                const bool stop = __any_sync(0xffffffffu, dead);
                const uint32_t nxt = stop ? 0x3fffffffu : sent;
                t.diff &= 1u;
                if (lane == 0) sh.items[(li + ahead) & 7] = static_cast<int>(nxt);
            }
            const float Ka = warp_max_nan(t.ka), Kb = warp_max_nan(t.kb);
            float tza = t.ka == -INFINITY ? 0.f : t.za * pow2_int(t.ka - Ka);
            float tzb = t.kb == -INFINITY ? 0.f : t.zb * pow2_int(t.kb - Kb);
#pragma unroll
            for (int m = 8; m > 0; m >>= 1) {
                tza += __shfl_xor_sync(0xffffffffu, tza, m); tzb += __shfl_xor_sync(0xffffffffu, tzb, m);
            }
            if (lane == 0) *reinterpret_cast<float4*>(sh.tot) = make_float4(Ka, Kb, tza, tzb);
            named_sync(bar_totals);
            // rank 0 hands the parts to the finish kernel, which folds them in double; the
            // previous pair gets its second-sweep sums
            if (rank == 0 && lane < C) {
                if (prev_item >= 0) P.records[prev_item].x[lane] = t.x;
                if (live) {
                    FSD_CHECK(P.timeout_flag + 2, item >= 0 && item < P.n_items && C <= kMaxGroupSize, kChkRecord);
                    PairRecord* r = P.records + item;
                    r->part[lane] = t;
                    if (lane == 0) { r->ncta = static_cast<uint32_t>(C); r->state = bad ? kRecordBadTree : kRecordStats; }
                }
            }
            }   // (the exchange that JS and TV need)
        }
        if (warp != static_cast<int>(li & (kStreamWarps - 1))) named_sync(bar_totals);
        const float4 tot = *reinterpret_cast<const float4*>(sh.tot);
        const float Ka = tot.x, Kb = tot.y, tZa = tot.z, tZb = tot.w;
        prev_item = -1;
        x_carry = 0.f;
        if (!live) break;
        prev_item = kSecondSweep ? item : -1;        // (no second-sweep sum to publish a round later)

        // ---- second sweep over the parked e values ----
        if (kSecondSweep) {
            const bool ok = tZa > 0.f && tZb > 0.f && tZa < 3.0e38f && tZb < 3.0e38f;   // false for NaN too
            const float iza = ok ? 1.0f / tZa : 0.f, izb = ok ? 1.0f / tZb : 0.f;
            const float ia = (ka == -INFINITY || !ok) ? 0.f : pow2_int(ka - Ka) * iza;
            const float ib = (kb == -INFINITY || !ok) ? 0.f : pow2_int(kb - Kb) * izb;
            uint64_t x2 = 0;
            float xt = 0.f;
            // s = p + q + 1e-37 keeps lg2 finite where both terms vanish; the shift is below one ulp of any s that matters
            const uint64_t ia2 = pack2(ia, ia), ib2 = pack2(ib, ib), tiny2 = pack2(1e-37f, 1e-37f);
#pragma unroll
            for (int s = 0; s < kMaxStagesPerPair; ++s) {
                if (s < ns) {
                    float e[VPT][EPT];
                    if (s < NT) {
#pragma unroll
                        for (int v = 0; v < VPT; ++v) tmem_ld<EPT>(taddr + (s * VPT + v) * EPT, e[v]);
                        tmem_wait_ld();
                    } else {
#pragma unroll
                        for (int v = 0; v < VPT; ++v) {
#pragma unroll
                            for (int j = 0; j < EPT; ++j) e[v][j] = ereg[(s - NT < 0 ? 0 : s - NT) * EPS + v * EPT + j];
                        }
                    }
#pragma unroll
                    for (int v = 0; v < VPT; ++v) {
#pragma unroll
                        for (int j = 0; j < EPV; j += 2) {
                            const uint64_t ea2 = pack2(e[v][j], e[v][j + 1]), eb2 = pack2(e[v][EPV + j], e[v][EPV + j + 1]);
                            if constexpr (DIV == FSD_DIV_JS) {
                                const uint64_t s2 = fma2(eb2, ib2, fma2(ea2, ia2, tiny2));
                                float s0, s1;
                                unpack2(s2, s0, s1);
                                x2 = fma2(s2, pack2(lg2(s0), lg2(s1)), x2);
                            } else {
                                // separately rounded products: a fused p - q would make TV(p, p) != 0
                                const uint64_t d2 = fma2(mul2(eb2, ib2), pack2(-1.f, -1.f), mul2(ea2, ia2));
                                float d0, d1;
                                unpack2(d2, d0, d1);
                                xt += fabsf(d0) + fabsf(d1);
                            }
                        }
                    }
                }
            }
            float x = sum2(x2) + xt;
#pragma unroll
            for (int m = 16; m > 0; m >>= 1) x += __shfl_xor_sync(0xffffffffu, x, m);
            x_carry = x;
        }

        // ---- next pair ----
        g += ns;
        ++li;
        item = sh.items[li & 7];
    }

    // ---- release tensor memory ----
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (tid == 0) {
        // Every copy started into this virtual CTA's ring has landed before the CTA may leave: normally the
        // first sweep consumed them all and these waits return at once; after a wait that ran out
        // some may still be on their way (a copy, once started, always completes).
        for (int slot = 0; slot < kRing; ++slot) {
            const uint32_t n = sh.armed[slot];
            if (n == 0) continue;
#pragma unroll 1
            for (uint32_t i = 0; i < kSpinLimit; ++i)
                if (mbar_try_wait(&sh.full[slot], (n - 1) & 1)) break;
        }
    }
    __syncthreads();
    if (threadIdx.x < 32) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(*tmem_base_slot), "r"(kStreamHalves * kTmemCols) : "memory");
    }
}

}  // namespace fsd
