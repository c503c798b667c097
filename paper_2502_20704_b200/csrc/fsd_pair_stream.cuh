// Streaming per-(row, position) kernel: every logit is read from HBM once.
//
// A (row, position) pair is split along the vocabulary over a thread-block cluster of C CTAs
// (C = 1, 2, 4 or 8, the smallest that lets a CTA's slice fit on chip).  Clusters are
// persistent and walk the pair list round-robin.  Per pair, each CTA
//   1. receives its slice of both rows in shared memory through a ring of bulk asynchronous
//      copies (cp.async.bulk + mbarrier; the next pair's slices stream in meanwhile),
//   2. sweeps the slice once from shared memory for each thread's exact maximum and a
//      bitwise "rows differ" flag,
//   3. sweeps it again computing e = 2^(log2e * (logit - thread max)) with one MUFU ex2 per
//      logit, the sums Z = sum e and S = sum e*y (and the KL sum), and parks the e values in
//      tensor memory (64 per thread) and registers (16 per thread),
//   4. combines (max, Z, S) over threads, warps, CTA and -- through distributed shared memory
//      and one cluster barrier -- the cluster,
//   5. sweeps the parked e values: p = e_a/Z_a, q = e_b/Z_b, JS needs sum (p+q) log2(p+q) (one
//      MUFU lg2 per pair), TV needs sum |p - q|; KL needs no second sweep.
// The logits themselves are never touched again after step 3, so HBM traffic is the
// algorithmic minimum; the special-function pipe (1 ex2 per logit + 1 lg2 per pair) is the
// co-bottleneck, which is why e values are kept rather than recomputed.
// Two CTAs share an SM so that one CTA's reduction / barrier bubbles are filled by the other.
#pragma once

#include "fsd_device.cuh"
#include "fsd_pair_generic.cuh"

namespace fsd {

constexpr int kStreamThreads = 512;
constexpr int kStreamWarps = kStreamThreads / 32;
constexpr int kRing = 6;                                   // stages in the shared-memory ring
constexpr int kStageRowBytes = kStreamThreads * 16;        // one 16-byte vector per thread and row
constexpr int kStageBytes = 2 * kStageRowBytes;
constexpr int kMaxStagesPerPair = kRing - 1;               // a pair's slice must be resident at once
constexpr int kTmemCols = 256;                             // per CTA: 16 warps -> 4 per lane quarter x 64 columns
constexpr int kTmemPerThread = 64;
constexpr int kMaxVecPerCta = kMaxStagesPerPair * kStreamThreads;
constexpr uint32_t kSpinLimit = 1u << 24;                  // polls before a wait gives up

struct StreamParams {
    PairParams pp;
    int nvec_row;              // 16-byte vectors per logit row
    int n_items;               // B * G
    int* timeout_flag;         // set to 1 if a bounded wait ran out (host reports FSD_ROW_TIMEOUT)
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
    for (uint32_t i = 0; i < kSpinLimit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
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
__device__ __forceinline__ uint32_t bf16x2_max(uint32_t a, uint32_t b) {
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

// ---- shared-memory layout ---------------------------------------------------------------
struct WarpStats {             // one per warp, written by lane 0 after the exponential sweep
    float ra, rb;              // warp reference (maximum logit) of each row
    float za, zb, sa, sb, kk;  // sums relative to the warp reference
    uint32_t diff;
};
struct CtaStats {              // one per CTA and parity, read by the whole cluster
    float ra, rb;
    double za, zb, sa, sb, kk;
    double x_prev;             // second-sweep sum of the PREVIOUS pair
    uint32_t diff;
};
struct Pending {               // what rank 0 needs to finish a pair once its second-sweep sum arrives
    int item;                  // -1 = nothing pending
    int finite, differ;
    float Ma, Mb;              // row maxima
    double Za, Zb, Sa, Sb, K;  // totals relative to the maxima
};
struct StreamShared {
    uint64_t full[kRing];
    uint64_t empty[kRing];
    uint32_t tmem_base;
    float bc_Ma, bc_Mb, bc_iZa, bc_iZb;    // broadcast of the pair's maxima and reciprocal normalisers
    WarpStats ws[kStreamWarps];
    float wx[kStreamWarps];                // per-warp second-sweep sums
    CtaStats xch[2];
    Pending pend;                          // written by warp 0, consumed by the last warp (rank 0 only)
};
constexpr size_t kStreamSmemBytes = kRing * kStageBytes + sizeof(StreamShared) + 128;

// ---- final scalar work of one pair (rank 0, one thread) --------------------------------
__device__ inline void finish_pair(const StreamParams& P, const Pending& pd, double X, int dt) {
    const PairParams& pp = P.pp;
    const int item = pd.item;
    float D = __int_as_float(0x7fc00000);
    if (pd.finite) {
        D = pd.differ ? static_cast<float>(combine_divergence(pp.div, pd.Za, pd.Zb, pd.Sa, pd.Sb, pd.K, X)) : 0.0f;
    }
    pp.divergence[item] = D;
    const int b = item / pp.G, i = item - b * pp.G;
    int trow = i;
    if (pp.parent != nullptr) trow = pp.parent[item] + 1;
    const size_t rb = static_cast<size_t>(pp.V) * (dt == FSD_BF16 ? 2 : 4);
    const char* a_row = static_cast<const char*>(pp.target) + (static_cast<size_t>(b) * (pp.G + 1) + trow) * rb;
    const char* b_row = static_cast<const char*>(pp.draft) + (static_cast<size_t>(b) * pp.G + i) * rb;
    // the sums are relative to the exact maxima, so the offsets used are exactly -M*log2e in double
    const float ca = -pd.Ma * kLog2e, cb = -pd.Mb * kLog2e;
    double Za = pd.Za, Zb = pd.Zb;
    if (pd.finite) {
        // log_prob() expects Z accumulated with the float offsets ca / cb; ours used exact references
        Za *= exp2(static_cast<double>(ca) + static_cast<double>(pd.Ma) * kLog2eD);
        Zb *= exp2(static_cast<double>(cb) + static_cast<double>(pd.Mb) * kLog2eD);
    }
    pp.item_bits[item] = accept_bit(pp, item, pd.finite != 0, D, a_row, b_row, dt, pd.Ma, ca, Za, pd.Mb, cb, Zb);
    pp.item_status[item] = pd.finite ? 0 : FSD_ROW_NONFINITE;
}

template <int DT, int DIV>
__global__ void __launch_bounds__(kStreamThreads, 2) fsd_pair_stream_kernel(StreamParams P) {
    constexpr int EPV = Logit<DT>::kPerVec;          // logits per 16-byte vector
    constexpr int EPT = 2 * EPV;                     // e values per thread and stage (both rows)
    constexpr int NT = (kTmemPerThread / EPT) < kMaxStagesPerPair ? (kTmemPerThread / EPT) : kMaxStagesPerPair;
    constexpr int NR = kMaxStagesPerPair - NT;       // stages kept in registers
    constexpr bool kSecondSweep = DIV != FSD_DIV_KL;
    constexpr float kYMin = -150.f;                  // ex2 flushes to zero below -126

    extern __shared__ unsigned char smem_raw[];
    unsigned char* ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    StreamShared& sh = *reinterpret_cast<StreamShared*>(ring + kRing * kStageBytes);

    cg::cluster_group cluster = cg::this_cluster();
    const int C = static_cast<int>(cluster.num_blocks());
    const int rank = static_cast<int>(cluster.block_rank());
    const int cluster_id = blockIdx.x / C, n_clusters = gridDim.x / C;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const PairParams& pp = P.pp;

    // this CTA's slice of every row, in vectors
    const int base = P.nvec_row / C, rem = P.nvec_row % C;
    const int vbeg = rank * base + (rank < rem ? rank : rem);
    const int vcnt = base + (rank < rem ? 1 : 0);
    const int ns = (vcnt + kStreamThreads - 1) / kStreamThreads;     // stages per pair (<= kMaxStagesPerPair)
    const size_t row_bytes = static_cast<size_t>(P.nvec_row) * 16;

    // ---- set-up: barriers, tensor memory ----
    if (blockIdx.x == 0 && tid == 0) *P.timeout_flag = 0;   // a wait needs far longer to run out than this store takes
    if (tid == 0) {
        for (int s = 0; s < kRing; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], kStreamWarps); }
        sh.pend.item = -1;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&sh.tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    // warp w owns tensor-memory lanes 32*(w%4)..+31 and columns 64*(w/4)..+63
    const uint32_t taddr = sh.tmem_base + (static_cast<uint32_t>(32 * (warp & 3)) << 16) + static_cast<uint32_t>(64 * (warp >> 2));

    bool dead = false;                               // a bounded wait of this thread ran out
    // ---- producer state (thread 0 only) ----
    int p_item = cluster_id, p_stage = 0;
    uint32_t p_g = 0;                                // stages issued so far
    auto item_rows = [&](int item, const char*& a_row, const char*& b_row) -> bool {
        const int b = item / pp.G, i = item - b * pp.G;
        int trow = i;
        if (pp.parent != nullptr) {
            const int par = __ldg(pp.parent + item);
            if (par < -1 || par >= i) return false;
            trow = par + 1;
        }
        a_row = static_cast<const char*>(pp.target) + (static_cast<size_t>(b) * (pp.G + 1) + trow) * row_bytes;
        b_row = static_cast<const char*>(pp.draft) + (static_cast<size_t>(b) * pp.G + i) * row_bytes;
        return true;
    };
    // issues the next stage if its ring slot is free (or, when `block`, waits for it); false if nothing was issued
    auto produce = [&](bool block) -> bool {
        while (p_item < P.n_items) {
            const char *a_row, *b_row;
            if (p_stage == 0 && !item_rows(p_item, a_row, b_row)) { p_item += n_clusters; continue; }   // bad tree node: no data
            break;
        }
        if (p_item >= P.n_items) return false;
        const uint32_t slot = p_g % kRing;
        if (p_g >= kRing) {
            const uint32_t parity = ((p_g / kRing) - 1) & 1;
            if (block) mbar_wait(&sh.empty[slot], parity, P.timeout_flag, dead);
            else if (!mbar_try_wait(&sh.empty[slot], parity)) return false;
        }
        const char *a_row, *b_row;
        item_rows(p_item, a_row, b_row);
        const int v0 = p_stage * kStreamThreads;
        const int nv = (vcnt - v0) < kStreamThreads ? (vcnt - v0) : kStreamThreads;
        const uint32_t bytes = static_cast<uint32_t>(nv) * 16;
        unsigned char* dst = ring + slot * kStageBytes;
        mbar_arrive_expect_tx(&sh.full[slot], 2 * bytes);
        bulk_g2s(dst, a_row + (static_cast<size_t>(vbeg) + v0) * 16, bytes, &sh.full[slot]);
        bulk_g2s(dst + kStageRowBytes, b_row + (static_cast<size_t>(vbeg) + v0) * 16, bytes, &sh.full[slot]);
        ++p_g;
        if (++p_stage == ns) { p_stage = 0; p_item += n_clusters; }
        return true;
    };
    if (tid == 0) { while (p_g < kRing && produce(false)) {} }

    float ereg[(NR > 0 ? NR : 1) * EPT];
    uint32_t g = 0;                                  // stages consumed so far
    int parity = 0;                                  // exchange slot parity
    float x_carry = 0.f;                             // this thread's share of the previous pair's second-sweep sum (warp-reduced, lane 0)
    bool have_prev = false;

    for (int item = cluster_id;; item += n_clusters) {
        const bool live = item < P.n_items;          // one extra round flushes the last pair's second sweep
        if (!live && !have_prev) break;
        bool bad = false;
        if (live && pp.parent != nullptr) {
            const int i = item % pp.G;
            const int par = __ldg(pp.parent + item);
            bad = par < -1 || par >= i;
        }
        const bool work = live && !bad;

        float ra = -INFINITY, rb = -INFINITY, za = 0.f, zb = 0.f, sa = 0.f, sb = 0.f, kk = 0.f;
        uint32_t diff = 0;
        if (work) {
            // ---- sweep A: exact thread maxima and the bitwise difference flag, from shared memory ----
            if (tid == 0) { while (p_g < g + ns && produce(true)) {} }
            __syncwarp();
#pragma unroll
            for (int s = 0; s < kMaxStagesPerPair; ++s) {
                if (s < ns) {
                    const uint32_t gs = g + s, slot = gs % kRing;
                    mbar_wait(&sh.full[slot], (gs / kRing) & 1, P.timeout_flag, dead);
                    if (s * kStreamThreads + tid < vcnt) {
                        const unsigned char* st = ring + slot * kStageBytes + tid * 16;
                        const uint4 va = *reinterpret_cast<const uint4*>(st);
                        const uint4 vb = *reinterpret_cast<const uint4*>(st + kStageRowBytes);
                        diff |= (va.x ^ vb.x) | (va.y ^ vb.y) | (va.z ^ vb.z) | (va.w ^ vb.w);
                        if constexpr (DT == FSD_BF16) {
                            const uint32_t ma = bf16x2_max(bf16x2_max(va.x, va.y), bf16x2_max(va.z, va.w));
                            const uint32_t mb = bf16x2_max(bf16x2_max(vb.x, vb.y), bf16x2_max(vb.z, vb.w));
                            ra = fmax_nan(ra, fmax_nan(bf16_lo(ma), bf16_hi(ma)));
                            rb = fmax_nan(rb, fmax_nan(bf16_lo(mb), bf16_hi(mb)));
                        } else {
                            ra = fmax_nan(ra, fmax_nan(fmax_nan(__uint_as_float(va.x), __uint_as_float(va.y)),
                                                       fmax_nan(__uint_as_float(va.z), __uint_as_float(va.w))));
                            rb = fmax_nan(rb, fmax_nan(fmax_nan(__uint_as_float(vb.x), __uint_as_float(vb.y)),
                                                       fmax_nan(__uint_as_float(vb.z), __uint_as_float(vb.w))));
                        }
                    }
                }
            }
            // ---- sweep B: exponentials, sums, park the e values ----
            const float ca = ra == -INFINITY ? 0.f : -ra * kLog2e;
            const float cb = rb == -INFINITY ? 0.f : -rb * kLog2e;
#pragma unroll
            for (int s = 0; s < kMaxStagesPerPair; ++s) {
                if (s < ns) {
                    const uint32_t gs = g + s, slot = gs % kRing;
                    float e[EPT];
                    if (s * kStreamThreads + tid < vcnt) {
                        const unsigned char* st = ring + slot * kStageBytes + tid * 16;
                        float xa[EPV], xb[EPV];
                        unpack_vec<DT>(*reinterpret_cast<const uint4*>(st), xa);
                        unpack_vec<DT>(*reinterpret_cast<const uint4*>(st + kStageRowBytes), xb);
#pragma unroll
                        for (int j = 0; j < EPV; ++j) {
                            const float ya_raw = fmaf(xa[j], kLog2e, ca), yb_raw = fmaf(xb[j], kLog2e, cb);
                            const float ya = fmaxf(ya_raw, kYMin), yb = fmaxf(yb_raw, kYMin);
                            const float ea = ex2(ya), eb = ex2(yb);
                            za += ea;
                            zb += eb;
                            if constexpr (DIV == FSD_DIV_JS) {
                                sa = fmaf(ea, ya, sa);
                                sb = fmaf(eb, yb, sb);
                            }
                            if constexpr (DIV == FSD_DIV_KL) {
                                // q = 0 < p must give +inf: the draft exponent is used unclamped
                                if (ea > 0.f) kk = fmaf(ea, ya - yb_raw, kk);
                            }
                            e[j] = ea;
                            e[EPV + j] = eb;
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < EPT; ++j) e[j] = 0.f;
                    }
                    if constexpr (kSecondSweep) {
                        if (s < NT) {
                            tmem_st<EPT>(taddr + s * EPT, e);
                        } else {
#pragma unroll
                            for (int j = 0; j < EPT; ++j) ereg[(s - NT < 0 ? 0 : s - NT) * EPT + j] = e[j];
                        }
                    }
                    // this warp is done with the slot
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sh.empty[slot]);
                    if (tid == 0) produce(false);
                    __syncwarp();
                }
            }
            g += ns;
            if constexpr (kSecondSweep) tmem_wait_st();

            // ---- thread -> warp: bring the sums to the warp's reference ----
            const float wa = warp_max_nan(ra), wb = warp_max_nan(rb);
            const float da = ra == -INFINITY ? 0.f : (ra - wa) * kLog2e, db = rb == -INFINITY ? 0.f : (rb - wb) * kLog2e;
            const float fa = ra == -INFINITY ? 0.f : ex2(da), fb = rb == -INFINITY ? 0.f : ex2(db);
            float v_za = za * fa, v_zb = zb * fb;
            float v_sa = fa * fmaf(da, za, sa), v_sb = fb * fmaf(db, zb, sb);
            float v_kk = fa * fmaf(da - db, za, kk);
#pragma unroll
            for (int m = 16; m > 0; m >>= 1) {
                v_za += __shfl_xor_sync(0xffffffffu, v_za, m);
                v_zb += __shfl_xor_sync(0xffffffffu, v_zb, m);
                if constexpr (DIV == FSD_DIV_JS) {
                    v_sa += __shfl_xor_sync(0xffffffffu, v_sa, m);
                    v_sb += __shfl_xor_sync(0xffffffffu, v_sb, m);
                }
                if constexpr (DIV == FSD_DIV_KL) v_kk += __shfl_xor_sync(0xffffffffu, v_kk, m);
            }
            const uint32_t wdiff = __reduce_or_sync(0xffffffffu, diff);
            if (lane == 0) {
                WarpStats& w = sh.ws[warp];
                w.ra = wa; w.rb = wb; w.za = v_za; w.zb = v_zb; w.sa = v_sa; w.sb = v_sb; w.kk = v_kk; w.diff = wdiff;
            }
        }
        if (lane == 0) sh.wx[warp] = x_carry;         // previous pair's second-sweep sum of this warp
        __syncthreads();                               // (A) warp statistics visible

        // ---- warp 0: CTA totals, publish to the cluster ----
        if (warp == 0) {
            double Za = 0, Zb = 0, Sa = 0, Sb = 0, K = 0, X = 0;
            float Ra = -INFINITY, Rb = -INFINITY;
            uint32_t df = 0;
            if (lane < kStreamWarps) {
                X = static_cast<double>(sh.wx[lane]);
                if (work) {
                    const WarpStats w = sh.ws[lane];
                    Ra = w.ra; Rb = w.rb; df = w.diff;
                    Za = w.za; Zb = w.zb; Sa = w.sa; Sb = w.sb; K = w.kk;
                }
            }
            const float cRa = warp_max_nan(Ra), cRb = warp_max_nan(Rb);
            // rescale each warp's sums to the CTA reference (double; -inf references carry zero sums)
            const double da = (Ra == -INFINITY) ? 0.0 : (static_cast<double>(Ra) - cRa) * kLog2eD;
            const double db = (Rb == -INFINITY) ? 0.0 : (static_cast<double>(Rb) - cRb) * kLog2eD;
            const double fa = (Ra == -INFINITY) ? 0.0 : exp2(da), fb = (Rb == -INFINITY) ? 0.0 : exp2(db);
            K = fa * (K + (da - db) * Za);
            Sa = fa * (Sa + da * Za); Sb = fb * (Sb + db * Zb);
            Za *= fa; Zb *= fb;
            Za = warp_sum(Za); Zb = warp_sum(Zb); Sa = warp_sum(Sa); Sb = warp_sum(Sb); K = warp_sum(K); X = warp_sum(X);
            df = __reduce_or_sync(0xffffffffu, df);
            if (lane == 0) {
                CtaStats& c = sh.xch[parity];
                c.ra = cRa; c.rb = cRb; c.za = Za; c.zb = Zb; c.sa = Sa; c.sb = Sb; c.kk = K; c.x_prev = X; c.diff = df;
            }
        }
        cluster.sync();                                // every CTA's statistics visible cluster-wide

        // ---- warp 0: cluster totals; broadcast what the second sweep needs; queue the finish ----
        if (warp == 0) {
            double Za = 0, Zb = 0, Sa = 0, Sb = 0, K = 0, X = 0;
            float Ra = -INFINITY, Rb = -INFINITY;
            uint32_t df = 0;
            if (lane < C) {
                const CtaStats* c = &cluster.map_shared_rank(&sh, lane)->xch[parity];
                Ra = c->ra; Rb = c->rb; Za = c->za; Zb = c->zb; Sa = c->sa; Sb = c->sb; K = c->kk; X = c->x_prev; df = c->diff;
            }
            const float Ma = warp_max_nan(Ra), Mb = warp_max_nan(Rb);
            const double da = (Ra == -INFINITY) ? 0.0 : (static_cast<double>(Ra) - Ma) * kLog2eD;
            const double db = (Rb == -INFINITY) ? 0.0 : (static_cast<double>(Rb) - Mb) * kLog2eD;
            const double fa = (Ra == -INFINITY) ? 0.0 : exp2(da), fb = (Rb == -INFINITY) ? 0.0 : exp2(db);
            K = fa * (K + (da - db) * Za);
            Sa = fa * (Sa + da * Za); Sb = fb * (Sb + db * Zb);
            Za *= fa; Zb *= fb;
            Za = warp_sum(Za); Zb = warp_sum(Zb); Sa = warp_sum(Sa); Sb = warp_sum(Sb); K = warp_sum(K); X = warp_sum(X);
            df = __reduce_or_sync(0xffffffffu, df);
            if (lane == 0) {
                // finish the previous pair now that its second-sweep sum is complete (rank 0 only)
                if (rank == 0 && sh.pend.item >= 0) {
                    finish_pair(P, sh.pend, X, DT);
                    sh.pend.item = -1;
                }
                if (live) {
                    const bool finite = work && isfinite(Ma) && isfinite(Mb) && isfinite(Za) && isfinite(Zb) && Za > 0.0 && Zb > 0.0;
                    sh.bc_Ma = Ma; sh.bc_Mb = Mb;
                    sh.bc_iZa = finite ? static_cast<float>(1.0 / Za) : 0.f;
                    sh.bc_iZb = finite ? static_cast<float>(1.0 / Zb) : 0.f;
                    if (rank == 0) {
                        Pending& pd = sh.pend;
                        if (bad) {
                            pp.divergence[item] = __int_as_float(0x7fc00000);
                            pp.item_bits[item] = 0;
                            pp.item_status[item] = FSD_ROW_BADTREE;
                        } else {
                            pd.item = item; pd.finite = finite; pd.differ = df != 0;
                            pd.Ma = Ma; pd.Mb = Mb; pd.Za = Za; pd.Zb = Zb; pd.Sa = Sa; pd.Sb = Sb; pd.K = K;
                        }
                    }
                }
            }
        }
        __syncthreads();                               // (B) broadcast visible
        if (tid == 0) { while (produce(false)) {} }
        __syncwarp();
        parity ^= 1;
        have_prev = false;
        x_carry = 0.f;
        if (!live) break;

        // ---- second sweep over the parked e values ----
        if (work && kSecondSweep) {
            const float Ma = sh.bc_Ma, Mb = sh.bc_Mb;
            const float ia = ra == -INFINITY ? 0.f : ex2((ra - Ma) * kLog2e) * sh.bc_iZa;
            const float ib = rb == -INFINITY ? 0.f : ex2((rb - Mb) * kLog2e) * sh.bc_iZb;
            float x = 0.f;
#pragma unroll
            for (int s = 0; s < kMaxStagesPerPair; ++s) {
                if (s < ns) {
                    float e[EPT];
                    if (s < NT) {
                        tmem_ld<EPT>(taddr + s * EPT, e);
                        tmem_wait_ld();
                    } else {
#pragma unroll
                        for (int j = 0; j < EPT; ++j) e[j] = ereg[(s - NT < 0 ? 0 : s - NT) * EPT + j];
                    }
                    if (tid == 0) produce(false);
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < EPV; ++j) {
                        if constexpr (DIV == FSD_DIV_JS) {
                            const float sm = fmaxf(fmaf(e[EPV + j], ib, e[j] * ia), 1e-37f);
                            x = fmaf(sm, lg2(sm), x);
                        } else {
                            x += fabsf(__fmul_rn(e[j], ia) - __fmul_rn(e[EPV + j], ib));
                        }
                    }
                }
            }
#pragma unroll
            for (int m = 16; m > 0; m >>= 1) x += __shfl_xor_sync(0xffffffffu, x, m);
            x_carry = x;
        }
        have_prev = true;
    }

    // ---- release tensor memory ----
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(sh.tmem_base), "r"(kTmemCols) : "memory");
    }
    cluster.sync();                                    // nobody leaves while a peer may still read its shared memory
}

}  // namespace fsd
