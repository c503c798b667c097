// Finish kernel: one thread-block cluster per batch row.
//   1. Turns the per-pair totals left by the streaming kernel into divergences and accept
//      bits (or takes the bits the generic kernel already wrote).
//   2. Finds the accepted prefix (chain) or the deepest accepted path (tree).
//   3. Draws the replacement / bonus token from one target row (and, for the SD residual, one
//      draft row) by an inverse CDF in vocabulary order.
//
// Drawing from P_T (the FSD rule, and every bonus token): each thread owns a contiguous chunk
// of the vocabulary; the weights are single-precision exponentials (one MUFU ex2 each, relative
// error at most a few 1e-7) summed in double precision, chunk sums are combined by a fixed-order
// scan (thread -> warp -> CTA -> cluster), and the warp of the first thread whose inclusive sum
// exceeds u * total re-walks that chunk with the same weights.  The cumulative sums therefore
// differ from exact ones by less than 1e-6 of the total: the token is the exact one whenever
// u * total lies further than that from both ends of its interval, and a neighbour otherwise.
// Drawing from the SD residual max(0, P_T - P_D) (Eq. 3) subtracts nearly equal numbers, so
// there the exponentials are double precision (a 256-entry table times a degree-4 polynomial,
// about ten fp64 operations) and the sums agree with a sequential double sum to rounding.
// Usually one pass over the two rows suffices for it: which entries carry residual weight
// depends on the ratio of the two normalisers only, the rejected pair's record gives that ratio
// closely enough to class every entry that is not within a margin of the boundary, and the
// chunk sums follow from the classed sums once the exact normalisers are known; entries inside
// the margin are settled one by one afterwards, and a row with too many of them in one thread
// takes a second pass.
#pragma once

#include "fsd_device.cuh"
#include "fsd_pair_generic.cuh"
#include "fsd_pair_stream.cuh"

namespace fsd {

constexpr int kFinishThreads = 512;
constexpr int kFinishWarps = kFinishThreads / 32;
constexpr int kMaxTreeNodes = 1024;

struct FinishParams {
    const void* target;        // [B, G+1, V]
    const void* draft;         // [B, G,   V]
    const int32_t* parent;     // tree only
    const int32_t* tokens;     // [B, G] or null
    const float* u_accept;     // [B, G] or null
    const float* u_sample;     // [B]
    int B, G, V;
    int div, mode, cmp, sample, max_depth;
    int vec;                   // rows are 16-byte aligned and a whole number of vectors
    float T;
    const PairRecord* records; // per-pair totals of the streaming kernel, or null (generic kernel ran)
    int32_t* item_bits;        // [B, G] read when records == null
    int32_t* item_status;      // [B, G] read when records == null
    const int* timeout_flag;   // nonzero: a bounded wait of the streaming kernel ran out (may be null)
    float* divergence;         // [B, G] written here when records != null
    int32_t* accept_len;       // [B]
    int32_t* path;             // [B, max_depth] (tree) or null
    int32_t* next_token;       // [B]
    int32_t* row_status;       // [B]
    int* debug_word;           // debug build: where failed range checks are recorded (may be null)
};

struct FinishExchange {        // what one CTA publishes to its cluster
    double d[4];
    int i[2];
};
constexpr int kExpTable = 256;

struct FinishShared {
    FinishExchange all[2][kMaxClusterSize];   // what the cluster's CTAs published, written by them (see cluster_exchange)
    double sc[kMaxClusterSize];
    double gather_d[2][kMaxClusterSize];   // one value per CTA of the cluster, written by the peers (see cluster_gather)
    int gather_i[2][kMaxClusterSize];
    float kref[kMaxTreeNodes];          // per pair: integer reference at or just above the target row's log2-sum-exp (NaN: none)
    double exp_table[kExpTable];   // 2^(j/256)
    double exp_consts[8];          // the constants of exp2_table (see exp2_consts)
    double red_d[32 * 2];
    float red_f[32 * 2];
    double warp_tot[32];
    int amb;                   // residual draw: some entry could not be classed in the first pass
    int cand;                  // lowest thread whose inclusive sum exceeds the target
    int last_pos;              // highest index with a positive weight in this CTA
    int token;
    int row_sel;               // target row the token is drawn from
    int n_acc;
    int bad;
    int best_key;              // depth * 2048 + (2047 - node) of the chosen tree node, or -1
    int16_t tree_jump[kMaxTreeNodes];
    int16_t tree_depth[kMaxTreeNodes];
    int8_t tree_ok[kMaxTreeNodes];
    int8_t tree_bit[kMaxTreeNodes];
};

// 2^y in double precision (relative error about 2e-16) for -1000 < y < 1000; 0 below, NaN for NaN.
// y = (k + r) / 256 with integer k and |r| <= 1/2: 2^y = 2^(k >> 8) * table[k & 255] * 2^(r/256),
// the last factor by a degree-4 polynomial in r (|r ln2 / 256| <= 1.4e-3, remainder < 5e-17).
__device__ __forceinline__ double exp2_table(double y, const double* table) {
    if (!(y > -1000.0)) return y != y ? y : 0.0;
    const double kMagic = 6755399441055744.0;                      // 1.5 * 2^52: the sum's low word is round(256 y)
    const double t = fma(y, 256.0, kMagic);
    const int k = __double2loint(t);
    const double r = fma(y, 256.0, kMagic - t);                    // 256 y - k, exact: |r| <= 1/2
    // coefficients (ln2 / 256)^i / i!
    double p = fma(r, 2.239395190875157e-12, 3.308302680541371e-09);
    p = fma(p, r, 3.665565596910106e-06);
    p = fma(p, r, 2.7076061740622863e-03);
    p = fma(p, r, 1.0);
    const double m = table[k & (kExpTable - 1)] * p;               // in [1, 2.0001)
    const int hi = __double2hiint(m) + ((k >> 8) << 20);           // scale by 2^(k >> 8): stays normal for |y| < 1000
    return __hiloint2double(hi, __double2loint(m));
}

// The same function, value for value above y = -990 and exactly 0 below about there, for the tight
// loops of the residual draw: no branch (callers clamp y and say when the result is to be 0; they
// have excluded NaN), and the constants
// come as arguments so that a loop keeps them in registers instead of rebuilding each 64-bit
// immediate at every use.
struct Exp2Consts { double magic, scale, c4, c3, c2, c1; };
__device__ __forceinline__ Exp2Consts exp2_consts(const double* opaque) {
    // read through shared memory: the compiler cannot turn them back into immediates
    return Exp2Consts{opaque[0], opaque[1], opaque[2], opaque[3], opaque[4], opaque[5]};
}
__device__ __forceinline__ double exp2_table_fast(double y, bool below, const double* table, const Exp2Consts& c) {
    const double t = fma(y, c.scale, c.magic);
    const int k = __double2loint(t);
    const double r = fma(y, c.scale, c.magic - t);
    double p = fma(r, c.c4, c.c3);
    p = fma(p, r, c.c2);
    p = fma(p, r, c.c1);
    p = fma(p, r, 1.0);
    const double m = table[k & (kExpTable - 1)] * p;
    const int hi = __double2hiint(m) + ((k >> 8) << 20);
    return below ? 0.0 : __hiloint2double(hi, __double2loint(m));     // a select, not a branch
}
// y = x * log2e - k for the tight loops: x is clamped in single precision at the logit below which
// y would pass -1000 (`xmin`, with a margin), and `below` tells exp2_table_fast to return exactly 0
__device__ __forceinline__ double exp2_of_logit(float x, float xmin, double nk, const double* table, const Exp2Consts& c) {
    const bool below = !(x > xmin);
    return exp2_table_fast(fma(static_cast<double>(fmaxf(x, xmin)), kLog2eD, nk), below, table, c);
}

// Every CTA of the cluster writes a FinishExchange into every CTA's shared memory (its own
// included); after one cluster barrier sh.all[buf] holds everybody's, in rank order, in every CTA.
// Like cluster_gather: `buf` alternates from one call to the next, and nobody reads a peer's
// memory afterwards.  Every thread passes the same `mine`.
__device__ __forceinline__ void cluster_exchange(cg::cluster_group& cluster, FinishShared& sh, int cs, int rank, int buf,
                                                 const FinishExchange& mine) {
    if (threadIdx.x < cs) cluster.map_shared_rank(&sh, threadIdx.x)->all[buf][rank] = mine;
    cluster.sync();
}

// Light exchange: every CTA writes one double and one int into every CTA's shared memory (its
// own included); after ONE cluster barrier sh.gather_d[buf] / gather_i[buf] hold the values of
// all CTAs, in rank order, in every CTA, and nobody reads a peer's memory (so a CTA may leave
// right afterwards).  `buf` alternates from one call to the next: a CTA that is already writing
// the next exchange cannot disturb the values a slower peer is still reading.  The peers must be
// known to have started (one cluster barrier earlier in the kernel).
__device__ __forceinline__ void cluster_gather(cg::cluster_group& cluster, FinishShared& sh, int cs, int rank, int buf, double v, int iv) {
    if (threadIdx.x < cs) {
        FinishShared* rs = cluster.map_shared_rank(&sh, threadIdx.x);
        rs->gather_d[buf][rank] = v;
        rs->gather_i[buf][rank] = iv;
    }
    cluster.sync();
}

// Divergence, accept bit and status of one pair from the streaming kernel's totals.
// A pair's totals from the parts its record holds (one per virtual CTA of the streaming group), in
// double: Z = sum 2^y, S = sum 2^y * y, K = sum 2^ya (ya - yb), all relative to the largest
// part reference (the parts' references are integers, so the factors are exact powers of two).
struct PairTotals {
    double Za, Zb, Sa, Sb, K, X;
    float ka, kb;
    uint32_t differ;
    uint32_t state;            // the record's state word
};
// 2^d for an integer-valued d <= 0, exact; 0 below the normal range
__device__ __forceinline__ double pow2_int_d(double d) {
    return d < -1022.0 ? 0.0 : __hiloint2double((1023 + static_cast<int>(d)) << 20, 0);
}
__device__ __forceinline__ double group_sum(double v) {       // over the kMaxGroupSize lanes of a record
#pragma unroll
    for (int m = kMaxGroupSize / 2; m > 0; m >>= 1) v += __shfl_xor_sync(0xffffffffu, v, m);
    return v;
}
// Called by all 32 lanes: lane 16*q + r folds part r of the record `rec` of group q (null: no
// record for this group); every lane of a group returns the group's totals.
__device__ inline PairTotals fold_record(const PairRecord* rec, int div) {
    const int r = threadIdx.x & (kMaxGroupSize - 1);
    PairTotals t;
    t.state = 0;
    Stats c;
    c.ka = -INFINITY; c.kb = -INFINITY; c.za = 0.f; c.zb = 0.f; c.s0 = 0.f; c.sb = 0.f; c.x = 0.f; c.diff = 0;
    float x = 0.f;
    if (rec != nullptr) {
        // every lane fetches its part at once with the count (one trip to L2); parts beyond the count are stale
        const Stats cr = rec->part[r];
        const float xr = rec->x[r];
        t.state = rec->state;
        if (r < static_cast<int>(rec->ncta)) { c = cr; x = xr; }
    }
    float ka = c.ka, kb = c.kb;                          // NaN references win
#pragma unroll
    for (int m = kMaxGroupSize / 2; m > 0; m >>= 1) {
        const float oa = __shfl_xor_sync(0xffffffffu, ka, m), ob = __shfl_xor_sync(0xffffffffu, kb, m);
        ka = (oa != oa || ka != ka) ? __int_as_float(0x7fc00000) : fmaxf(ka, oa);
        kb = (ob != ob || kb != kb) ? __int_as_float(0x7fc00000) : fmaxf(kb, ob);
    }
    t.ka = ka; t.kb = kb;
    const double da = c.ka == -INFINITY ? 0.0 : static_cast<double>(c.ka) - ka;
    const double db = c.kb == -INFINITY ? 0.0 : static_cast<double>(c.kb) - kb;
    const double fa = (c.ka == -INFINITY || da != da) ? 0.0 : pow2_int_d(da);
    const double fb = (c.kb == -INFINITY || db != db) ? 0.0 : pow2_int_d(db);
    t.Za = group_sum(fa * c.za); t.Zb = group_sum(fb * c.zb);
    t.Sa = 0.0; t.Sb = 0.0; t.K = 0.0;
    if (div == FSD_DIV_KL) {
        const bool inf = c.s0 == INFINITY;
        const double k = inf ? 0.0 : fa * (static_cast<double>(c.s0) + (da - db) * c.za);
        t.K = group_sum(k);
        const unsigned any_inf = __ballot_sync(0xffffffffu, inf) >> (threadIdx.x & 16) & 0xffffu;
        if (any_inf) t.K = static_cast<double>(INFINITY);
    } else {
        t.Sa = group_sum(fa * (static_cast<double>(c.s0) + da * c.za));
        t.Sb = group_sum(fb * (static_cast<double>(c.sb) + db * c.zb));
    }
    t.X = group_sum(static_cast<double>(x));
    uint32_t df = c.diff;
#pragma unroll
    for (int m = kMaxGroupSize / 2; m > 0; m >>= 1) df |= __shfl_xor_sync(0xffffffffu, df, m);
    t.differ = df;
    return t;
}

__device__ inline void judge_record(const FinishParams& P, int item, const PairTotals& r, double lnZa, double lnZb,
                                    const void* a_row, const void* b_row, int dt, float& D_out, int& bit_out, int& st_out) {
    if (r.state & kRecordBadTree) {
        D_out = __int_as_float(0x7fc00000); bit_out = 0; st_out = FSD_ROW_BADTREE;
        return;
    }
    const bool finite = isfinite(r.ka) && isfinite(r.kb) && r.Za > 0.0 && r.Zb > 0.0 && isfinite(r.Za) && isfinite(r.Zb);
    float D = __int_as_float(0x7fc00000);
    if (finite) D = r.differ ? static_cast<float>(combine_divergence(P.div, r.Za, r.Zb, lnZa, lnZb, r.Sa, r.Sb, r.K, r.X)) : 0.0f;
    const bool div_ok = finite && passes(D, P.T, P.cmp);
    int bit = div_ok;
    if (P.mode != FSD_MODE_FSD) {
        bool ratio_ok = false;
        if (finite) {
            const int x = P.tokens[item];
            if (x >= 0 && x < P.V) {
                const float ax = dt == FSD_BF16 ? load_logit<FSD_BF16>(a_row, x) : load_logit<FSD_F32>(a_row, x);
                const float bx = dt == FSD_BF16 ? load_logit<FSD_BF16>(b_row, x) : load_logit<FSD_F32>(b_row, x);
                double pacc;                                                    // Eq. 1
                if (bx == -INFINITY) {
                    pacc = (ax != -INFINITY) ? 1.0 : 0.0;
                } else {
                    // ln P(x) = (x*log2e - k) ln2 - ln Z with the same float log2e the sums were built with
                    const double la = (static_cast<double>(ax) * static_cast<double>(kLog2e) - r.ka) * kLn2D - lnZa;
                    const double lb = (static_cast<double>(bx) * static_cast<double>(kLog2e) - r.kb) * kLn2D - lnZb;
                    pacc = exp(la - lb);
                    pacc = pacc < 1.0 ? pacc : 1.0;
                }
                ratio_ok = static_cast<double>(P.u_accept[item]) < pacc;        // Eq. 2
            }
        }
        bit = P.mode == FSD_MODE_SD ? ratio_ok : (div_ok || ratio_ok);          // Eq. 6
    }
    D_out = D; bit_out = bit; st_out = finite ? 0 : FSD_ROW_NONFINITE;
}

// Calls f(k, a_k, b_k) for k in [k0, k1) in order; 16-byte loads when `vec` (then k0 is a
// multiple of the vector width and V a multiple of it).  b_k is 0 unless `with_b`.
template <int DT, typename F>
__device__ __forceinline__ void for_chunk(const void* a_row, const void* b_row, int k0, int k1, bool vec, bool with_b, F f) {
    constexpr int EPV = Logit<DT>::kPerVec;
    if (vec) {
        for (int k = k0; k < k1; k += EPV) {
            float xa[EPV], xb[EPV];
            unpack_vec<DT>(ldg_vec(a_row, k / EPV), xa);
            if (with_b) {
                unpack_vec<DT>(ldg_vec(b_row, k / EPV), xb);
            } else {
#pragma unroll
                for (int j = 0; j < EPV; ++j) xb[j] = 0.f;
            }
#pragma unroll
            for (int j = 0; j < EPV; ++j) f(k + j, xa[j], xb[j]);
        }
    } else {
        for (int k = k0; k < k1; ++k) f(k, load_logit<DT>(a_row, k), with_b ? load_logit<DT>(b_row, k) : 0.f);
    }
}

// Tree: the deepest node whose whole path passes (ties: lowest index), its depth and path.
// Called by all threads of the CTA; leaves sh.n_acc / sh.row_sel and writes the path if `pth` is given.
__device__ __noinline__ void tree_select(const int32_t* par, int G, int max_depth, int32_t* pth, FinishShared& sh) {
    const int tid = threadIdx.x, lane = tid & 31;
    // Depth of every node and "all nodes from the root down to it pass", by pointer jumping:
    // every node keeps (nodes counted, all pass, next ancestor) for the stretch of its path it
    // has seen so far and doubles that stretch each round, so ceil(log2 N) rounds do for any
    // tree shape (a serial walk takes N dependent steps for a chain-shaped tree of N nodes).
    const bool good = !(sh.bad & FSD_ROW_BADTREE);
    constexpr int kPer = (kMaxTreeNodes + kFinishThreads - 1) / kFinishThreads;
    if (tid == 0) sh.best_key = -1;
    if (good) {
        for (int j = tid; j < G; j += kFinishThreads) {
            sh.tree_jump[j] = static_cast<int16_t>(par[j]);
            sh.tree_depth[j] = 1;
            sh.tree_ok[j] = sh.tree_bit[j];
        }
        __syncthreads();
        for (int span = 1; span < G; span <<= 1) {
            int nj[kPer], nd[kPer], no[kPer];
#pragma unroll
            for (int q = 0; q < kPer; ++q) {
                const int j = tid + q * kFinishThreads;
                nj[q] = -1; nd[q] = 0; no[q] = 0;
                if (j < G) {
                    const int p = sh.tree_jump[j];
                    nj[q] = p; nd[q] = sh.tree_depth[j]; no[q] = sh.tree_ok[j];
                    if (p >= 0) { nj[q] = sh.tree_jump[p]; nd[q] += sh.tree_depth[p]; no[q] &= sh.tree_ok[p]; }
                }
            }
            __syncthreads();
#pragma unroll
            for (int q = 0; q < kPer; ++q) {
                const int j = tid + q * kFinishThreads;
                if (j < G) {
                    sh.tree_jump[j] = static_cast<int16_t>(nj[q]);
                    sh.tree_depth[j] = static_cast<int16_t>(nd[q]);
                    sh.tree_ok[j] = static_cast<int8_t>(no[q]);
                }
            }
            __syncthreads();
        }
        // deepest passing node within max_depth, ties to the lowest index
        int key = -1;
        for (int j = tid; j < G; j += kFinishThreads) {
            const int d = sh.tree_depth[j];
            if (sh.tree_ok[j] && d <= max_depth) {
                const int k = d * 2048 + (2047 - j);
                key = k > key ? k : key;
            }
        }
        key = __reduce_max_sync(0xffffffffu, key);
        if (lane == 0 && key >= 0) atomicMax(&sh.best_key, key);
    }
    __syncthreads();
    if (tid == 0) {
        const int key = sh.best_key;
        const int best = key < 0 ? -1 : 2047 - (key & 2047), best_depth = key < 0 ? 0 : key >> 11;
        sh.n_acc = best_depth;
        sh.row_sel = best + 1;
        if (pth != nullptr) {
            for (int d = 0; d < max_depth; ++d) pth[d] = -1;
            for (int j = best, d = best_depth - 1; j >= 0 && d >= 0; j = par[j], --d) pth[d] = j;
        }
    }
}

template <int DT>
__global__ void __launch_bounds__(kFinishThreads, 2) fsd_finish_kernel(FinishParams P) {
    __shared__ FinishShared sh;
    cg::cluster_group cluster = cg::this_cluster();
    const int cs = static_cast<int>(cluster.num_blocks());
    const int rank = static_cast<int>(cluster.block_rank());
    const int b = blockIdx.x / cs;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int G = P.G, V = P.V;
    const size_t rb = static_cast<size_t>(V) * Logit<DT>::kBytes;
    const char* t_base = static_cast<const char*>(P.target) + static_cast<size_t>(b) * (G + 1) * rb;
    const char* d_base = static_cast<const char*>(P.draft) + static_cast<size_t>(b) * G * rb;
    const bool tree = P.parent != nullptr;

    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");     // "this CTA has started": waited for below
    if (tid == 0) { sh.cand = 0x7fffffff; sh.last_pos = -1; sh.n_acc = G; sh.bad = 0; sh.row_sel = 0; sh.token = -1; sh.amb = 0; }
    __syncthreads();
    // everything above touched no global memory; what follows reads what the pair kernel wrote
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");       // every CTA of the cluster runs: its shared memory may be written

    // ---- 1. divergences, accept bits, status of this row's pairs ----
    // (asked for now, needed later: each is a trip to L2 or HBM of its own)
    const float u_draw = P.u_sample[b];
    int st = 0, first = G;
    if (tid == 0 && P.timeout_flag != nullptr && *reinterpret_cast<const volatile int*>(P.timeout_flag) != 0) st |= FSD_ROW_TIMEOUT;
    if (P.records != nullptr) {
        // two pairs per warp: sixteen lanes fold a pair's record, the first of them judges it
        for (int i0 = 2 * warp; i0 < G; i0 += 2 * (blockDim.x >> 5)) {
            const int i = i0 + (lane >> 4);
            const int item = b * G + i;
            const PairTotals tot = fold_record(i < G ? P.records + item : nullptr, P.div);
            // the two logarithms the judgement needs, by two lanes at once
            const double lz = log((lane & 15) == 1 ? tot.Zb : tot.Za);
            const double lnZa = lz, lnZb = __shfl_down_sync(0xffffffffu, lz, 1);
            if (i < G && (lane & 15) == 0) {
                int trow = i;
                if (tree) {
                    const int par = P.parent[item];
                    trow = (par >= -1 && par < i) ? par + 1 : 0;
                }
                float D;
                int bit, s;
                judge_record(P, item, tot, lnZa, lnZb, t_base + static_cast<size_t>(trow) * rb, d_base + static_cast<size_t>(i) * rb, DT, D, bit, s);
                if (rank == 0) P.divergence[item] = D;
                st |= s;
                if (i < kMaxTreeNodes) {
                    const float za = static_cast<float>(tot.Za);
                    const bool ok = s == 0 && isfinite(tot.ka) && za > 0.f && za < 3.0e38f;
                    sh.kref[i] = ok ? ceilf(tot.ka + log2f(za)) : __int_as_float(0x7fc00000);
                }
                if (tree) sh.tree_bit[i] = static_cast<int8_t>(bit);
                else if (!bit && i < first) first = i;
            }
        }
    } else {
        for (int i = tid; i < G; i += blockDim.x) {
            const int item = b * G + i;
            const int bit = P.item_bits[item];
            st |= P.item_status[item];
            if (tree) sh.tree_bit[i] = static_cast<int8_t>(bit);
            else if (!bit && i < first) first = i;
        }
    }
    st = __reduce_or_sync(0xffffffffu, st);
    first = __reduce_min_sync(0xffffffffu, first);
    if (lane == 0) {
        if (st) atomicOr(&sh.bad, st);
        if (!tree) atomicMin(&sh.n_acc, first);
    }
    __syncthreads();

    // ---- 2. accepted prefix (chain) or deepest accepted path (tree) ----
    if (!tree) {
        if (tid == 0) sh.row_sel = sh.n_acc;
    } else {
        tree_select(P.parent + static_cast<size_t>(b) * G, G, P.max_depth,
                    rank == 0 ? P.path + static_cast<size_t>(b) * P.max_depth : nullptr, sh);
        __syncthreads();
        FSD_CHECK(P.debug_word, sh.row_sel >= 0 && sh.row_sel <= G && sh.n_acc >= 0 && sh.n_acc <= P.max_depth, kChkPath);
    }
    __syncthreads();
    const int n = sh.n_acc, row_sel = sh.row_sel;
    FSD_CHECK(P.debug_word, row_sel >= 0 && row_sel <= G && n >= 0 && n <= (tree ? P.max_depth : G), kChkRow);
    int status = sh.bad;
    if (status & FSD_ROW_BADTREE) {                      // uniform over the cluster
        if (rank == 0 && tid == 0) { P.accept_len[b] = 0; P.next_token[b] = -1; P.row_status[b] = status; }
        return;
    }

    // ---- 3. token draw ----
    constexpr int EPV = Logit<DT>::kPerVec;
    const bool vec = P.vec != 0;
    const bool residual0 = (P.mode != FSD_MODE_FSD) && !tree && n < G;
    const bool greedy = P.sample == FSD_SAMPLE_GREEDY;
    const char* a_row = t_base + static_cast<size_t>(row_sel) * rb;
    const char* b_row = d_base + static_cast<size_t>(residual0 ? n : 0) * rb;
    const double* tab = sh.exp_table;

    // contiguous chunk of the vocabulary owned by this thread
    const int tt = cs * blockDim.x;
    const int L = vec ? ((V / EPV + tt - 1) / tt) * EPV : (V + tt - 1) / tt;
    const long long k0l = static_cast<long long>(rank * blockDim.x + tid) * L;
    const int k0 = k0l < V ? static_cast<int>(k0l) : V;
    const int k1 = (k0l + L) < V ? static_cast<int>(k0l + L) : V;
    FSD_CHECK(P.debug_word, k0 >= 0 && k0 <= k1 && k1 <= V && (!vec || k0 % EPV == 0), kChkChunk);
    FinishExchange mine;
    const FinishExchange* all = sh.all[0];
    double* const sc = sh.sc;

    // ---- fast path: inverse CDF over P_T (the FSD rule, and every bonus token) ----
    if (!residual0 && !greedy) {
        // Reference exponent k (log2 domain, an integer) at or just above the row's log-sum-exp, so
        // that every exponent is <= 0 and those of the entries that carry mass are small (their
        // rounding error stays far below the 1e-6 the draw may be off by).  When the row was a
        // pair's target row the pair's record gives the log-sum-exp; otherwise one pass for the
        // row maximum.
        float kref = 0.f;
        bool have_ref = false;
        if (P.records != nullptr && !tree && n < G && n < kMaxTreeNodes) {
            kref = sh.kref[n];                            // left by the thread that judged the rejected pair
            have_ref = kref == kref;
        }
        if (!have_ref) {
            float m[1] = {-INFINITY};
            for_chunk<DT>(a_row, b_row, k0, k1, vec, false, [&](int, float xa, float) { m[0] = fmaxf(m[0], xa); });
            block_max<1>(m, sh.red_f);
            cluster_gather(cluster, sh, cs, rank, 0, m[0], 0);
            double M = -INFINITY;
            for (int r = 0; r < cs; ++r) M = fmax(M, sh.gather_d[0][r]);
            if (!isfinite(M)) {                           // no finite logit, or +inf: uniform over the cluster
                if (rank == 0 && tid == 0) { P.accept_len[b] = n; P.next_token[b] = -1; P.row_status[b] = status | FSD_ROW_NONFINITE; }
                return;
            }
            kref = ceilf(static_cast<float>(M) * kLog2e);
        }
        // weight of one entry: 2^(logit * log2e - k), the same float in every pass
        const float nk = -kref;
        auto weight = [&](float xa) -> float { return ex2(fmaf(xa, kLog2e, nk)); };
        double csum = 0.0;
        for_chunk<DT>(a_row, b_row, k0, k1, vec, false, [&](int, float xa, float) { csum += static_cast<double>(weight(xa)); });
        // inclusive / exclusive scan of the chunk sums over the CTA, fixed order
        double incl = csum;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const double up = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += up;
        }
        double excl = __shfl_up_sync(0xffffffffu, incl, 1);
        if (lane == 0) excl = 0.0;
        if (lane == 31) sh.warp_tot[warp] = incl;
        __syncthreads();
        double wpre = 0.0, cta_tot = 0.0;
        for (int w = 0; w < kFinishWarps; ++w) {
            if (w == warp) wpre = cta_tot;
            cta_tot += sh.warp_tot[w];
        }
        incl += wpre;
        excl += wpre;
        cluster_gather(cluster, sh, cs, rank, 1, cta_tot, 0);
        double W = 0.0;
        for (int r = 0; r < cs; ++r) W += sh.gather_d[1][r];
        if (!(isfinite(W) && W > 0.0)) {                  // NaN logit (or nothing representable): uniform over the cluster
            if (rank == 0 && tid == 0) { P.accept_len[b] = n; P.next_token[b] = -1; P.row_status[b] = status | FSD_ROW_NONFINITE; }
            return;
        }
        if (rank == 0 && tid == 0) { P.accept_len[b] = n; P.row_status[b] = status; }
        const double t = static_cast<double>(u_draw) * W;
        double cpre = 0.0, run = 0.0;
        int owner = -1;
        for (int r = 0; r < cs && owner < 0; ++r) {
            cpre = run;
            run += sh.gather_d[1][r];
            if (run > t) owner = r;
        }
        auto last_with_weight = [&]() -> int {           // highest index of this thread's chunk whose weight is positive
            int lastp = -1;
            for_chunk<DT>(a_row, b_row, k0, k1, vec, false, [&](int k, float xa, float) { if (weight(xa) > 0.f) lastp = k; });
            return lastp;
        };
        if (owner < 0) {                                  // t >= W after rounding (uniform): the last token that has weight
            const int lp = __reduce_max_sync(0xffffffffu, last_with_weight());
            if (lane == 0 && lp >= 0) atomicMax(&sh.last_pos, lp);
            __syncthreads();
            cluster_gather(cluster, sh, cs, rank, 0, 0.0, sh.last_pos);
            int best = -1;
            for (int r = 0; r < cs; ++r) best = sh.gather_i[0][r] > best ? sh.gather_i[0][r] : best;
            if (rank == 0 && tid == 0) P.next_token[b] = best;
            return;
        }
        if (owner != rank) return;
        const double t_local = t - cpre;
        if (csum > 0.0 && incl > t_local) atomicMin(&sh.cand, tid);
        __syncthreads();
        const int c = sh.cand;
        if (c == 0x7fffffff) {                            // crossing lost to rounding inside this CTA
            const int lp = __reduce_max_sync(0xffffffffu, last_with_weight());
            if (lane == 0 && lp >= 0) atomicMax(&sh.last_pos, lp);
            __syncthreads();
            if (tid == 0) P.next_token[b] = sh.last_pos;
        } else if (warp == (c >> 5)) {
            // The warp of the thread whose chunk holds the crossing walks that chunk together: lane j
            // takes the chunk's j-th unit (a 16-byte vector, or one entry of an unaligned row) and sums
            // its weights in index order; every lane then adds the units' sums in order until the
            // running sum passes the target, and the lane of that unit finds the entry.
            const int src = c & 31;
            const int ck0 = __shfl_sync(0xffffffffu, k0, src), ck1 = __shfl_sync(0xffffffffu, k1, src);
            double run = __shfl_sync(0xffffffffu, excl, src);
            const int U = vec ? EPV : 1;
            int tok = -1, lastp = -1;
            for (int u0 = ck0; u0 < ck1 && tok < 0; u0 += 32 * U) {
                const int uk = u0 + lane * U;
                float w[EPV];
#pragma unroll
                for (int j = 0; j < EPV; ++j) w[j] = 0.f;
                if (uk < ck1) {
                    if (vec) {
                        float xa[EPV];
                        unpack_vec<DT>(ldg_vec(a_row, uk / EPV), xa);
#pragma unroll
                        for (int j = 0; j < EPV; ++j) w[j] = weight(xa[j]);
                    } else {
                        w[0] = weight(load_logit<DT>(a_row, uk));
                    }
                }
                double usum = 0.0;
                int ulast = -1;
#pragma unroll
                for (int j = 0; j < EPV; ++j) {
                    usum += static_cast<double>(w[j]);
                    if (w[j] > 0.f) ulast = uk + j;
                }
                int hit = -1;                            // unit in which the running sum passes the target
                double before = 0.0;                     // the running sum in front of that unit
                const int nunits = min(32, (ck1 - u0 + U - 1) / U);
                for (int j = 0; j < nunits; ++j) {
                    const double sj = __shfl_sync(0xffffffffu, usum, j);
                    if (hit < 0) {
                        if (sj > 0.0 && run + sj > t_local) { hit = j; before = run; }
                        else run += sj;
                    }
                }
                lastp = max(lastp, __reduce_max_sync(0xffffffffu, ulast));
                if (hit >= 0) {
                    int t_here = -1;
                    if (lane == hit) {
                        double r2 = before;
#pragma unroll
                        for (int j = 0; j < EPV; ++j) {
                            r2 += static_cast<double>(w[j]);
                            if (t_here < 0 && w[j] > 0.f && r2 > t_local) t_here = uk + j;
                        }
                        if (t_here < 0) t_here = ulast;   // lost to the order of the additions: the unit's last entry with weight
                    }
                    tok = __shfl_sync(0xffffffffu, t_here, hit);
                }
            }
            if (tok < 0) tok = lastp;
            FSD_CHECK(P.debug_word, tok >= -1 && tok < V, kChkToken);
            if (lane == 0) P.next_token[b] = tok;
        }
        return;
    }

    // the paths below take their exponentials in double precision from a table
    if (tid < kExpTable) sh.exp_table[tid] = exp2(static_cast<double>(tid) * (1.0 / kExpTable));
    if (tid == 0) {
        sh.exp_consts[0] = 6755399441055744.0; sh.exp_consts[1] = 256.0;
        sh.exp_consts[2] = 2.239395190875157e-12; sh.exp_consts[3] = 3.308302680541371e-09;
        sh.exp_consts[4] = 3.665565596910106e-06; sh.exp_consts[5] = 2.7076061740622863e-03;
    }
    __syncthreads();

    // ---- references.  A residual draw follows a rejection, so the rejected pair's record has
    //      references (log2 domain) for both rows, near their maxima and common to the cluster;
    //      otherwise one pass for the CTA-local maxima (exact), and for the greedy FSD choice the
    //      argmax of the logits ----
    double kra = 0.0, krb = 0.0;
    double zea = 0.0, zeb = 0.0;
    bool common = false;
    if (residual0 && P.records != nullptr) {
        const PairRecord* r = P.records + (static_cast<size_t>(b) * G + n);
        if (r->state & kRecordStats) {
            float fa = -INFINITY, fb = -INFINITY;
            bool nan = false;
            for (uint32_t c = 0; c < r->ncta && c < kMaxGroupSize; ++c) {
                const float a = r->part[c].ka, q = r->part[c].kb;
                nan = nan || a != a || q != q;
                fa = fmaxf(fa, a); fb = fmaxf(fb, q);
            }
            if (!nan && isfinite(fa) && isfinite(fb)) {
                kra = fa; krb = fb; common = true;
                // the record's (single-precision) normalisers on these references: an estimate of Z_a / Z_b
                for (uint32_t c = 0; c < r->ncta && c < kMaxGroupSize; ++c) {
                    const float a = r->part[c].ka, q = r->part[c].kb;
                    if (a != -INFINITY) zea += static_cast<double>(r->part[c].za) * pow2_int_d(static_cast<double>(a) - fa);
                    if (q != -INFINITY) zeb += static_cast<double>(r->part[c].zb) * pow2_int_d(static_cast<double>(q) - fb);
                }
            }
        }
    }
    float mx[2] = {-INFINITY, -INFINITY};
    int amax = 0x7fffffff;
    float amax_v = -INFINITY;
    if (!common) {
        for_chunk<DT>(a_row, b_row, k0, k1, vec, residual0, [&](int k, float xa, float xb) {
            if (xa > amax_v) { amax_v = xa; amax = k; }
            mx[1] = fmaxf(mx[1], xb);
        });
        mx[0] = amax_v;
        block_max<2>(mx, sh.red_f);
    }
    const double Ra = common ? 0.0 : mx[0], Rb = common ? 0.0 : mx[1];   // this CTA's references (logit domain)

    if (greedy && !residual0) {
        // argmax of P_T == argmax of the logits, ties to the lowest index
        float best = amax_v;
        int idx = amax;
#pragma unroll
        for (int m = 16; m > 0; m >>= 1) {
            const float ob = __shfl_xor_sync(0xffffffffu, best, m);
            const int oi = __shfl_xor_sync(0xffffffffu, idx, m);
            if (ob > best || (ob == best && oi < idx)) { best = ob; idx = oi; }
        }
        if (lane == 0) { sh.red_d[warp * 2] = best; sh.red_d[warp * 2 + 1] = idx; }
        __syncthreads();
        best = static_cast<float>(sh.red_d[0]); idx = static_cast<int>(sh.red_d[1]);
        for (int w = 1; w < kFinishWarps; ++w) {
            const float ob = static_cast<float>(sh.red_d[w * 2]);
            const int oi = static_cast<int>(sh.red_d[w * 2 + 1]);
            if (ob > best || (ob == best && oi < idx)) { best = ob; idx = oi; }
        }
        // a NaN or +inf logit, or no finite logit, makes the row invalid: detect through the sum of the logits' signs
        float bad_v = 0.f;
        for_chunk<DT>(a_row, b_row, k0, k1, vec, false, [&](int, float xa, float) { if (xa != xa || xa == INFINITY) bad_v = 1.f; });
        float bv[1] = {bad_v};
        block_max<1>(bv, sh.red_f);
        mine.d[0] = best; mine.d[1] = bv[0]; mine.d[2] = 0; mine.d[3] = 0; mine.i[0] = idx; mine.i[1] = 0;
        cluster_exchange(cluster, sh, cs, rank, 0, mine);
        double gb = all[0].d[0], gbad = all[0].d[1];
        int gi = all[0].i[0];
        for (int r = 1; r < cs; ++r) {
            if (all[r].d[0] > gb || (all[r].d[0] == gb && all[r].i[0] < gi)) { gb = all[r].d[0]; gi = all[r].i[0]; }
            gbad = fmax(gbad, all[r].d[1]);
        }
        const bool ok = gbad == 0.0 && gb > -INFINITY;
        if (rank == 0 && tid == 0) {
            P.accept_len[b] = n;
            P.next_token[b] = ok ? gi : -1;
            P.row_status[b] = status | (ok ? 0 : FSD_ROW_NONFINITE);
        }
        return;
    }

    // with common references (the usual case): y = x * log2e - k; logits below xmin give 2^y < 2^-990 and count as 0
    const Exp2Consts ec = exp2_consts(sh.exp_consts);
    const double nka = -kra, nkb = -krb;
    const float xmin_a = static_cast<float>((kra - 990.0) * kLn2D), xmin_b = static_cast<float>((krb - 990.0) * kLn2D);

    // ---- residual only: global normalisers of both rows (double) ----
    double Ma = Ra, Mb = Rb, iZa = 0.0, iZb = 0.0;
    bool residual = residual0;
    // One pass instead of two, where it can be shown to give the same sums.  An entry has residual
    // weight iff e_a / Z_a > e_b / Z_b, i.e. e_a > rho * e_b with rho = Z_a / Z_b, which is known
    // only after the pass -- but the record gives rho to about 1e-6.  Entries are classed against
    // rho_est * (1 +- 1e-4): for those clearly above, e_a and e_b are summed separately, and the
    // chunk's residual weight is then sum e_a / Z_a - sum e_b / Z_b with the exact normalisers.
    // The few entries between the two bounds (about one in 10^4) are remembered, two a thread, and
    // settled with the exact normalisers afterwards; a thread with more of them, or an estimate
    // that turns out further than 5e-5 off, sends the whole row through the second pass instead.
    double sa = 0.0, sb = 0.0;
    int lastp1 = -1, amb = 0, namb = 0, ak0 = -1, ak1 = -1;
    bool one_pass = false;
    if (residual0) {
        double z[2] = {0.0, 0.0};
        if (common && vec) {
            // the usual case (a rejected pair with a record): both rows, two independent exponentials an entry
            const bool classify = !greedy && zea > 0.0 && zeb > 0.0 && isfinite(zea) && isfinite(zeb);
            const double rho_est = classify ? zea / zeb : 0.0;
            const double rho_hi = rho_est * (1.0 + 1e-4), rho_lo = rho_est * (1.0 - 1e-4);
            for (int k = k0; k < k1; k += EPV) {
                float xa[EPV], xb[EPV];
                unpack_vec<DT>(ldg_vec(a_row, k / EPV), xa);
                unpack_vec<DT>(ldg_vec(b_row, k / EPV), xb);
#pragma unroll
                for (int e = 0; e < EPV; ++e) {
                    const double pa = exp2_of_logit(xa[e], xmin_a, nka, tab, ec);
                    const double pb = exp2_of_logit(xb[e], xmin_b, nkb, tab, ec);
                    z[0] += pa;
                    z[1] += pb;
                    if (pa > rho_hi * pb) { sa += pa; sb += pb; lastp1 = k + e; }
                    else if (!(pa < rho_lo * pb) && pa > 0.0) {            // (pa == 0: no weight whatever rho is)
                        if (namb == 0) ak0 = k + e; else ak1 = k + e;
                        ++namb;
                    }
                }
            }
            if (!classify || namb > 2) amb = 1;
            if (amb) atomicOr(&sh.amb, 1);
        } else
        for_chunk<DT>(a_row, b_row, k0, k1, vec, true, [&](int, float xa, float xb) {
            if (common) {
                z[0] += exp2_of_logit(xa, xmin_a, nka, tab, ec);
                z[1] += exp2_of_logit(xb, xmin_b, nkb, tab, ec);
            } else {
                if (Ra > -INFINITY) z[0] += exp2_table((static_cast<double>(xa) - Ra) * kLog2eD, tab);
                if (Rb > -INFINITY) z[1] += exp2_table((static_cast<double>(xb) - Rb) * kLog2eD, tab);
            }
        });
        block_sum<2>(z, sh.red_d);                        // (its barriers also order the flag above)
        mine.d[0] = Ra; mine.d[1] = Rb; mine.d[2] = z[0]; mine.d[3] = z[1]; mine.i[0] = (common && vec) ? sh.amb : 1; mine.i[1] = 0;
        cluster_exchange(cluster, sh, cs, rank, 0, mine);
        Ma = -INFINITY; Mb = -INFINITY;
        for (int r = 0; r < cs; ++r) { Ma = fmax(Ma, all[r].d[0]); Mb = fmax(Mb, all[r].d[1]); }
        double Za = 0.0, Zb = 0.0;
        for (int r = 0; r < cs; ++r) {
            if (all[r].d[0] > -INFINITY) Za += all[r].d[2] * exp2_table((all[r].d[0] - Ma) * kLog2eD, tab);
            if (all[r].d[1] > -INFINITY) Zb += all[r].d[3] * exp2_table((all[r].d[1] - Mb) * kLog2eD, tab);
        }
        const bool a_ok = isfinite(Ma) && isfinite(Za) && Za > 0.0, b_ok = isfinite(Mb) && isfinite(Zb) && Zb > 0.0;
        if (!a_ok) {                                      // uniform over the cluster
            if (rank == 0 && tid == 0) { P.accept_len[b] = n; P.next_token[b] = -1; P.row_status[b] = status | FSD_ROW_NONFINITE; }
            return;
        }
        if (!b_ok) { residual = false; status |= FSD_ROW_NONFINITE; }
        else { iZa = 1.0 / Za; iZb = 1.0 / Zb; }
        int any_amb = 0;
        for (int r = 0; r < cs; ++r) any_amb |= all[r].i[0];
        one_pass = b_ok && any_amb == 0 && fabs(zea * Zb - zeb * Za) <= 5e-5 * zeb * Za;     // |rho_est - rho| <= 5e-5 rho
    }

    for (int attempt = 0; attempt < 2; ++attempt) {
        // weight of one vocabulary entry: P_T relative to this CTA's maximum, or the SD residual
        auto weight = [&](float xa, float xb) -> double {
            if (common) {                                  // the same values as the tight loops
                const double pa = exp2_of_logit(xa, xmin_a, nka, tab, ec);
                if (!residual) return pa;
                const double r = pa * iZa - exp2_of_logit(xb, xmin_b, nkb, tab, ec) * iZb;
                return r > 0.0 ? r : 0.0;
            }
            if (!residual) return Ra > -INFINITY ? exp2_table((static_cast<double>(xa) - Ra) * kLog2eD, tab) : 0.0;
            const double r = exp2_table((static_cast<double>(xa) - Ma) * kLog2eD, tab) * iZa -
                             exp2_table((static_cast<double>(xb) - Mb) * kLog2eD, tab) * iZb;
            return r > 0.0 ? r : 0.0;
        };
        double csum = 0.0, wbest = 0.0;
        int lastp = -1, kbest = 0x7fffffff;
        if (attempt == 0 && one_pass && residual) {
            csum = sa * iZa - sb * iZb;
            if (!(csum > 0.0)) csum = 0.0;
            lastp = csum > 0.0 ? lastp1 : -1;
            for (int j = 0; j < namb; ++j) {              // the entries that were too close to call, now with the exact normalisers
                const int k = j == 0 ? ak0 : ak1;
                const double r = exp2_of_logit(load_logit<DT>(a_row, k), xmin_a, nka, tab, ec) * iZa -
                                 exp2_of_logit(load_logit<DT>(b_row, k), xmin_b, nkb, tab, ec) * iZb;
                if (r > 0.0) { csum += r; lastp = k > lastp ? k : lastp; }
            }
        } else if (common && vec && residual && !greedy) {
            for (int k = k0; k < k1; k += EPV) {
                float xa[EPV], xb[EPV];
                unpack_vec<DT>(ldg_vec(a_row, k / EPV), xa);
                unpack_vec<DT>(ldg_vec(b_row, k / EPV), xb);
#pragma unroll
                for (int e = 0; e < EPV; ++e) {
                    const double pa = exp2_of_logit(xa[e], xmin_a, nka, tab, ec);
                    const double pb = exp2_of_logit(xb[e], xmin_b, nkb, tab, ec);
                    const double r = pa * iZa - pb * iZb;
                    if (r > 0.0) { csum += r; lastp = k + e; }
                }
            }
        } else
        for_chunk<DT>(a_row, b_row, k0, k1, vec, residual, [&](int k, float xa, float xb) {
            const double w = weight(xa, xb);
            csum += w;
            if (w > 0.0) lastp = k;
            if (greedy && w > wbest) { wbest = w; kbest = k; }
        });
        // inclusive / exclusive scan of the chunk sums over the CTA, fixed order
        double incl = csum;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const double up = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += up;
        }
        double excl = __shfl_up_sync(0xffffffffu, incl, 1);
        if (lane == 0) excl = 0.0;
        if (lane == 31) sh.warp_tot[warp] = incl;
        if (greedy) {                                     // residual arg-max of the warp, ties to the lowest index
#pragma unroll
            for (int m = 16; m > 0; m >>= 1) {
                const double ob = shfl_xor_d(wbest, m);
                const int oi = __shfl_xor_sync(0xffffffffu, kbest, m);
                if (ob > wbest || (ob == wbest && oi < kbest)) { wbest = ob; kbest = oi; }
            }
            if (lane == 0) { sh.red_d[warp * 2] = wbest; sh.red_d[warp * 2 + 1] = kbest; }
        }
        const int lp = __reduce_max_sync(0xffffffffu, lastp);
        if (lane == 0 && lp >= 0) atomicMax(&sh.last_pos, lp);
        __syncthreads();
        double wpre = 0.0, cta_tot = 0.0;
        for (int w = 0; w < kFinishWarps; ++w) {
            if (w == warp) wpre = cta_tot;
            cta_tot += sh.warp_tot[w];
        }
        incl += wpre;
        excl += wpre;
        if (greedy) {
            wbest = sh.red_d[0]; kbest = static_cast<int>(sh.red_d[1]);
            for (int w = 1; w < kFinishWarps; ++w) {
                const double ob = sh.red_d[w * 2];
                const int oi = static_cast<int>(sh.red_d[w * 2 + 1]);
                if (ob > wbest || (ob == wbest && oi < kbest)) { wbest = ob; kbest = oi; }
            }
        }
        mine.d[0] = cta_tot; mine.d[1] = Ra; mine.d[2] = wbest; mine.d[3] = 0; mine.i[0] = sh.last_pos; mine.i[1] = kbest;
        cluster_exchange(cluster, sh, cs, rank, 1 - (attempt & 1), mine);
        all = sh.all[1 - (attempt & 1)];

        // cluster totals on a common reference
        double M = -INFINITY;
        for (int r = 0; r < cs; ++r) M = fmax(M, all[r].d[1]);
        double W = 0.0;
        __syncthreads();                                  // everybody is done with the last attempt's factors
        if (tid < cs) sc[tid] = residual ? 1.0 : (all[tid].d[1] > -INFINITY ? exp2_table((all[tid].d[1] - M) * kLog2eD, tab) : 0.0);
        __syncthreads();
        for (int r = 0; r < cs; ++r) W += all[r].d[0] * sc[r];
        if (residual && !(W > 0.0)) {                     // no residual mass: draw from P_T (uniform decision)
            residual = false;
            __syncthreads();
            if (tid == 0) sh.last_pos = -1;
            __syncthreads();
            continue;
        }
        if (!residual && !(isfinite(M) && isfinite(W) && W > 0.0)) {     // uniform over the cluster
            if (rank == 0 && tid == 0) { P.accept_len[b] = n; P.next_token[b] = -1; P.row_status[b] = status | FSD_ROW_NONFINITE; }
            return;
        }
        if (rank == 0 && tid == 0) { P.accept_len[b] = n; P.row_status[b] = status; }

        if (greedy) {                                     // residual arg-max over the cluster
            double gb = all[0].d[2];
            int gi = all[0].i[1];
            for (int r = 1; r < cs; ++r)
                if (all[r].d[2] > gb || (all[r].d[2] == gb && all[r].i[1] < gi)) { gb = all[r].d[2]; gi = all[r].i[1]; }
            if (rank == 0 && tid == 0) P.next_token[b] = gi;
            return;
        }

        const double t = static_cast<double>(u_draw) * W;
        double cpre = 0.0, run = 0.0;
        int owner = -1, last_any = -1;
        for (int r = 0; r < cs; ++r) {
            if (owner < 0) {
                cpre = run;
                run += all[r].d[0] * sc[r];
                if (run > t) owner = r;
            }
            if (all[r].i[0] > last_any) last_any = all[r].i[0];
        }
        if (owner < 0) {                                  // t >= W after rounding: the last token that has weight
            if (rank == 0 && tid == 0) P.next_token[b] = last_any;
            return;
        }
        if (owner != rank) return;
        const double t_local = (t - cpre) / sc[owner];    // the target on this CTA's own scale
        if (csum > 0.0 && incl > t_local) atomicMin(&sh.cand, tid);
        __syncthreads();
        const int c = sh.cand;
        if (c == 0x7fffffff) {                            // crossing lost to rounding inside this CTA
            if (tid == 0) P.next_token[b] = sh.last_pos;
        } else if (warp == (c >> 5)) {
            // the warp of the thread whose chunk holds the crossing walks that chunk together
            const int src = c & 31;
            const int ck0 = __shfl_sync(0xffffffffu, k0, src), ck1 = __shfl_sync(0xffffffffu, k1, src);
            double base = __shfl_sync(0xffffffffu, excl, src);
            int tok = 0x7fffffff;
            const int fallback = __shfl_sync(0xffffffffu, lastp, src);
            for (int kb = ck0; kb < ck1; kb += 32) {
                const int k = kb + lane;
                double w = 0.0;
                if (k < ck1) w = weight(load_logit<DT>(a_row, k), residual ? load_logit<DT>(b_row, k) : 0.f);
                double run = w;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const double up = __shfl_up_sync(0xffffffffu, run, d);
                    if (lane >= d) run += up;
                }
                run += base;
                if (k < ck1 && run > t_local && k < tok) tok = k;
                base = __shfl_sync(0xffffffffu, run, 31);
            }
            tok = __reduce_min_sync(0xffffffffu, tok);
            FSD_CHECK(P.debug_word, (tok != 0x7fffffff ? tok : fallback) >= -1 && (tok != 0x7fffffff ? tok : fallback) < V, kChkToken);
            if (lane == 0) P.next_token[b] = tok != 0x7fffffff ? tok : fallback;
        }
        return;
    }
}
}  // namespace fsd
