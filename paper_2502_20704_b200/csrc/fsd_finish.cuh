// Finish kernel: one thread-block cluster per batch row.  Finds the accepted prefix
// (chain) or the deepest accepted path (tree) from the per-pair accept bits, then draws
// the replacement / bonus token from one target row (and, for the SD residual, one
// draft row) by an inverse CDF in vocabulary order.
//
// The draw must land on the same token as a sequential double-precision sum would, so
// this kernel evaluates its exponentials and partial sums in double precision: each
// thread owns a contiguous chunk of the vocabulary, chunk sums are combined by a
// fixed-order scan (thread -> warp -> CTA -> cluster), the first thread whose inclusive
// sum exceeds u * total re-walks its chunk.  The rows involved are a 1/(2*gamma+1)
// share of the logits, and the fp64 pipe is otherwise idle.
#pragma once

#include "fsd_device.cuh"

namespace fsd {

constexpr int kFinishThreads = 512;
constexpr int kMaxClusterSize = 8;
constexpr int kMaxTreeNodes = 1024;

struct FinishParams {
    const void* target;        // [B, G+1, V]
    const void* draft;         // [B, G,   V]
    const int32_t* parent;     // tree only
    const float* u_sample;     // [B]
    int B, G, V;
    int mode, sample, max_depth;
    const int32_t* item_bits;
    const int32_t* item_status;
    const int* timeout_flag;   // nonzero: a bounded wait of the streaming kernel ran out (may be null)
    int32_t* accept_len;       // [B]
    int32_t* path;             // [B, max_depth] (tree) or null
    int32_t* next_token;       // [B]
    int32_t* row_status;       // [B]
};

struct FinishShared {
    double slot_d[2];          // values this CTA publishes to its cluster
    int slot_i[2];
    double red_d[32 * 2];
    float red_f[32 * 2];
    double warp_tot[32];
    int cand;                  // lowest thread whose inclusive sum exceeds the target
    int last_pos;              // highest index with a positive weight in this CTA
    int row_sel;               // target row the token is drawn from
    int n_acc;
    int bad;
    int16_t tree_depth[kMaxTreeNodes];
    int8_t tree_ok[kMaxTreeNodes];
};

// Every CTA of the cluster publishes two doubles and two ints and reads everybody's.
// Two cluster barriers: after the writes, and after the reads (so slots can be reused).
__device__ __forceinline__ void cluster_exchange(cg::cluster_group& cluster, FinishShared& sh, int cs,
                                                 double d0, double d1, int i0, int i1,
                                                 double (&od0)[kMaxClusterSize], double (&od1)[kMaxClusterSize],
                                                 int (&oi0)[kMaxClusterSize], int (&oi1)[kMaxClusterSize]) {
    if (threadIdx.x == 0) {
        sh.slot_d[0] = d0; sh.slot_d[1] = d1;
        sh.slot_i[0] = i0; sh.slot_i[1] = i1;
    }
    cluster.sync();
#pragma unroll
    for (int r = 0; r < kMaxClusterSize; ++r) {
        if (r < cs) {
            const FinishShared* rs = cluster.map_shared_rank(&sh, r);
            od0[r] = rs->slot_d[0]; od1[r] = rs->slot_d[1];
            oi0[r] = rs->slot_i[0]; oi1[r] = rs->slot_i[1];
        } else {
            od0[r] = 0.0; od1[r] = 0.0; oi0[r] = 0; oi1[r] = 0;
        }
    }
    cluster.sync();
}

template <int DT>
__global__ void __launch_bounds__(kFinishThreads) fsd_finish_kernel(FinishParams P) {
    __shared__ FinishShared sh;
    cg::cluster_group cluster = cg::this_cluster();
    const int cs = static_cast<int>(cluster.num_blocks());
    const int rank = static_cast<int>(cluster.block_rank());
    const int b = blockIdx.x / cs;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int G = P.G, V = P.V;
    const int32_t* bits = P.item_bits + static_cast<size_t>(b) * G;
    const int32_t* ist = P.item_status + static_cast<size_t>(b) * G;

    // ---- accepted prefix / accepted path (every CTA computes it; rank 0 writes it) ----
    if (tid == 0) { sh.cand = 0x7fffffff; sh.last_pos = -1; sh.n_acc = G; sh.bad = 0; sh.row_sel = 0; }
    __syncthreads();
    int st = 0;
    for (int i = tid; i < G; i += blockDim.x) st |= ist[i];
    if (tid == 0 && P.timeout_flag != nullptr && *P.timeout_flag != 0) st |= FSD_ROW_TIMEOUT;
    st = __reduce_or_sync(0xffffffffu, st);
    if (lane == 0 && st) atomicOr(&sh.bad, st);
    if (P.parent == nullptr) {
        int first = G;
        for (int i = tid; i < G; i += blockDim.x)
            if (!bits[i]) { first = i; break; }
        first = __reduce_min_sync(0xffffffffu, first);
        if (lane == 0) atomicMin(&sh.n_acc, first);
        __syncthreads();
        if (tid == 0) sh.row_sel = sh.n_acc;
    } else {
        __syncthreads();
        if (tid == 0) {
            const int32_t* par = P.parent + static_cast<size_t>(b) * G;
            int best = -1, best_depth = 0;
            if (!(sh.bad & FSD_ROW_BADTREE)) {
                for (int j = 0; j < G; ++j) {
                    const int p = par[j];
                    const int d = p < 0 ? 1 : sh.tree_depth[p] + 1;
                    const bool ok = bits[j] && (p < 0 || sh.tree_ok[p]);
                    sh.tree_depth[j] = static_cast<int16_t>(d);
                    sh.tree_ok[j] = ok;
                    if (ok && d <= P.max_depth && d > best_depth) { best = j; best_depth = d; }
                }
            }
            sh.n_acc = best_depth;
            sh.row_sel = best + 1;
            if (rank == 0) {
                int32_t* pth = P.path + static_cast<size_t>(b) * P.max_depth;
                for (int d = 0; d < P.max_depth; ++d) pth[d] = -1;
                for (int j = best, d = best_depth - 1; j >= 0; j = par[j], --d) pth[d] = j;
            }
        }
    }
    __syncthreads();
    const int n = sh.n_acc, row_sel = sh.row_sel;
    int status = sh.bad;
    if (status & FSD_ROW_BADTREE) {                      // uniform over the cluster
        if (rank == 0 && tid == 0) {
            P.accept_len[b] = 0;
            P.next_token[b] = -1;
            P.row_status[b] = status;
        }
        return;
    }
    const bool residual0 = (P.mode != FSD_MODE_FSD) && P.parent == nullptr && n < G;

    const size_t rb = static_cast<size_t>(V) * Logit<DT>::kBytes;
    const char* a_row = static_cast<const char*>(P.target) + (static_cast<size_t>(b) * (G + 1) + row_sel) * rb;
    const char* b_row = static_cast<const char*>(P.draft) + (static_cast<size_t>(b) * G + (residual0 ? n : 0)) * rb;

    // contiguous chunk of the vocabulary owned by this thread
    const int tt = cs * blockDim.x;
    const int L = (V + tt - 1) / tt;
    const int g = rank * blockDim.x + tid;
    const long long k0l = static_cast<long long>(g) * L;
    const int k0 = k0l < V ? static_cast<int>(k0l) : V;
    const int k1 = (k0l + L) < V ? static_cast<int>(k0l + L) : V;

    double xd0[kMaxClusterSize], xd1[kMaxClusterSize];
    int xi0[kMaxClusterSize], xi1[kMaxClusterSize];

    // ---- maxima (exact) and, for the greedy FSD choice, the argmax of the logits ----
    float mx[2] = {-INFINITY, -INFINITY};
    int amax = 0x7fffffff;
    for (int k = k0; k < k1; ++k) {
        const float a = load_logit<DT>(a_row, k);
        if (a > mx[0]) { mx[0] = a; amax = k; }
        if (residual0) mx[1] = fmaxf(mx[1], load_logit<DT>(b_row, k));
    }
    const float my_max = mx[0];
    block_max<2>(mx, sh.red_f);
    cluster_exchange(cluster, sh, cs, mx[0], mx[1], 0, 0, xd0, xd1, xi0, xi1);
    double Ma = -INFINITY, Mb = -INFINITY;
    for (int r = 0; r < cs; ++r) { Ma = fmax(Ma, xd0[r]); Mb = fmax(Mb, xd1[r]); }

    // ---- normalisers in double ----
    double z[2] = {0.0, 0.0};
    for (int k = k0; k < k1; ++k) {
        z[0] += exp(static_cast<double>(load_logit<DT>(a_row, k)) - Ma);
        if (residual0) z[1] += exp(static_cast<double>(load_logit<DT>(b_row, k)) - Mb);
    }
    block_sum<2>(z, sh.red_d);
    cluster_exchange(cluster, sh, cs, z[0], z[1], 0, 0, xd0, xd1, xi0, xi1);
    double Za = 0.0, Zb = 0.0;
    for (int r = 0; r < cs; ++r) { Za += xd0[r]; Zb += xd1[r]; }
    const bool a_ok = isfinite(Ma) && isfinite(Za) && Za > 0.0;
    bool residual = residual0 && isfinite(Mb) && isfinite(Zb) && Zb > 0.0;
    if (!a_ok) {                                          // uniform over the cluster
        if (rank == 0 && tid == 0) {
            P.accept_len[b] = n;
            P.next_token[b] = -1;
            P.row_status[b] = status | FSD_ROW_NONFINITE;
        }
        return;
    }
    const double iZa = 1.0 / Za, iZb = residual ? 1.0 / Zb : 0.0;
    auto weight = [&](int k, bool res) -> double {
        const double ea = exp(static_cast<double>(load_logit<DT>(a_row, k)) - Ma);
        if (!res) return ea;
        const double r = ea * iZa - exp(static_cast<double>(load_logit<DT>(b_row, k)) - Mb) * iZb;
        return r > 0.0 ? r : 0.0;
    };

    int token = -1;
    for (int attempt = 0; attempt < 2; ++attempt) {
        // chunk sum, last positive index and (greedy) the largest weight of the chunk
        double csum = 0.0, wbest = 0.0;
        int lastp = -1, kbest = 0x7fffffff;
        const bool need_w = residual || P.sample != FSD_SAMPLE_GREEDY;
        for (int k = k0; need_w && k < k1; ++k) {
            const double w = weight(k, residual);
            csum += w;
            if (w > 0.0) lastp = k;
            if (w > wbest) { wbest = w; kbest = k; }
        }
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
        const int nwarps = blockDim.x >> 5;
        for (int w = 0; w < nwarps; ++w) {
            if (w == warp) wpre = cta_tot;
            cta_tot += sh.warp_tot[w];
        }
        incl += wpre;
        excl += wpre;

        if (P.sample == FSD_SAMPLE_GREEDY) {
            // FSD: argmax of p == argmax of the logits; residual: argmax of max(0, p - q)
            double best = residual ? wbest : static_cast<double>(my_max);
            int idx = residual ? kbest : amax;
            // block arg-max with ties to the lowest index
#pragma unroll
            for (int m = 16; m > 0; m >>= 1) {
                const double ob = shfl_xor_d(best, m);
                const int oi = __shfl_xor_sync(0xffffffffu, idx, m);
                if (ob > best || (ob == best && oi < idx)) { best = ob; idx = oi; }
            }
            __syncthreads();
            if (lane == 0) { sh.red_d[warp * 2] = best; sh.red_d[warp * 2 + 1] = static_cast<double>(idx); }
            __syncthreads();
            best = sh.red_d[0];
            idx = static_cast<int>(sh.red_d[1]);
            for (int w = 1; w < nwarps; ++w) {
                const double ob = sh.red_d[w * 2];
                const int oi = static_cast<int>(sh.red_d[w * 2 + 1]);
                if (ob > best || (ob == best && oi < idx)) { best = ob; idx = oi; }
            }
            cluster_exchange(cluster, sh, cs, best, cta_tot, idx, 0, xd0, xd1, xi0, xi1);
            double tot = 0.0;
            for (int r = 0; r < cs; ++r) tot += xd1[r];
            if (residual && !(tot > 0.0)) { residual = false; continue; }   // no residual mass: use P_T
            best = xd0[0]; idx = xi0[0];
            for (int r = 1; r < cs; ++r)
                if (xd0[r] > best || (xd0[r] == best && xi0[r] < idx)) { best = xd0[r]; idx = xi0[r]; }
            token = idx;
            break;
        }

        // highest positive index of this CTA (fallback when rounding leaves no crossing)
        int lp = __reduce_max_sync(0xffffffffu, lastp);
        if (lane == 0 && lp >= 0) atomicMax(&sh.last_pos, lp);
        __syncthreads();
        cluster_exchange(cluster, sh, cs, cta_tot, 0.0, sh.last_pos, 0, xd0, xd1, xi0, xi1);
        double W = 0.0;
        for (int r = 0; r < cs; ++r) W += xd0[r];
        if (residual && !(W > 0.0)) {                     // no residual mass: use P_T (uniform decision)
            residual = false;
            if (tid == 0) sh.last_pos = -1;
            __syncthreads();
            continue;
        }
        const double t = static_cast<double>(P.u_sample[b]) * W;
        // the CTA whose inclusive total first exceeds t
        double cpre = 0.0, run = 0.0;
        int owner = -1, last_any = -1;
        for (int r = 0; r < cs; ++r) {
            if (r == rank) cpre = run;
            run += xd0[r];
            if (owner < 0 && run > t) owner = r;
            if (xi0[r] > last_any) last_any = xi0[r];
        }
        int result = -1;
        if (owner < 0) {
            result = last_any;                            // t >= W after rounding: last token with weight
        } else if (owner == rank) {
            if (csum > 0.0 && cpre + incl > t) atomicMin(&sh.cand, tid);
            __syncthreads();
            const int c = sh.cand;
            if (c == 0x7fffffff) {
                if (tid == 0) sh.slot_i[1] = sh.last_pos; // crossing lost to rounding inside this CTA
            } else if (tid == c) {
                double running = cpre + excl;
                int tok = lastp;
                for (int k = k0; k < k1; ++k) {
                    running += weight(k, residual);
                    if (running > t) { tok = k; break; }
                }
                sh.slot_i[1] = tok;
            }
            __syncthreads();
            result = sh.slot_i[1];
        }
        // publish the owner's result to the cluster
        cluster_exchange(cluster, sh, cs, 0.0, 0.0, result, 0, xd0, xd1, xi0, xi1);
        token = owner < 0 ? result : xi0[owner];
        break;
    }

    if (rank == 0 && tid == 0) {
        P.accept_len[b] = n;
        P.next_token[b] = token;
        P.row_status[b] = status | ((residual0 && !(isfinite(Mb) && isfinite(Zb) && Zb > 0.0)) ? FSD_ROW_NONFINITE : 0);
    }
}

}  // namespace fsd
