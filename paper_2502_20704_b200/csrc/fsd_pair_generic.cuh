// Generic per-(row, position) kernel: one CTA per pair, three sweeps over the two
// logit rows (maximum; normalisers and the single-sweep sums; the sweep that needs
// both normalisers).  Works for any V and alignment; the vectorised instantiation is
// used when rows are 16-byte aligned.  The second and third sweeps re-read the rows
// through L2, so this kernel is the fallback for shapes the streaming kernel does not
// take, not the fast path.
#pragma once

#include "fsd_device.cuh"

namespace fsd {

struct PairParams {
    const void* target;        // [B, G+1, V]
    const void* draft;         // [B, G,   V]
    const int32_t* tokens;     // [B, G] or null
    const float* u_accept;     // [B, G] or null
    const int32_t* parent;     // [B, G] (tree) or null (chain)
    int B, G, V;
    int div, mode, cmp;
    float T;
    float* divergence;         // [B, G]
    int32_t* item_bits;        // [B, G] accept bit per pair
    int32_t* item_status;      // [B, G] FSD_ROW_* flags per pair
    int* debug_word;           // debug build: where failed range checks are recorded (may be null)
};

// Final scalar work for one pair, done by one thread in double precision.
//   Ma, Mb   row maxima;  ca, cb  the float offsets -M*log2(e) every exponent used
//   Za, Zb   sum_k 2^(y_k), y_k = fma(logit_k, log2e, c)
//   Sa, Sb   sum_k 2^(y_k) * y_k                        (entropy terms)
//   K        sum_k 2^(ya_k) * (ya_k - yb_k)             (KL, Appendix C.1)
//   X        JS: sum_k s_k log2 s_k with s = p + q;  TV: sum_k |p_k - q_k|
// Returns the divergence in nats (NaN when a row is not a valid distribution).
// The variant with lnZa, lnZb takes the two logarithms from the caller (computed by two lanes at once).
__device__ inline double combine_divergence(int div, double Za, double Zb, double lnZa, double lnZb, double Sa, double Sb, double K, double X) {
    double D;
    if (div == FSD_DIV_KL) {
        D = kLn2D * K / Za - lnZa + lnZb;
    } else if (div == FSD_DIV_JS) {
        // sum p ln p = ln2 * Sa/Za - ln Za (the offset error in c cancels between the two terms);
        // sum m ln m with m = s/2 and sum s = 2:  (ln2/2) * X - ln2
        const double Pp = kLn2D * Sa / Za - lnZa, Pq = kLn2D * Sb / Zb - lnZb;
        D = 0.5 * (Pp + Pq) - (0.5 * kLn2D * X - kLn2D);
    } else {
        D = 0.5 * X;
    }
    return D < 0.0 ? 0.0 : D;   // NaN stays NaN
}
__device__ inline double combine_divergence(int div, double Za, double Zb, double Sa, double Sb, double K, double X) {
    return combine_divergence(div, Za, Zb, log(Za), log(Zb), Sa, Sb, K, X);
}

// ln P(x) of one token from its logit and the row's normaliser, in double.
__device__ inline double log_prob(float logit, float M, float c, double Z) {
    // Z was accumulated with exponents offset by c instead of the exact -M*log2e
    const double delta = static_cast<double>(c) + static_cast<double>(M) * kLog2eD;
    return (static_cast<double>(logit) - static_cast<double>(M)) - (log(Z) - delta * kLn2D);
}

// Acceptance bit of one pair from its divergence and (for SD / rFSD) the ratio test.
__device__ inline int accept_bit(int mode, int cmp, float T, const int32_t* tokens, const float* u_accept, int V,
                                 int item, bool finite, float D, const void* a_row, const void* b_row, int dt,
                                 float Ma, float ca, double Za, float Mb, float cb, double Zb) {
    bool div_ok = finite && passes(D, T, cmp);
    if (mode == FSD_MODE_FSD) return div_ok;
    bool ratio_ok = false;
    if (finite) {
        const int x = tokens[item];
        if (x >= 0 && x < V) {
            const float ax = dt == FSD_BF16 ? load_logit<FSD_BF16>(a_row, x) : load_logit<FSD_F32>(a_row, x);
            const float bx = dt == FSD_BF16 ? load_logit<FSD_BF16>(b_row, x) : load_logit<FSD_F32>(b_row, x);
            double pacc;                                                    // Eq. 1
            if (bx == -INFINITY) {
                pacc = (ax != -INFINITY) ? 1.0 : 0.0;
            } else {
                pacc = exp(log_prob(ax, Ma, ca, Za) - log_prob(bx, Mb, cb, Zb));
                pacc = pacc < 1.0 ? pacc : 1.0;
            }
            ratio_ok = static_cast<double>(u_accept[item]) < pacc;          // Eq. 2
        }
    }
    return mode == FSD_MODE_SD ? ratio_ok : (div_ok || ratio_ok);            // Eq. 6
}

// What the three sweeps leave for the pair's final scalar work.
struct GenericSums {
    float Ma, Mb, ca, cb;
    double Za, Zb, Sa, Sb, K, X;
    bool finite;
};

// The three sweeps over one pair of rows by the whole CTA; every thread returns the same sums.
// `red_d` holds at least 32 * 5 doubles, `red_f` at least 32 * 2 floats.
template <int DT, bool VEC>
__device__ inline GenericSums generic_pair_sums(const char* a_row, const char* b_row, int V, int div, double* red_d, float* red_f) {
    constexpr int EPV = Logit<DT>::kPerVec;
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int nvec = V / EPV;
    GenericSums r;

    // sweep 1: row maxima (exact)
    float mx[2] = {-INFINITY, -INFINITY};
    if constexpr (VEC) {
        for (int v = tid; v < nvec; v += nthr) {
            float xa[EPV], xb[EPV];
            unpack_vec<DT>(ldg_vec(a_row, v), xa);
            unpack_vec<DT>(ldg_vec(b_row, v), xb);
#pragma unroll
            for (int e = 0; e < EPV; ++e) { mx[0] = fmaxf(mx[0], xa[e]); mx[1] = fmaxf(mx[1], xb[e]); }
        }
    } else {
        for (int k = tid; k < V; k += nthr) {
            mx[0] = fmaxf(mx[0], load_logit<DT>(a_row, k));
            mx[1] = fmaxf(mx[1], load_logit<DT>(b_row, k));
        }
    }
    block_max<2>(mx, red_f);
    const float Ma = mx[0], Mb = mx[1];
    const float ca = -Ma * kLog2e, cb = -Mb * kLog2e;

    // sweep 2: normalisers, entropy sums, KL sum
    float za = 0.f, zb = 0.f, sa = 0.f, sb = 0.f, kk = 0.f;
    auto term2 = [&](float a, float bq) {
        const float ya = fmaf(a, kLog2e, ca), yb = fmaf(bq, kLog2e, cb);
        const float ea = ex2(ya), eb = ex2(yb);
        za += ea;
        zb += eb;
        sa += ea > 0.f ? ea * ya : 0.f;
        sb += eb > 0.f ? eb * yb : 0.f;
        kk += ea > 0.f ? ea * (ya - yb) : 0.f;
    };
    if constexpr (VEC) {
        for (int v = tid; v < nvec; v += nthr) {
            float xa[EPV], xb[EPV];
            unpack_vec<DT>(ldg_vec(a_row, v), xa);
            unpack_vec<DT>(ldg_vec(b_row, v), xb);
#pragma unroll
            for (int e = 0; e < EPV; ++e) term2(xa[e], xb[e]);
        }
    } else {
        for (int k = tid; k < V; k += nthr) term2(load_logit<DT>(a_row, k), load_logit<DT>(b_row, k));
    }
    double s2[5] = {za, zb, sa, sb, kk};
    block_sum<5>(s2, red_d);
    const double Za = s2[0], Zb = s2[1];
    const bool finite = isfinite(Ma) && isfinite(Mb) && isfinite(Za) && isfinite(Zb) && Za > 0.0 && Zb > 0.0;

    // sweep 3: the sums that need both normalisers (JS: s log2 s; TV: |p - q|)
    double X = 0.0;
    if (finite && div != FSD_DIV_KL) {
        const float ia = static_cast<float>(1.0 / Za), ib = static_cast<float>(1.0 / Zb);
        const bool js = div == FSD_DIV_JS;
        float acc = 0.f;
        auto term3 = [&](float a, float bq) {
            // explicit roundings: a fused p - q would keep one product unrounded and make TV(p, p) != 0
            const float p = __fmul_rn(ex2(fmaf(a, kLog2e, ca)), ia), q = __fmul_rn(ex2(fmaf(bq, kLog2e, cb)), ib);
            if (js) {
                // below the normal range lg2 (which flushes its operand) would return -inf;
                // such a term is smaller than 1e-35 and left out
                const float s = p + q;
                acc += s >= 1.17549435e-38f ? s * lg2(s) : 0.f;
            } else {
                acc += fabsf(p - q);
            }
        };
        if constexpr (VEC) {
            for (int v = tid; v < nvec; v += nthr) {
                float xa[EPV], xb[EPV];
                unpack_vec<DT>(ldg_vec(a_row, v), xa);
                unpack_vec<DT>(ldg_vec(b_row, v), xb);
#pragma unroll
                for (int e = 0; e < EPV; ++e) term3(xa[e], xb[e]);
            }
        } else {
            for (int k = tid; k < V; k += nthr) term3(load_logit<DT>(a_row, k), load_logit<DT>(b_row, k));
        }
        double s3[1] = {acc};
        block_sum<1>(s3, red_d);
        X = s3[0];
    }
    r.Ma = Ma; r.Mb = Mb; r.ca = ca; r.cb = cb;
    r.Za = Za; r.Zb = Zb; r.Sa = s2[2]; r.Sb = s2[3]; r.K = s2[4]; r.X = X;
    r.finite = finite;
    return r;
}

template <int DT, bool VEC>
__global__ void __launch_bounds__(512) fsd_pair_generic_kernel(PairParams P) {
    __shared__ double red_d[32 * 5];
    __shared__ float red_f[32 * 2];

    const int item = blockIdx.x;
    const int b = item / P.G, i = item - b * P.G;
    FSD_CHECK(P.debug_word, b < P.B, kChkItem);
    int trow = i;
    if (P.parent != nullptr) {
        const int par = P.parent[item];
        if (par < -1 || par >= i) {
            if (threadIdx.x == 0) {
                P.divergence[item] = __int_as_float(0x7fc00000);
                P.item_bits[item] = 0;
                P.item_status[item] = FSD_ROW_BADTREE;
            }
            return;
        }
        trow = par + 1;
    }
    const size_t rb = static_cast<size_t>(P.V) * Logit<DT>::kBytes;
    const char* a_row = static_cast<const char*>(P.target) + (static_cast<size_t>(b) * (P.G + 1) + trow) * rb;
    const char* b_row = static_cast<const char*>(P.draft) + (static_cast<size_t>(b) * P.G + i) * rb;
    const GenericSums r = generic_pair_sums<DT, VEC>(a_row, b_row, P.V, P.div, red_d, red_f);

    if (threadIdx.x == 0) {
        float D = __int_as_float(0x7fc00000);
        if (r.finite) D = static_cast<float>(combine_divergence(P.div, r.Za, r.Zb, r.Sa, r.Sb, r.K, r.X));
        P.divergence[item] = D;
        P.item_bits[item] = accept_bit(P.mode, P.cmp, P.T, P.tokens, P.u_accept, P.V, item, r.finite, D, a_row, b_row, DT,
                                       r.Ma, r.ca, r.Za, r.Mb, r.cb, r.Zb);
        P.item_status[item] = r.finite ? 0 : FSD_ROW_NONFINITE;
    }
}

}  // namespace fsd
