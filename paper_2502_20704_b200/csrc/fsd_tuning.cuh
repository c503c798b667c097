// Threshold tuning on the divergences a verification call returns (Section "Selecting T": the
// threshold is tuned on a small development set by looking at the speed each candidate gives;
// Discussion: the FSD decision is deterministic given the divergences, so token-level labels can
// be dumped).  The accepted length of a row at threshold T is the index of its first position
// that fails D cmp T (NaN never passes); the speed proxy is the mean accepted length.
//
// With P[b, k] = max(D[b, 0..k]) (NaN once a NaN has been seen) the accepted length of row b is
// the number of k with P[b, k] cmp T, so
//   * a sweep needs one pass per candidate threshold, and
//   * the smallest T that reaches a wanted mean accepted length is an order statistic of the
//     multiset {P[b, k]}: the ceil(target * B)-th smallest value v (T = v under <=, the next
//     float above v under <).  It is found by a most-significant-byte-first radix selection on
//     the float bit patterns (monotone for non-negative floats), four passes of 256 bins.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

#include "fsd_device.cuh"

namespace fsd {

constexpr int kTuneThreads = 1024;
constexpr uint32_t kKeyInf = 0x7f800000u;     // keys above this are NaN (or negative): never accepted

// Sortable key of a prefix maximum: divergences are >= 0, so the bit pattern orders them; -0 and
// negative inputs count as 0, NaN as "never".
__device__ __forceinline__ uint32_t tune_key(float p) {
    if (p != p) return 0xffffffffu;
    return p <= 0.f ? 0u : __float_as_uint(p);
}

// ---- sweep: one CTA per candidate threshold -------------------------------------------------
__global__ void __launch_bounds__(256) fsd_threshold_sweep_kernel(const float* __restrict__ D, int B, int G,
                                                                  const float* __restrict__ thresholds, int cmp,
                                                                  float* __restrict__ mean_len, float* __restrict__ frac) {
    __shared__ unsigned long long part[8];
    const float T = thresholds[blockIdx.x];
    unsigned long long total = 0;
    for (int b = threadIdx.x; b < B; b += blockDim.x) {
        const float* row = D + static_cast<size_t>(b) * G;
        int n = 0;
        while (n < G && passes(row[n], T, cmp)) ++n;
        total += static_cast<unsigned long long>(n);
    }
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) total += __shfl_xor_sync(0xffffffffu, total, m);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = total;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long t = 0;
        for (int w = 0; w < static_cast<int>(blockDim.x >> 5); ++w) t += part[w];
        mean_len[blockIdx.x] = static_cast<float>(static_cast<double>(t) / static_cast<double>(B));
        frac[blockIdx.x] = static_cast<float>(static_cast<double>(t) / (static_cast<double>(B) * static_cast<double>(G)));
    }
}

// ---- calibration: one CTA, radix selection over the prefix maxima ----------------------------
// Calls f(key, valid) for every prefix maximum of the rows this thread owns.  Every thread of the
// CTA makes the same number of calls (rows past the end come with valid = false), so f may use
// full-warp collectives.
template <typename F>
__device__ __forceinline__ void for_prefix_maxima(const float* __restrict__ D, int B, int G, F f) {
    for (int b0 = 0; b0 < B; b0 += blockDim.x) {
        const int b = b0 + threadIdx.x;
        const bool valid = b < B;
        const float* row = D + static_cast<size_t>(valid ? b : 0) * G;
        float p = 0.f;
        bool nan = false;
        for (int k = 0; k < G; ++k) {
            const float d = row[k];
            nan = nan || d != d;
            p = fmaxf(p, d);
            f(nan ? 0xffffffffu : tune_key(p), valid);
        }
    }
}

__global__ void __launch_bounds__(kTuneThreads) fsd_calibrate_kernel(const float* __restrict__ D, int B, int G, float target,
                                                                     int cmp, float* __restrict__ T_out,
                                                                     float* __restrict__ achieved_out) {
    __shared__ unsigned int hist[256];         // B * positions fits an int
    __shared__ unsigned long long s_total;
    __shared__ unsigned long long s_rank;      // rank still to be found inside the selected bin (1-based)
    __shared__ uint32_t s_prefix;              // the key's bytes selected so far
    __shared__ int s_found;

    // positions that must be accepted: ceil(target * B), within [0, B * G]
    const double want = ceil(static_cast<double>(target) * static_cast<double>(B));
    const double most = static_cast<double>(B) * static_cast<double>(G);
    const unsigned long long need = want <= 0.0 ? 0ull : static_cast<unsigned long long>(want < most ? want : most);
    // (the host refuses negative and NaN targets)

    if (threadIdx.x == 0) { s_rank = need; s_prefix = 0; s_found = 1; }
    __syncthreads();

    if (need > 0) {
        for (int byte = 3; byte >= 0; --byte) {
            for (int i = threadIdx.x; i < 256; i += blockDim.x) hist[i] = 0;
            __syncthreads();
            const uint32_t prefix = s_prefix;
            const uint32_t high_mask = byte == 3 ? 0u : (0xffffffffu << (8 * (byte + 1)));
            for_prefix_maxima(D, B, G, [&](uint32_t key, bool valid) {
                // lanes that hit the same bin add once (keys cluster in a few bins: plain atomics would serialise)
                const bool in = valid && key <= kKeyInf && (key & high_mask) == prefix;
                const uint32_t bin = in ? ((key >> (8 * byte)) & 255u) : 256u;
                const unsigned peers = __match_any_sync(0xffffffffu, bin);
                if (in && (threadIdx.x & 31) == __ffs(peers) - 1) atomicAdd(&hist[bin], static_cast<unsigned int>(__popc(peers)));
            });
            __syncthreads();
            if (threadIdx.x == 0) {
                unsigned long long rank = s_rank, run = 0;
                int bin = -1;
                for (int i = 0; i < 256; ++i) {
                    if (run + hist[i] >= rank) { bin = i; break; }
                    run += hist[i];
                }
                if (bin < 0) {
                    s_found = 0;                        // fewer acceptable positions than needed
                } else {
                    s_rank = rank - run;
                    s_prefix = prefix | (static_cast<uint32_t>(bin) << (8 * byte));
                }
            }
            __syncthreads();
            if (!s_found) break;
        }
    }

    // the threshold, then the mean accepted length it gives (one more pass)
    float T;
    if (need == 0) {
        T = 0.f;
    } else if (!s_found) {
        T = INFINITY;
    } else {
        const float v = __uint_as_float(s_prefix);
        T = cmp == FSD_CMP_LE ? v : (v == INFINITY ? INFINITY : __uint_as_float(s_prefix + 1u));   // next float above v
    }
    __syncthreads();
    if (threadIdx.x == 0) s_total = 0;
    __syncthreads();
    unsigned long long mine = 0;
    for_prefix_maxima(D, B, G, [&](uint32_t key, bool valid) {
        if (valid && key <= kKeyInf && passes(__uint_as_float(key), T, cmp)) ++mine;
    });
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, m);
    if ((threadIdx.x & 31) == 0 && mine) atomicAdd(&s_total, mine);
    __syncthreads();
    if (threadIdx.x == 0) {
        *T_out = T;
        *achieved_out = static_cast<float>(static_cast<double>(s_total) / static_cast<double>(B));
    }
}

// ---- labels: each position on its own ---------------------------------------------------------
__global__ void fsd_accept_labels_kernel(const float* __restrict__ D, size_t n, float T, int cmp, uint8_t* __restrict__ labels) {
    const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
    for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += stride)
        labels[i] = passes(D[i], T, cmp) ? 1 : 0;
}

}  // namespace fsd
