// Device-side helpers shared by the verification kernels: logit loads with exact
// widening, fast base-2 exponent/logarithm, and fixed-order block reductions.
#pragma once

#include <cooperative_groups.h>
#include <cstdint>
#include <cuda_runtime.h>

#include "fsd_verify.h"

// Index and range checks of the debug build (-DFSD_DEBUG_CHECKS, see build.py): a failed check
// sets a bit in the workspace's debug word and the access goes ahead as in the release build --
// the checks are there to show that it never happens, on inputs of every shape the tests run.
// `word` is the third int of the workspace's flag block; null disables the check.
#ifdef FSD_DEBUG_CHECKS
#define FSD_CHECK(word, cond, code) do { if ((word) != nullptr && !(cond)) atomicOr((word), (code)); } while (0)
#else
#define FSD_CHECK(word, cond, code) do { } while (0)
#endif

namespace fsd {

namespace cg = cooperative_groups;

// bits of the debug word
constexpr int kChkItem = 1, kChkSlice = 2, kChkStage = 4, kChkTmem = 8, kChkRecord = 16, kChkRow = 32, kChkChunk = 64,
              kChkToken = 128, kChkPath = 256;

constexpr float  kLog2e  = 1.4426950408889634f;
constexpr double kLog2eD = 1.4426950408889634074;
constexpr double kLn2D   = 0.69314718055994530942;

// ---- logit storage -------------------------------------------------------------
template <int DT> struct Logit;
template <> struct Logit<FSD_F32> {
    using elem = float;
    static constexpr int kBytes = 4;
    static constexpr int kPerVec = 4;   // logits per 16-byte vector
};
template <> struct Logit<FSD_BF16> {
    using elem = uint16_t;
    static constexpr int kBytes = 2;
    static constexpr int kPerVec = 8;
};

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

template <int DT>
__device__ __forceinline__ float load_logit(const void* row, int k) {
    if constexpr (DT == FSD_BF16) {
        return __uint_as_float(static_cast<uint32_t>(__ldg(static_cast<const uint16_t*>(row) + k)) << 16);
    } else {
        return __ldg(static_cast<const float*>(row) + k);
    }
}

// one 16-byte vector of logits, widened to float
template <int DT>
__device__ __forceinline__ void unpack_vec(const uint4& v, float (&x)[Logit<DT>::kPerVec]) {
    if constexpr (DT == FSD_BF16) {
        x[0] = bf16_lo(v.x); x[1] = bf16_hi(v.x);
        x[2] = bf16_lo(v.y); x[3] = bf16_hi(v.y);
        x[4] = bf16_lo(v.z); x[5] = bf16_hi(v.z);
        x[6] = bf16_lo(v.w); x[7] = bf16_hi(v.w);
    } else {
        x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y);
        x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
    }
}

__device__ __forceinline__ uint4 ldg_vec(const void* row, int v) {
    return __ldg(static_cast<const uint4*>(row) + v);
}

// ---- special functions (one MUFU instruction each) ---------------------------
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float lg2(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// ---- warp / block reductions in a fixed order ----------------------------------
__device__ __forceinline__ double shfl_xor_d(double v, int m) { return __shfl_xor_sync(0xffffffffu, v, m); }

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) v += shfl_xor_d(v, m);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, m));
    return v;
}

// Sums N doubles over the block; every thread returns with the totals in v.
// `scratch` holds at least 32 * N doubles.  Ends with a barrier, so scratch may be reused.
template <int N>
__device__ __forceinline__ void block_sum(double (&v)[N], double* scratch) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
#pragma unroll
    for (int j = 0; j < N; ++j) v[j] = warp_sum(v[j]);
    if (lane == 0) {
#pragma unroll
        for (int j = 0; j < N; ++j) scratch[warp * N + j] = v[j];
    }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < N; ++j) {
        double s = 0.0;
        for (int w = 0; w < nwarps; ++w) s += scratch[w * N + j];
        v[j] = s;
    }
    __syncthreads();
}

template <int N>
__device__ __forceinline__ void block_max(float (&v)[N], float* scratch) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
#pragma unroll
    for (int j = 0; j < N; ++j) v[j] = warp_max(v[j]);
    if (lane == 0) {
#pragma unroll
        for (int j = 0; j < N; ++j) scratch[warp * N + j] = v[j];
    }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < N; ++j) {
        float s = scratch[j];
        for (int w = 1; w < nwarps; ++w) s = fmaxf(s, scratch[w * N + j]);
        v[j] = s;
    }
    __syncthreads();
}

// threshold test of Eq. 4 (NaN never passes)
__device__ __forceinline__ bool passes(float D, float T, int cmp) {
    return cmp == FSD_CMP_LE ? (D <= T) : (D < T);
}

}  // namespace fsd
