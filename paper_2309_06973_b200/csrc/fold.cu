// Module 1, the Model Pre-Processor: fold every BatchNorm into the convolution in front of it
// (Section III-D), applied here to a rebuilt (compacted) variant in its destination arena:
//   s_o   = gamma_o / sqrt(var_o + eps)
//   W_f[o] = W[o] * s_o                       (in place)
//   b_f[o] = beta_o + (bias_o - mean_o) * s_o  (bias_o = 0 without a bias)
// Two launches: k_fold_prepare (a block per BatchNorm) writes s into the arena slot of gamma and b_f into the
// slot of beta (the BatchNorm vectors have no further use once folded) and lists the 16 KB tiles of the rebuilt
// tensor in front of it; k_fold_scale multiplies the weights of the listed tiles, four 16-byte vectors per thread.  Arithmetic is fp32; bf16 weights are widened, scaled and
// rounded to nearest even.
#include <algorithm>

#include "dnns_internal.cuh"

namespace dnns {

namespace {

constexpr int kThreads = 256;

struct FoldArgs {
    char* arena;
    const uint64_t* offsets;  // [n_items] byte offsets of the rebuilt items
    const int32_t* shapes;    // [n_tensors][2] rebuilt (O', I')
};

template <int DT>
__global__ void __launch_bounds__(kThreads) k_fold_prepare(Tables tb, FoldArgs fa, uint32_t* __restrict__ job_count,
                                                           FoldJob* __restrict__ jobs) {
    constexpr uint32_t kTileElems = kTileBytes / Elem<DT>::kBytes;
    constexpr int kBatch = 4;  // channels per thread whose loads are issued together
    __shared__ uint32_t s_first;
    const uint32_t b = blockIdx.x;
    const BnDesc bn = tb.bns[b];
    const int32_t On = fa.shapes[2 * bn.tensor];
    const uint32_t Ln = (uint32_t)fa.shapes[2 * bn.tensor + 1] * tb.tensors[bn.tensor].KK;
    const uint32_t base = tb.n_tensors + 4 * b;
    float* gamma = reinterpret_cast<float*>(fa.arena + fa.offsets[base]);
    float* beta = reinterpret_cast<float*>(fa.arena + fa.offsets[base + 1]);
    const float* mean = reinterpret_cast<const float*>(fa.arena + fa.offsets[base + 2]);
    const float* var = reinterpret_cast<const float*>(fa.arena + fa.offsets[base + 3]);
    const float* bias = bn.bias_item >= 0 ? reinterpret_cast<const float*>(fa.arena + fa.offsets[bn.bias_item]) : nullptr;
    char* w = fa.arena + fa.offsets[bn.tensor];
    // the tiles of the rebuilt tensor join the list the second kernel works through
    const uint32_t total = (uint32_t)On * Ln, n_tiles = (total + kTileElems - 1) / kTileElems;
    if (threadIdx.x == 0) s_first = n_tiles ? atomicAdd(job_count, n_tiles) : 0u;
    for (int a0 = threadIdx.x; a0 < On; a0 += kThreads * kBatch) {
        float g[kBatch], vr[kBatch], mn[kBatch], be[kBatch], bi[kBatch];
#pragma unroll
        for (int t = 0; t < kBatch; ++t) {
            const int a = a0 + t * kThreads;
            const bool in = a < On;
            g[t] = in ? gamma[a] : 0.0f, vr[t] = in ? var[a] : 1.0f, mn[t] = in ? mean[a] : 0.0f, be[t] = in ? beta[a] : 0.0f;
            bi[t] = in && bias ? bias[a] : 0.0f;
        }
#pragma unroll
        for (int t = 0; t < kBatch; ++t) {
            const int a = a0 + t * kThreads;
            if (a >= On) continue;
            const float s = g[t] / sqrtf(vr[t] + bn.eps);
            gamma[a] = s;
            beta[a] = fmaf(bi[t] - mn[t], s, be[t]);
        }
    }
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < n_tiles; i += kThreads)
        jobs[s_first + i] = FoldJob{w, gamma, Ln, total, i * kTileElems, 0u};
}

__device__ __forceinline__ uint32_t bf16_round(float x) {
    const uint32_t u = __float_as_uint(x);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (u >> 16) | 0x40u;  // NaN stays NaN
    return (u + 0x7FFFu + ((u >> 16) & 1u)) >> 16;
}

// W[o] *= s_o over the rebuilt tensors, a block per listed 16 KB tile and round.  A thread holds four 16-byte
// vectors of a tile; the row of a vector is one division, and a vector inside one row (nearly all of them) is
// scaled by one factor.
template <int DT>
__device__ __forceinline__ uint32_t scaled_word(uint32_t x, float s_lo, float s_hi) {
    if (DT == DNNS_F32) return __float_as_uint(__uint_as_float(x) * s_lo);
    const float a = __uint_as_float(x << 16) * s_lo, b = __uint_as_float(x & 0xFFFF0000u) * s_hi;
    return bf16_round(a) | (bf16_round(b) << 16);
}

template <int DT>
__global__ void __launch_bounds__(kTileThreads, 4) k_fold_scale(const uint32_t* __restrict__ job_count, const FoldJob* __restrict__ jobs) {
    constexpr uint32_t VE = Elem<DT>::kPerVec;
    const uint32_t n_jobs = *job_count;
    for (uint32_t i = blockIdx.x; i < n_jobs; i += gridDim.x) {
        const FoldJob job = jobs[i];
        const uint32_t Ln = job.Ln, total = job.total, e0 = job.e0, On = total / Ln;
        char* w = job.w;
        const float* __restrict__ scale = job.scale;
        uint4 v[kVecPerThread];
        uint32_t f[kVecPerThread];
#pragma unroll
        for (int u = 0; u < kVecPerThread; ++u) {
            f[u] = e0 + (u * kTileThreads + threadIdx.x) * VE;
            if (f[u] + VE <= total) v[u] = *reinterpret_cast<const uint4*>(w + (size_t)f[u] * Elem<DT>::kBytes);
        }
#pragma unroll
        for (int u = 0; u < kVecPerThread; ++u) {
            if (f[u] >= total) continue;
            uint32_t a = f[u] / Ln, rem = f[u] - a * Ln;
            if (f[u] + VE <= total) {
                uint32_t x[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
                if (rem + VE <= Ln) {
                    const float s = scale[a];
#pragma unroll
                    for (int q = 0; q < 4; ++q) x[q] = scaled_word<DT>(x[q], s, s);
                } else {
                    // the vector crosses into the next row (or rows, when rows are shorter than a vector)
                    float se[VE];
#pragma unroll
                    for (uint32_t e = 0; e < VE; ++e) {
                        se[e] = scale[a];
                        if (++rem == Ln) rem = 0, ++a;
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q) x[q] = DT == DNNS_F32 ? scaled_word<DT>(x[q], se[q], se[q]) : scaled_word<DT>(x[q], se[(2 * q) % VE], se[(2 * q + 1) % VE]);
                }
                *reinterpret_cast<uint4*>(w + (size_t)f[u] * Elem<DT>::kBytes) = make_uint4(x[0], x[1], x[2], x[3]);
            } else {
                float s = scale[a];
                for (uint32_t e = 0; f[u] + e < total; ++e) {
                    if (DT == DNNS_F32) {
                        float* p = reinterpret_cast<float*>(w) + f[u] + e;
                        *p = *p * s;
                    } else {
                        uint16_t* p = reinterpret_cast<uint16_t*>(w) + f[u] + e;
                        *p = (uint16_t)bf16_round(__uint_as_float((uint32_t)*p << 16) * s);
                    }
                    if (++rem == Ln) {
                        rem = 0;
                        ++a;
                        if (a < On) s = scale[a];
                    }
                }
            }
        }
    }
}

}  // namespace

int launch_fold(const Tables& tb, void* arena, const uint64_t* offsets, const int32_t* shapes, uint32_t* job_count,
                FoldJob* jobs, int n_sm, cudaStream_t st) {
    if (tb.n_bn == 0) return 0;
    const FoldArgs fa{static_cast<char*>(arena), offsets, shapes};
    if (cudaMemsetAsync(job_count, 0, sizeof(uint32_t), st) != cudaSuccess) return -1;
    const int grid = (int)std::min<uint32_t>(tb.n_tiles, (uint32_t)n_sm * 8u);
    if (tb.dtype == DNNS_F32) {
        { ScopedKernel t("k_fold_prepare", st); k_fold_prepare<DNNS_F32><<<tb.n_bn, kThreads, 0, st>>>(tb, fa, job_count, jobs); }
        { ScopedKernel t("k_fold_scale", st); k_fold_scale<DNNS_F32><<<grid, kTileThreads, 0, st>>>(job_count, jobs); }
    } else {
        { ScopedKernel t("k_fold_prepare", st); k_fold_prepare<DNNS_BF16><<<tb.n_bn, kThreads, 0, st>>>(tb, fa, job_count, jobs); }
        { ScopedKernel t("k_fold_scale", st); k_fold_scale<DNNS_BF16><<<grid, kTileThreads, 0, st>>>(job_count, jobs); }
    }
    return cudaGetLastError() == cudaSuccess ? 2 : -1;
}

}  // namespace dnns
