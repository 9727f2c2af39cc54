// Module 1, the Model Pre-Processor: fold every BatchNorm into the convolution in front of it
// (Section III-D), applied here to a rebuilt (compacted) variant in its destination arena:
//   s_o   = gamma_o / sqrt(var_o + eps)
//   W_f[o] = W[o] * s_o                       (in place)
//   b_f[o] = beta_o + (bias_o - mean_o) * s_o  (bias_o = 0 without a bias)
// Two launches: k_fold_prepare writes s into the arena slot of gamma and b_f into the slot of
// beta (the BatchNorm vectors have no further use once folded); k_fold_scale multiplies the
// weights, 16 bytes per thread and step.  Arithmetic is fp32; bf16 weights are widened, scaled and
// rounded to nearest even.
#include "dnns_internal.cuh"

namespace dnns {

namespace {

constexpr int kThreads = 256;

struct FoldArgs {
    char* arena;
    const uint64_t* offsets;  // [n_items] byte offsets of the rebuilt items
    const int32_t* shapes;    // [n_tensors][2] rebuilt (O', I')
};

__global__ void __launch_bounds__(kThreads) k_fold_prepare(Tables tb, FoldArgs fa) {
    const uint32_t b = blockIdx.x;
    const BnDesc bn = tb.bns[b];
    const int32_t On = fa.shapes[2 * bn.tensor];
    const uint32_t base = tb.n_tensors + 4 * b;
    float* gamma = reinterpret_cast<float*>(fa.arena + fa.offsets[base]);
    float* beta = reinterpret_cast<float*>(fa.arena + fa.offsets[base + 1]);
    const float* mean = reinterpret_cast<const float*>(fa.arena + fa.offsets[base + 2]);
    const float* var = reinterpret_cast<const float*>(fa.arena + fa.offsets[base + 3]);
    const float* bias = bn.bias_item >= 0 ? reinterpret_cast<const float*>(fa.arena + fa.offsets[bn.bias_item]) : nullptr;
    for (int a = threadIdx.x; a < On; a += kThreads) {
        const float s = gamma[a] / sqrtf(var[a] + bn.eps);
        const float shift = (bias ? bias[a] : 0.0f) - mean[a];
        gamma[a] = s;
        beta[a] = fmaf(shift, s, beta[a]);
    }
}

__device__ __forceinline__ uint32_t bf16_round(float x) {
    const uint32_t u = __float_as_uint(x);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (u >> 16) | 0x40u;  // NaN stays NaN
    return (u + 0x7FFFu + ((u >> 16) & 1u)) >> 16;
}

template <int DT>
__global__ void __launch_bounds__(kThreads) k_fold_scale(Tables tb, FoldArgs fa) {
    constexpr uint32_t VE = Elem<DT>::kPerVec;
    const uint32_t b = blockIdx.y;
    const BnDesc bn = tb.bns[b];
    const TensorDesc& d = tb.tensors[bn.tensor];
    const uint32_t On = fa.shapes[2 * bn.tensor], Ln = (uint32_t)fa.shapes[2 * bn.tensor + 1] * d.KK;
    const uint32_t total = On * Ln;
    if (total == 0) return;
    char* w = fa.arena + fa.offsets[bn.tensor];
    const float* scale = reinterpret_cast<const float*>(fa.arena + fa.offsets[tb.n_tensors + 4 * b]);
    for (uint32_t f = (blockIdx.x * kThreads + threadIdx.x) * VE; f < total; f += gridDim.x * kThreads * VE) {
        uint32_t a = f / Ln, rem = f - a * Ln;
        float s = scale[a];
        if (f + VE <= total) {
            uint4 v = *reinterpret_cast<uint4*>(w + (size_t)f * Elem<DT>::kBytes);
            uint32_t x[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (uint32_t e = 0; e < VE; ++e) {
                if (DT == DNNS_F32) {
                    x[e] = __float_as_uint(__uint_as_float(x[e]) * s);
                } else {
                    const uint32_t sh = 16 * (e & 1);
                    const float y = __uint_as_float(((x[e >> 1] >> sh) & 0xFFFFu) << 16) * s;
                    x[e >> 1] = (x[e >> 1] & ~(0xFFFFu << sh)) | (bf16_round(y) << sh);
                }
                if (++rem == Ln) {
                    rem = 0;
                    ++a;
                    if (a < On) s = scale[a];
                }
            }
            *reinterpret_cast<uint4*>(w + (size_t)f * Elem<DT>::kBytes) = make_uint4(x[0], x[1], x[2], x[3]);
        } else {
            for (uint32_t e = 0; f + e < total; ++e) {
                if (DT == DNNS_F32) {
                    float* p = reinterpret_cast<float*>(w) + f + e;
                    *p = *p * s;
                } else {
                    uint16_t* p = reinterpret_cast<uint16_t*>(w) + f + e;
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

}  // namespace

int launch_fold(const Tables& tb, void* arena, const uint64_t* offsets, const int32_t* shapes, cudaStream_t st) {
    if (tb.n_bn == 0) return 0;
    const FoldArgs fa{static_cast<char*>(arena), offsets, shapes};
    k_fold_prepare<<<tb.n_bn, kThreads, 0, st>>>(tb, fa);
    const dim3 grid(128, tb.n_bn);  // tensors differ a lot in size: many slices keep the large ones spread out
    if (tb.dtype == DNNS_F32) k_fold_scale<DNNS_F32><<<grid, kThreads, 0, st>>>(tb, fa);
    else k_fold_scale<DNNS_BF16><<<grid, kThreads, 0, st>>>(tb, fa);
    return cudaGetLastError() == cudaSuccess ? 2 : -1;
}

}  // namespace dnns
