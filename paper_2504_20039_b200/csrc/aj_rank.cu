// Top-K rule, first step: per row of hidden states, the logit of that row's draft token,
//
//   thr[j] = sum_k h[j, k] * W[k, tok[j]]          fp32, one warp per row,
//
// which the projection kernels then use as the threshold when they count the vocabulary entries
// that outrank the draft token.  Row i of a sequence predicts draft token i; the last row (and, for
// a draft token outside the vocabulary, the row itself) gets +inf, which nothing outranks.  The
// kernel also zeroes the counters, so the cycle needs no separate clearing pass.
#include "aj_internal.cuh"

#include <cuda_bf16.h>

namespace aj {

namespace {

template <typename T> __device__ inline float as_float(T x);
template <> __device__ inline float as_float<float>(float x) { return x; }
template <> __device__ inline float as_float<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T>
__global__ void __launch_bounds__(128) rank_prepare_kernel(RankPrepArgs a) {
    const int lane = threadIdx.x & 31;
    const int j = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);  // row of hidden states
    const int M = a.B * a.R;
    if (j >= M) return;
    const int b = j / a.R, i = j % a.R;
    int tk = -1;
    if (i < a.K) {
        tk = a.draft_tok[(size_t)b * a.K + i];
        if (tk < 0 || tk >= a.V) tk = -1;  // an id outside the vocabulary is never accepted
    }
    float s = 0.0f;
    if (tk >= 0) {
        const T *h = reinterpret_cast<const T *>(a.h) + (size_t)j * a.d;
        const T *W = reinterpret_cast<const T *>(a.W);
        for (int k = lane; k < a.d; k += 32) {
            const float w = as_float(a.w_layout == 0 ? W[(size_t)tk * a.d + k] : W[(size_t)k * a.V + tk]);
            s = fmaf(as_float(h[k]), w, s);
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    }
    if (lane == 0) {
        a.thr[j] = tk >= 0 ? s : INFINITY;
        a.tok[j] = tk;
        a.cnt[j] = 0u;
    }
}

}  // namespace

cudaError_t launch_rank_prepare(const RankPrepArgs &a, cudaStream_t stream) {
    const int M = a.B * a.R;
    const int blocks = (M + 3) / 4;
    if (a.dtype == 0)
        rank_prepare_kernel<__nv_bfloat16><<<blocks, 128, 0, stream>>>(a);
    else
        rank_prepare_kernel<float><<<blocks, 128, 0, stream>>>(a);
    return cudaGetLastError();
}

}  // namespace aj
