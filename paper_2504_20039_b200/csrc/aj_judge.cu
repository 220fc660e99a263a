// Mismatch mask, judge at mismatches, accepted-prefix scan: one block per sequence.
//
//   y[j]    = index stored in the row's packed key                    (greedy target tokens)
//   mis[i]  = draft_tok[i] != y[i]
//   p[i]    = sigmoid(b + w . [h_draft[i+1] ; h_target[i+1]])         only where mis[i]
//   stop    = first i with mis[i] and not (p[i] < tau)                ballot + ffs over the window
//   accept_len = stop (K if none), next_tok = y[accept_len]
//
// A warp takes one mismatching position at a time: 128-bit loads of the features, fp32
// accumulate, shuffle reduction.
#include "aj_internal.cuh"

#include <cuda_bf16.h>

namespace aj {

namespace {

__device__ inline float dot8_bf16(const uint4 &x, const float4 &w0, const float4 &w1) {
    const __nv_bfloat162 *p = reinterpret_cast<const __nv_bfloat162 *>(&x);
    const float2 a = __bfloat1622float2(p[0]), b = __bfloat1622float2(p[1]);
    const float2 c = __bfloat1622float2(p[2]), e = __bfloat1622float2(p[3]);
    float s = a.x * w0.x;
    s = fmaf(a.y, w0.y, s);
    s = fmaf(b.x, w0.z, s);
    s = fmaf(b.y, w0.w, s);
    s = fmaf(c.x, w1.x, s);
    s = fmaf(c.y, w1.y, s);
    s = fmaf(e.x, w1.z, s);
    s = fmaf(e.y, w1.w, s);
    return s;
}

// partial dot product of one feature block held by this lane
__device__ inline float block_dot(const void *x, const float *w, int n, int dtype, int lane) {
    float s = 0.0f;
    if (x == nullptr || n <= 0) return s;
    if (dtype == 0) {
        const bool vec = (n % 8 == 0) && ((reinterpret_cast<uintptr_t>(x) & 15) == 0) &&
                         ((reinterpret_cast<uintptr_t>(w) & 15) == 0);
        if (vec) {
            const uint4 *xv = reinterpret_cast<const uint4 *>(x);
            const float4 *wv = reinterpret_cast<const float4 *>(w);
            for (int c = lane; c < n / 8; c += 32) s += dot8_bf16(__ldg(xv + c), __ldg(wv + 2 * c), __ldg(wv + 2 * c + 1));
        } else {
            const __nv_bfloat16 *xs = reinterpret_cast<const __nv_bfloat16 *>(x);
            for (int f = lane; f < n; f += 32) s = fmaf(__bfloat162float(xs[f]), w[f], s);
        }
    } else {
        const bool vec = (n % 4 == 0) && ((reinterpret_cast<uintptr_t>(x) & 15) == 0) &&
                         ((reinterpret_cast<uintptr_t>(w) & 15) == 0);
        if (vec) {
            const float4 *xv = reinterpret_cast<const float4 *>(x);
            const float4 *wv = reinterpret_cast<const float4 *>(w);
            for (int c = lane; c < n / 4; c += 32) {
                const float4 a = __ldg(xv + c), b = __ldg(wv + c);
                s = fmaf(a.x, b.x, s);
                s = fmaf(a.y, b.y, s);
                s = fmaf(a.z, b.z, s);
                s = fmaf(a.w, b.w, s);
            }
        } else {
            const float *xs = reinterpret_cast<const float *>(x);
            for (int f = lane; f < n; f += 32) s = fmaf(xs[f], w[f], s);
        }
    }
    return s;
}

__global__ void __launch_bounds__(512) judge_scan_kernel(JudgeArgs a) {
    extern __shared__ int smem[];
    int *y_s = smem;               // [K+1]
    int *rej_s = smem + a.K + 1;   // [K]
    const int b = blockIdx.x;
    const int K = a.K, R = a.K + 1;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const size_t esz = a.dtype == 0 ? 2 : 4;

    for (int j = threadIdx.x; j < R; j += blockDim.x) {
        const unsigned long long key = a.keys[(size_t)b * R + j];
        const int y = key_index(key);
        y_s[j] = y;
        if (a.target_tok) a.target_tok[(size_t)b * R + j] = y;
        if (a.top1_val) a.top1_val[(size_t)b * R + j] = key_value(key);
    }
    __syncthreads();

    for (int i = warp; i < K; i += nwarps) {
        const bool mis = a.draft_tok[(size_t)b * K + i] != y_s[i];  // warp-uniform
        float p = __int_as_float(0x7fc00000);                      // NaN where the judge is not consulted
        int rej = 0;
        if (mis) {
            const size_t row = (size_t)b * R + (i + 1);  // the hidden states that encode draft token i
            const char *xd = a.h_draft ? reinterpret_cast<const char *>(a.h_draft) + row * a.d_draft * esz : nullptr;
            const char *xt = reinterpret_cast<const char *>(a.h_target) + row * a.d * esz;
            float s = block_dot(xd, a.judge_w, a.d_draft, a.dtype, lane) +
                      block_dot(xt, a.judge_w + a.d_draft, a.d, a.dtype, lane);
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
            const float z = a.judge_b + s;
            p = 1.0f / (1.0f + expf(-z));
            const bool forgiven = (a.tau <= 0.0f) ? false : (a.tau >= 1.0f) ? true : (p < a.tau);
            rej = forgiven ? 0 : 1;
        }
        if (lane == 0) {
            rej_s[i] = rej;
            if (a.judge_p) a.judge_p[(size_t)b * K + i] = p;
        }
    }
    __syncthreads();

    if (warp == 0) {
        int first = K;
        for (int base = 0; base < K; base += 32) {
            const int i = base + lane;
            const unsigned m = __ballot_sync(0xffffffffu, i < K && rej_s[i] != 0);
            if (m) {
                first = base + __ffs(m) - 1;
                break;
            }
        }
        if (lane == 0) {
            a.accept_len[b] = first;
            a.next_tok[b] = y_s[first];
        }
    }
}

}  // namespace

cudaError_t launch_judge_scan(const JudgeArgs &a, cudaStream_t stream) {
    const int threads = 512;
    const size_t smem = (size_t)(2 * a.K + 1) * sizeof(int);
    judge_scan_kernel<<<a.B, threads, smem, stream>>>(a);
    return cudaGetLastError();
}

}  // namespace aj
