// CUDA-core projection + running argmax: logit[m,v] = sum_k h[m,k] * W[k,v], fp32 accumulate,
// per-row (max, argmax) merged into packed keys.  This is the path for fp32 storage and for
// layouts / widths the tensor-core kernel does not take; it is also selectable for bf16 with
// AJ_FLAG_FORCE_SIMT.  One warp owns a contiguous slice of the vocabulary and walks it for
// ROWS rows of h at a time.
#include "aj_internal.cuh"

#include <cuda_bf16.h>

namespace aj {

namespace {

constexpr int ROWS = 8;

__device__ inline float load_as_float(const float *p, size_t i) { return p[i]; }
__device__ inline float load_as_float(const __nv_bfloat16 *p, size_t i) { return __bfloat162float(p[i]); }

template <typename T>
__global__ void __launch_bounds__(256) simt_gemm_argmax_kernel(const T *__restrict__ h, const T *__restrict__ W,
                                                               int M, int d, int V, int w_layout, int v_offset,
                                                               unsigned long long *__restrict__ keys, const Publish pub,
                                                               const RankArgs rk, const Noise nz) {
    const int lane = threadIdx.x & 31;
    const int warps_per_block = blockDim.x >> 5;
    const long long warp = (long long)blockIdx.x * warps_per_block + (threadIdx.x >> 5);
    const long long warps_total = (long long)gridDim.x * warps_per_block;
    const int per = (int)((V + warps_total - 1) / warps_total);
    const long long v0l = warp * per;
    const int v0 = (int)(v0l < V ? v0l : V);  // a warp past the end has an empty slice
    const int v1 = min(V, v0 + per);

    for (int m0 = 0; m0 < M && v0 < v1; m0 += ROWS) {
        float best[ROWS];
        int bidx[ROWS];
        unsigned ahead[ROWS];  // top-K rule: entries of this slice that outrank the row's draft token
        float thr[ROWS];
        int tok[ROWS];
#pragma unroll
        for (int r = 0; r < ROWS; r++) {
            best[r] = -INFINITY;
            bidx[r] = v0;
            ahead[r] = 0;
            thr[r] = (rk.thr && m0 + r < M) ? rk.thr[m0 + r] : INFINITY;
            tok[r] = (rk.thr && m0 + r < M) ? rk.tok[m0 + r] : -1;
        }
        for (int v = v0; v < v1; v++) {
            float acc[ROWS];
#pragma unroll
            for (int r = 0; r < ROWS; r++) acc[r] = 0.0f;
            for (int k = lane; k < d; k += 32) {
                const float w = (w_layout == 0) ? load_as_float(W, (size_t)v * d + k)
                                                : load_as_float(W, (size_t)k * V + v);
#pragma unroll
                for (int r = 0; r < ROWS; r++) {
                    const int m = min(m0 + r, M - 1);  // rows past the end repeat the last row; never flushed
                    acc[r] = fmaf(load_as_float(h, (size_t)m * d + k), w, acc[r]);
                }
            }
#pragma unroll
            for (int r = 0; r < ROWS; r++) {
                float s = acc[r];
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
                if (nz.temperature > 0.0f) s = noisy_score(nz, s, min(m0 + r, M - 1), v + v_offset);
                if (s > best[r]) {  // strict: the first (lowest) index keeps a tie
                    best[r] = s;
                    bidx[r] = v;
                }
                if (v != tok[r] && (s > thr[r] || (s == thr[r] && v < tok[r]))) ahead[r]++;
            }
        }
        if (lane == 0) {
#pragma unroll
            for (int r = 0; r < ROWS; r++)
                if (m0 + r < M) {
                    atomicMax(&keys[m0 + r], pack_key(best[r], bidx[r] + v_offset));
                    if (rk.thr && ahead[r]) atomicAdd(rk.cnt + m0 + r, ahead[r]);
                }
        }
    }
    publish_keys(pub, keys);
}

}  // namespace

cudaError_t launch_simt_gemm_argmax(const GemmArgs &a, int num_sms, cudaStream_t stream) {
    const int threads = 256;
    const int warps_per_block = threads / 32;
    long long want_warps = a.V;  // at most one vocabulary entry per warp
    long long max_blocks = (long long)num_sms * 8;
    long long blocks = (want_warps + warps_per_block - 1) / warps_per_block;
    if (blocks > max_blocks) blocks = max_blocks;
    if (blocks < 1) blocks = 1;
    if (a.dtype == 0)
        simt_gemm_argmax_kernel<__nv_bfloat16><<<(unsigned)blocks, threads, 0, stream>>>(
            (const __nv_bfloat16 *)a.h, (const __nv_bfloat16 *)a.W, a.M, a.d, a.V, a.w_layout, a.v_offset, a.keys, a.pub, a.rank,
            a.noise);
    else
        simt_gemm_argmax_kernel<float><<<(unsigned)blocks, threads, 0, stream>>>(
            (const float *)a.h, (const float *)a.W, a.M, a.d, a.V, a.w_layout, a.v_offset, a.keys, a.pub, a.rank, a.noise);
    return cudaGetLastError();
}

}  // namespace aj
