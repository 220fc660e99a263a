// Fitting the classifier: L2-regularised logistic regression on device-resident features.
//
//   f(w, b) = 1/2 w.w + C * sum_i log(1 + exp(-s_i (x_i.w + b))),   s_i = +1 if labels[i] != 0 else -1
//
// (the intercept is not regularised; this is scikit-learn's convention, which the paper uses).
// One evaluation of f and its gradient is ONE pass over X: a CTA stages a block of rows in shared
// memory (cp.async, four buffers, two or three in flight), computes the rows' scores z = x.w + b from the
// staged copy, turns them into residuals r_i = -C s_i sigma(-s_i z_i), and adds r_i x_i to its
// own gradient accumulator from the same staged copy.  Every thread owns a fixed set of 16-byte
// feature chunks in both phases and keeps their weights and gradient sums in registers.  CTAs write their partial gradients and partial losses to
// separate slots, which a second kernel (gradient) and the host (loss, intercept) add in a fixed
// order, so an evaluation does not depend on scheduling.  The minimiser is found by L-BFGS on the
// host in fp64 (two-loop recursion, Armijo backtracking); only w travels down and the gradient up.
#include "../../include/aj_verify.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include <type_traits>
#include <vector>

namespace aj {

namespace {

constexpr int LR_THREADS = 512;
constexpr int LR_WARPS = LR_THREADS / 32;
constexpr int LR_NBUF = 4;     // shared-memory buffers of one row block each
constexpr int LR_RB_MAX = 8;   // rows per block at most (score accumulators per thread)
constexpr int LR_MAXC = 4;     // 16-byte feature chunks a thread owns at most: rows of up to 32 KB
constexpr int LR_SMEM_BUDGET = 220 * 1024;

__device__ inline void cp_async_16(void *smem_dst, const void *gmem_src) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gmem_src) : "memory");
}
__device__ inline void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ inline void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// the features of one 16-byte chunk of a staged row as floats
template <bool BF16> struct Chunk;
template <> struct Chunk<true> {
    static constexpr int ELEMS = 8;
    static __device__ inline void load(const char *p, float (&x)[8]) {
        const uint4 v = *reinterpret_cast<const uint4 *>(p);
        const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&v);
#pragma unroll
        for (int i = 0; i < 4; i++) {
            const float2 f = __bfloat1622float2(h[i]);
            x[2 * i] = f.x;
            x[2 * i + 1] = f.y;
        }
    }
};
template <> struct Chunk<false> {
    static constexpr int ELEMS = 4;
    static __device__ inline void load(const char *p, float (&x)[8]) {
        const float4 v = *reinterpret_cast<const float4 *>(p);
        x[0] = v.x, x[1] = v.y, x[2] = v.z, x[3] = v.w;
        x[4] = x[5] = x[6] = x[7] = 0.0f;
    }
};

struct LrArgs {
    const char *X;           // [n, F], rows of row_bytes bytes
    const uint8_t *labels;   // [n]
    long long n;
    int F, rb;               // features; rows per block
    size_t row_bytes;
    const float *w;          // [F]
    float b, C;
    float *partial_g;        // [grid, F]
    double *partial_loss;    // [grid]
    double *partial_gb;      // [grid]
};

// Thread t owns the chunks t, t + LR_THREADS, ... of every row: their weights and its share of the
// CTA's gradient stay in registers for the whole launch; shared memory holds only the staged rows.
// MAXC: chunks a thread owns at most; RB: rows per block (a shorter last block takes the guarded path).
template <bool BF16, int MAXC, int RB>
__global__ void __launch_bounds__(LR_THREADS, 1) lr_loss_grad_kernel(const LrArgs a) {
    extern __shared__ __align__(16) char lr_smem[];
    constexpr int EPC = Chunk<BF16>::ELEMS;
    constexpr int rb = RB;
    const int F = a.F, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int chunks = F / EPC;
    const int row_bytes = (int)a.row_bytes;           // at most 32 KB
    const int stage_bytes = rb * row_bytes;
    float *z_part = reinterpret_cast<float *>(lr_smem);         // [2][LR_WARPS][LR_RB_MAX], alternating between blocks
    char *x_s = reinterpret_cast<char *>(z_part + 2 * LR_WARPS * LR_RB_MAX);  // [LR_NBUF][rb rows]

    float wv[MAXC][8], g[MAXC][8];
#pragma unroll
    for (int k = 0; k < MAXC; k++) {
        const int c = tid + k * LR_THREADS;
#pragma unroll
        for (int i = 0; i < 8; i++) {
            wv[k][i] = (c < chunks && i < EPC) ? a.w[(size_t)c * EPC + i] : 0.0f;
            g[k][i] = 0.0f;
        }
    }
    const long long nblk = (a.n + rb - 1) / rb;
    auto issue = [&](long long blk, int buf) {
        if (blk < nblk) {
            const long long row0 = blk * rb;
            const int bytes = (int)(a.n - row0 < rb ? a.n - row0 : rb) * row_bytes;
            const char *src = a.X + (size_t)row0 * a.row_bytes;
            char *dst = x_s + buf * stage_bytes;
            for (int off = tid * 16; off < bytes; off += LR_THREADS * 16) cp_async_16(dst + off, src + off);
        }
        cp_async_commit();  // an empty group keeps the count of pending groups uniform
    };
    for (int i = 0; i < LR_NBUF - 1; i++) issue((long long)blockIdx.x + (long long)i * gridDim.x, i);

    double loss = 0.0, gb = 0.0;  // lane 0 of warp 0 only
    long long it = 0;
    for (long long blk = blockIdx.x; blk < nblk; blk += gridDim.x, ++it) {
        cp_async_wait<LR_NBUF - 2>();
        __syncthreads();  // the block's rows are visible to every thread, and every thread is done with the block before
        issue(blk + (long long)(LR_NBUF - 1) * gridDim.x, (int)((it + LR_NBUF - 1) % LR_NBUF));  // refills that block's buffer
        const char *xb = x_s + (int)(it % LR_NBUF) * stage_bytes;
        const long long row0 = blk * rb;
        const int rows = (int)(a.n - row0 < rb ? a.n - row0 : rb);
        const bool full = rows == rb;  // all blocks but possibly the last

        // scores: every thread adds its chunks' share of every row's dot product
        float zp[RB];
#pragma unroll
        for (int r = 0; r < RB; r++) zp[r] = 0.0f;
#pragma unroll
        for (int k = 0; k < MAXC; k++) {
            const int c = tid + k * LR_THREADS;
            if (c < chunks) {
                const char *xc = xb + c * 16;
#pragma unroll
                for (int r = 0; r < RB; r++) {
                    if (full || r < rows) {
                        float x[8];
                        Chunk<BF16>::load(xc + r * row_bytes, x);
#pragma unroll
                        for (int i = 0; i < EPC; i++) zp[r] = fmaf(x[i], wv[k][i], zp[r]);
                    }
                }
            }
        }
#pragma unroll
        for (int r = 0; r < RB; r++) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) zp[r] += __shfl_xor_sync(0xffffffffu, zp[r], off);
            if (lane == 0) z_part[((int)(it & 1) * LR_WARPS + warp) * LR_RB_MAX + r] = zp[r];
        }
        __syncthreads();
        // every warp finishes the rows itself (lane r: row r), so that none waits for another
        float softplus = 0.0f, res = 0.0f;
        if (lane < rows) {
            float z = a.b;
#pragma unroll
            for (int k = 0; k < LR_WARPS; k++) z += z_part[((int)(it & 1) * LR_WARPS + k) * LR_RB_MAX + lane];  // fixed order
            const float s = a.labels[row0 + lane] ? 1.0f : -1.0f;
            const float t = s * z;
            const float e = expf(-fabsf(t));
            softplus = log1pf(e) + fmaxf(-t, 0.0f);                            // log(1 + exp(-t))
            const float sig = t >= 0.0f ? e / (1.0f + e) : 1.0f / (1.0f + e);  // sigma(-t)
            res = -a.C * s * sig;
        }
        if (warp == 0) {  // the sums are kept by one warp; lanes without a row contribute zeros
            double l = softplus, gg = res;
            for (int off = 16; off > 0; off >>= 1) {
                l += __shfl_xor_sync(0xffffffffu, l, off);
                gg += __shfl_xor_sync(0xffffffffu, gg, off);
            }
            if (lane == 0) {
                loss += l;
                gb += gg;
            }
        }
        float rr_row[RB];
#pragma unroll
        for (int r = 0; r < RB; r++) rr_row[r] = __shfl_sync(0xffffffffu, res, r);

        // gradient: the same chunks, the same staged rows
#pragma unroll
        for (int k = 0; k < MAXC; k++) {
            const int c = tid + k * LR_THREADS;
            if (c < chunks) {
                const char *xc = xb + c * 16;
#pragma unroll
                for (int r = 0; r < RB; r++) {
                    if (full || r < rows) {
                        float x[8];
                        Chunk<BF16>::load(xc + r * row_bytes, x);
                        const float rr = rr_row[r];
#pragma unroll
                        for (int i = 0; i < EPC; i++) g[k][i] = fmaf(rr, x[i], g[k][i]);
                    }
                }
            }
        }
    }
    cp_async_wait<0>();
#pragma unroll
    for (int k = 0; k < MAXC; k++) {
        const int c = tid + k * LR_THREADS;
        if (c < chunks) {
#pragma unroll
            for (int i = 0; i < EPC; i++) a.partial_g[(size_t)blockIdx.x * F + (size_t)c * EPC + i] = g[k][i];
        }
    }
    if (tid == 0) {
        a.partial_loss[blockIdx.x] = loss;
        a.partial_gb[blockIdx.x] = gb;
    }
}

__global__ void lr_reduce_kernel(const float *__restrict__ partial_g, int parts, int F, float *__restrict__ g) {
    const int f = blockIdx.x * blockDim.x + threadIdx.x;
    if (f >= F) return;
    float s = 0.0f;
    for (int k = 0; k < parts; k++) s += partial_g[(size_t)k * F + f];  // fixed order
    g[f] = s;
}

struct Workspace {
    float *w_dev = nullptr, *g_dev = nullptr, *partial_g = nullptr;
    double *partial_ld = nullptr;  // [2 * grid]: losses, then intercept gradients
    float *w_host = nullptr, *g_host = nullptr;
    double *ld_host = nullptr;
    ~Workspace() {
        cudaFree(w_dev);
        cudaFree(g_dev);
        cudaFree(partial_g);
        cudaFree(partial_ld);
        cudaFreeHost(w_host);
        cudaFreeHost(g_host);
        cudaFreeHost(ld_host);
    }
};

}  // namespace

}  // namespace aj

extern "C" aj_status aj_lr_fit(int device, const void *X, const uint8_t *labels, long long n, int F, aj_dtype dtype, float C,
                               int max_iter, float tol, float *w_out, float *b_out, int *iters_out, float *stats_out,
                               void *cuda_stream) {
    using namespace aj;
    if (!X || !labels || !w_out || !b_out || n < 1 || F < 1 || !(C > 0.0f) || max_iter < 1 || !(tol >= 0.0f)) return AJ_ERR_INVALID_ARG;
    if (dtype != AJ_BF16 && dtype != AJ_F32) return AJ_ERR_INVALID_ARG;
    const size_t esz = dtype == AJ_BF16 ? 2 : 4;
    const size_t row_bytes = (size_t)F * esz;
    if (row_bytes % 16 != 0 || (reinterpret_cast<uintptr_t>(X) & 15) != 0) return AJ_ERR_UNSUPPORTED;
    const size_t fixed = 2 * LR_WARPS * LR_RB_MAX * sizeof(float);
    if (row_bytes > (size_t)LR_MAXC * LR_THREADS * 16) return AJ_ERR_UNSUPPORTED;  // a thread owns at most LR_MAXC chunks of a row
    if (fixed + LR_NBUF * row_bytes > (size_t)LR_SMEM_BUDGET) return AJ_ERR_UNSUPPORTED;  // a row must fit four times
    int rb = (int)((LR_SMEM_BUDGET - fixed) / (LR_NBUF * row_bytes));
    if (rb > LR_RB_MAX) rb = LR_RB_MAX;
    const size_t smem = fixed + (size_t)LR_NBUF * rb * row_bytes;

    int prev = 0;
    if (cudaGetDevice(&prev) != cudaSuccess || cudaSetDevice(device) != cudaSuccess) return AJ_ERR_CUDA;
    struct Restore {
        int d;
        ~Restore() { cudaSetDevice(d); }
    } restore{prev};
    int cc_major = 0, num_sms = 0;
    if (cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess)
        return AJ_ERR_CUDA;
    if (cc_major != 10) return AJ_ERR_NOT_SM100;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int maxc = (int)((row_bytes / 16 + LR_THREADS - 1) / LR_THREADS);  // 1 .. LR_MAXC
    using Kernel = void (*)(const LrArgs);
    auto pick_rb = [&](auto bf, auto mc) -> Kernel {
        constexpr bool B = decltype(bf)::value;
        constexpr int M = decltype(mc)::value;
        switch (rb) {
            case 1: return lr_loss_grad_kernel<B, M, 1>;
            case 2: return lr_loss_grad_kernel<B, M, 2>;
            case 3: return lr_loss_grad_kernel<B, M, 3>;
            case 4: return lr_loss_grad_kernel<B, M, 4>;
            case 5: return lr_loss_grad_kernel<B, M, 5>;
            case 6: return lr_loss_grad_kernel<B, M, 6>;
            case 7: return lr_loss_grad_kernel<B, M, 7>;
            default: return lr_loss_grad_kernel<B, M, 8>;
        }
    };
    auto pick_mc = [&](auto bf) -> Kernel {
        switch (maxc) {
            case 1: return pick_rb(bf, std::integral_constant<int, 1>{});
            case 2: return pick_rb(bf, std::integral_constant<int, 2>{});
            default: return pick_rb(bf, std::integral_constant<int, LR_MAXC>{});
        }
    };
    Kernel kernel = dtype == AJ_BF16 ? pick_mc(std::true_type{}) : pick_mc(std::false_type{});
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return AJ_ERR_CUDA;
    const long long nblk = (n + rb - 1) / rb;
    const int grid = (int)(nblk < num_sms ? nblk : num_sms);

    Workspace ws;
    if (cudaMalloc(&ws.w_dev, F * sizeof(float)) != cudaSuccess || cudaMalloc(&ws.g_dev, F * sizeof(float)) != cudaSuccess ||
        cudaMalloc(&ws.partial_g, (size_t)grid * F * sizeof(float)) != cudaSuccess ||
        cudaMalloc(&ws.partial_ld, 2 * (size_t)grid * sizeof(double)) != cudaSuccess ||
        cudaMallocHost(&ws.w_host, F * sizeof(float)) != cudaSuccess || cudaMallocHost(&ws.g_host, F * sizeof(float)) != cudaSuccess ||
        cudaMallocHost(&ws.ld_host, 2 * (size_t)grid * sizeof(double)) != cudaSuccess) {
        cudaGetLastError();
        return AJ_ERR_CUDA;
    }

    const int D = F + 1;  // the intercept is the last coordinate
    bool cuda_ok = true;
    cudaEvent_t ev0 = nullptr, ev1 = nullptr;
    if (cudaEventCreate(&ev0) != cudaSuccess || cudaEventCreate(&ev1) != cudaSuccess) return AJ_ERR_CUDA;
    struct Events {
        cudaEvent_t a, b;
        ~Events() {
            cudaEventDestroy(a);
            cudaEventDestroy(b);
        }
    } events{ev0, ev1};
    double kernel_ms = 0.0;
    // f and its gradient at v (fp64 on the host, w rounded to fp32 for the device)
    auto eval = [&](const std::vector<double> &v, std::vector<double> &grad) -> double {
        for (int f = 0; f < F; f++) ws.w_host[f] = (float)v[f];
        LrArgs a;
        a.X = static_cast<const char *>(X);
        a.labels = labels;
        a.n = n;
        a.F = F;
        a.rb = rb;
        a.row_bytes = row_bytes;
        a.w = ws.w_dev;
        a.b = (float)v[F];
        a.C = C;
        a.partial_g = ws.partial_g;
        a.partial_loss = ws.partial_ld;
        a.partial_gb = ws.partial_ld + grid;
        cuda_ok = cuda_ok && cudaMemcpyAsync(ws.w_dev, ws.w_host, F * sizeof(float), cudaMemcpyHostToDevice, stream) == cudaSuccess;
        cudaEventRecord(ev0, stream);
        kernel<<<grid, LR_THREADS, smem, stream>>>(a);
        cudaEventRecord(ev1, stream);
        lr_reduce_kernel<<<(F + 255) / 256, 256, 0, stream>>>(ws.partial_g, grid, F, ws.g_dev);
        cuda_ok = cuda_ok && cudaGetLastError() == cudaSuccess;
        cuda_ok = cuda_ok && cudaMemcpyAsync(ws.g_host, ws.g_dev, F * sizeof(float), cudaMemcpyDeviceToHost, stream) == cudaSuccess;
        cuda_ok = cuda_ok && cudaMemcpyAsync(ws.ld_host, ws.partial_ld, 2 * (size_t)grid * sizeof(double), cudaMemcpyDeviceToHost, stream) == cudaSuccess;
        cuda_ok = cuda_ok && cudaStreamSynchronize(stream) == cudaSuccess;
        if (!cuda_ok) return 0.0;
        float ms = 0.0f;
        if (cudaEventElapsedTime(&ms, ev0, ev1) == cudaSuccess) kernel_ms += ms;
        double loss = 0.0, gb = 0.0, ww = 0.0;
        for (int k = 0; k < grid; k++) {
            loss += ws.ld_host[k];
            gb += ws.ld_host[grid + k];
        }
        for (int f = 0; f < F; f++) {
            const double wf = (double)ws.w_host[f];
            ww += wf * wf;
            grad[f] = wf + (double)ws.g_host[f];
        }
        grad[F] = gb;
        return 0.5 * ww + (double)C * loss;
    };
    auto max_abs = [&](const std::vector<double> &x) {
        double m = 0.0;
        for (double t : x) m = fabs(t) > m ? fabs(t) : m;
        return m;
    };
    auto dot = [&](const std::vector<double> &x, const std::vector<double> &y) {
        double s = 0.0;
        for (int i = 0; i < D; i++) s += x[i] * y[i];
        return s;
    };

    constexpr int HIST = 10;
    std::vector<double> v(D, 0.0), g(D), vn(D), gn(D), dir(D), alpha(HIST);
    std::vector<std::vector<double>> S, Y;
    std::vector<double> rho;
    double f = eval(v, g);
    int iters = 0, evals = 1;
    while (cuda_ok && iters < max_iter && max_abs(g) > (double)tol) {
        // two-loop recursion: dir = -H g
        dir = g;
        const int m = (int)S.size();
        for (int k = m - 1; k >= 0; k--) {
            alpha[k] = rho[k] * dot(S[k], dir);
            for (int i = 0; i < D; i++) dir[i] -= alpha[k] * Y[k][i];
        }
        if (m > 0) {
            const double gamma = dot(S[m - 1], Y[m - 1]) / dot(Y[m - 1], Y[m - 1]);
            for (int i = 0; i < D; i++) dir[i] *= gamma;
        }
        for (int k = 0; k < m; k++) {
            const double beta = rho[k] * dot(Y[k], dir);
            for (int i = 0; i < D; i++) dir[i] += (alpha[k] - beta) * S[k][i];
        }
        double slope = -dot(g, dir);  // along -dir
        if (!(slope < 0.0)) {         // not a descent direction: forget the history
            S.clear(), Y.clear(), rho.clear();
            dir = g;
            slope = -dot(g, g);
        }
        double step = (m == 0 && S.empty()) ? 1.0 / (1.0 + sqrt(dot(g, g))) : 1.0;
        double fn = f;
        bool moved = false;
        for (int ls = 0; ls < 30 && cuda_ok; ls++) {
            for (int i = 0; i < D; i++) vn[i] = v[i] - step * dir[i];
            fn = eval(vn, gn);
            evals++;
            if (fn <= f + 1e-4 * step * slope) {
                moved = true;
                break;
            }
            step *= 0.5;
        }
        if (!moved) break;  // no decrease within fp32 evaluation noise: this is as far as it goes
        std::vector<double> s(D), y(D);
        for (int i = 0; i < D; i++) {
            s[i] = vn[i] - v[i];
            y[i] = gn[i] - g[i];
        }
        const double sy = dot(s, y);
        if (sy > 1e-12 * sqrt(dot(s, s) * dot(y, y))) {
            if ((int)S.size() == HIST) {
                S.erase(S.begin());
                Y.erase(Y.begin());
                rho.erase(rho.begin());
            }
            S.push_back(s);
            Y.push_back(y);
            rho.push_back(1.0 / sy);
        }
        v.swap(vn);
        g.swap(gn);
        f = fn;
        iters++;
    }
    if (!cuda_ok) {
        cudaGetLastError();
        return AJ_ERR_CUDA;
    }
    for (int i = 0; i < F; i++) ws.w_host[i] = (float)v[i];
    if (cudaMemcpyAsync(w_out, ws.w_host, F * sizeof(float), cudaMemcpyHostToDevice, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess)
        return AJ_ERR_CUDA;
    *b_out = (float)v[F];
    if (iters_out) {
        iters_out[0] = iters;
        iters_out[1] = evals;
    }
    if (stats_out) {
        stats_out[0] = (float)max_abs(g);
        stats_out[1] = (float)kernel_ms;
    }
    return AJ_OK;
}
