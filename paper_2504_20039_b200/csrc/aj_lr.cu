// Fitting the classifier: L2-regularised logistic regression on device-resident features.
//
//   f(w, b) = 1/2 w.w + C * sum_i log(1 + exp(-s_i (x_i.w + b))),   s_i = +1 if labels[i] != 0 else -1
//
// (the intercept is not regularised; this is scikit-learn's convention, which the paper uses).
// One evaluation of f and its gradient is ONE pass over X: a group of warps loads a row into
// registers (the next one is in flight meanwhile), computes its score z = x.w + b, turns it into the
// residual r = -C s sigma(-s z), and adds r x to its gradient sums from the same registers.  CTAs
// write their partial gradients and partial losses to separate slots, which a second kernel
// (gradient) and the host (loss, intercept) add in a fixed
// order, so an evaluation does not depend on scheduling.  The minimiser is found by L-BFGS on the
// host in fp64 (two-loop recursion, Armijo backtracking); only w travels down and the gradient up.
#include "../../include/aj_verify.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include <mutex>
#include <type_traits>
#include <vector>

namespace aj {

namespace {

constexpr int LR_THREADS = 512;
constexpr int LR_WARPS = LR_THREADS / 32;
constexpr int LR_CPL_MAX = 6;  // 16-byte chunks of a row a lane owns at most

// the features of one 16-byte chunk of a row as floats
template <bool BF16> struct Chunk;
template <> struct Chunk<true> {
    static constexpr int ELEMS = 8;
    static __device__ inline void unpack(const uint4 &v, float (&x)[8]) {
        const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; i++) {  // a bf16 is the upper half of an fp32
            x[2 * i] = __uint_as_float(u[i] << 16);
            x[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
        }
    }
};
template <> struct Chunk<false> {
    static constexpr int ELEMS = 4;
    static __device__ inline void unpack(const uint4 &v, float (&x)[8]) {
        x[0] = __uint_as_float(v.x), x[1] = __uint_as_float(v.y), x[2] = __uint_as_float(v.z), x[3] = __uint_as_float(v.w);
        x[4] = x[5] = x[6] = x[7] = 0.0f;
    }
};

struct LrArgs {
    const char *X;           // [n, F], rows of row_bytes bytes
    const uint8_t *labels;   // [n]
    long long n;
    int F;
    size_t row_bytes;
    const float *w;          // [F]
    float b, C;
    float *partial_g;        // [grid, F]
    double *partial_loss;    // [grid]
    double *partial_gb;      // [grid]
};

// A group of G warps takes one row at a time: lane l of the group owns the 16-byte chunks l, l + 32 G, ...
// (CPL of them at most) of every row the group takes, loads them straight from global memory into
// registers one row ahead, and keeps its share of the gradient in registers for the whole launch.
// The groups of a CTA run independently of one another; the warps of a group meet once per row at a
// named barrier to add their partial scores.  The weights are read from shared memory.
template <bool BF16, int CPL, int G>
__global__ void __launch_bounds__(LR_THREADS, 1) lr_loss_grad_kernel(const LrArgs a) {
    extern __shared__ __align__(16) char lr_smem[];
    constexpr int EPC = Chunk<BF16>::ELEMS;
    constexpr int GROUPS = LR_WARPS / G;
    constexpr int GL = 32 * G;  // lanes of a group
    const int F = a.F, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int chunks = F / EPC;
    // weights as two arrays of float4 (first and second half of every chunk): conflict-free 16-byte reads
    float4 *w_lo = reinterpret_cast<float4 *>(lr_smem);
    float4 *w_hi = w_lo + chunks;                                              // bf16 only
    float *zbuf = reinterpret_cast<float *>(lr_smem + (size_t)F * 4);          // [GROUPS][2][G] partial scores
    double *red = reinterpret_cast<double *>(zbuf + 2 * LR_WARPS);             // [2][GROUPS] losses, intercept gradients
    for (int c = tid; c < chunks; c += LR_THREADS) {
        const float4 *src = reinterpret_cast<const float4 *>(a.w + (size_t)c * EPC);
        w_lo[c] = src[0];
        if (BF16) w_hi[c] = src[1];
    }
    __syncthreads();

    const int group = warp / G, wg = warp % G, gl = wg * 32 + lane;
    const long long ngroups = (long long)gridDim.x * GROUPS;
    float g[CPL][8];
#pragma unroll
    for (int j = 0; j < CPL; j++)
#pragma unroll
        for (int i = 0; i < 8; i++) g[j][i] = 0.0f;
    uint4 xc[CPL], xn[CPL];
    auto load_row = [&](long long row, uint4 (&x)[CPL]) {
        const uint4 *src = reinterpret_cast<const uint4 *>(a.X + (size_t)row * a.row_bytes);
#pragma unroll
        for (int j = 0; j < CPL; j++) {
            const int c = j * GL + gl;
            x[j] = (row < a.n && c < chunks) ? __ldcs(src + c) : make_uint4(0u, 0u, 0u, 0u);
        }
    };
    long long row = (long long)blockIdx.x * GROUPS + group;
    load_row(row, xc);
    unsigned label = row < a.n ? a.labels[row] : 0u, label_next = 0u;  // fetched a row ahead, like the features
    double loss = 0.0, gb = 0.0;  // lane 0 of the group's first warp
    for (int it = 0; row < a.n; row += ngroups, ++it) {
        load_row(row + ngroups, xn);  // in flight while this row is worked on
        label_next = row + ngroups < a.n ? a.labels[row + ngroups] : 0u;

        float zp = 0.0f;
#pragma unroll
        for (int j = 0; j < CPL; j++) {
            const int c = j * GL + gl;
            if (c < chunks) {
                float x[8];
                Chunk<BF16>::unpack(xc[j], x);
                const float4 lo = w_lo[c];
                zp = fmaf(x[0], lo.x, zp), zp = fmaf(x[1], lo.y, zp), zp = fmaf(x[2], lo.z, zp), zp = fmaf(x[3], lo.w, zp);
                if (BF16) {
                    const float4 hi = w_hi[c];
                    zp = fmaf(x[4], hi.x, zp), zp = fmaf(x[5], hi.y, zp), zp = fmaf(x[6], hi.z, zp), zp = fmaf(x[7], hi.w, zp);
                }
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) zp += __shfl_xor_sync(0xffffffffu, zp, off);
        float z = zp;
        if (G > 1) {  // add the G warps' partial scores: a fixed tree, the same in every warp
            float *slot = zbuf + (group * 2 + (it & 1)) * G;
            if (lane == 0) slot[wg] = zp;
            asm volatile("bar.sync %0, %1;" ::"r"(1 + group), "r"(GL) : "memory");
            float v = lane < G ? slot[lane] : 0.0f;
#pragma unroll
            for (int off = G / 2; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
            z = __shfl_sync(0xffffffffu, v, 0);
        }
        z += a.b;
        const float s = label ? 1.0f : -1.0f;
        const float t = s * z;
        // sigma(-t) = 1 / (1 + exp(t)) from the hardware exponential and reciprocal (about 1e-6 relative; the
        // same bits in every warp of the group); exp(t) = inf gives 0, exp(t) = 0 gives 1
        const float sig = __fdividef(1.0f, 1.0f + __expf(t));
        const float res = -a.C * s * sig;
        if (wg == 0) {  // the loss is kept by the group's first warp only: log(1 + exp(-t)), accurately
            const float e = expf(-fabsf(t));
            const float softplus = log1pf(e) + fmaxf(-t, 0.0f);
            if (lane == 0) {
                loss += softplus;
                gb += res;
            }
        }
#pragma unroll
        for (int j = 0; j < CPL; j++) {
            const int c = j * GL + gl;
            if (c < chunks) {
                float x[8];
                Chunk<BF16>::unpack(xc[j], x);
#pragma unroll
                for (int i = 0; i < EPC; i++) g[j][i] = fmaf(res, x[i], g[j][i]);
            }
        }
#pragma unroll
        for (int j = 0; j < CPL; j++) xc[j] = xn[j];
        label = label_next;
    }

    // the groups' gradients are added in shared memory, one group after the other (the weights are done with)
    __syncthreads();
    float *acc = reinterpret_cast<float *>(lr_smem);
    for (int sel = 0; sel < GROUPS; sel++) {
        if (group == sel) {
#pragma unroll
            for (int j = 0; j < CPL; j++) {
                const int c = j * GL + gl;
                if (c < chunks) {
#pragma unroll
                    for (int i = 0; i < EPC; i++) acc[c * EPC + i] = (sel == 0 ? 0.0f : acc[c * EPC + i]) + g[j][i];
                }
            }
            if (gl == 0) {
                red[sel] = loss;
                red[GROUPS + sel] = gb;
            }
        }
        __syncthreads();
    }
    for (int f = tid; f < F; f += LR_THREADS) a.partial_g[(size_t)blockIdx.x * F + f] = acc[f];
    if (tid == 0) {
        double l = 0.0, gg = 0.0;
        for (int k = 0; k < GROUPS; k++) {
            l += red[k];
            gg += red[GROUPS + k];
        }
        a.partial_loss[blockIdx.x] = l;
        a.partial_gb[blockIdx.x] = gg;
    }
}

__global__ void lr_reduce_kernel(const float *__restrict__ partial_g, int parts, int F, float *__restrict__ g) {
    const int f = blockIdx.x * blockDim.x + threadIdx.x;
    if (f >= F) return;
    float s = 0.0f;
    for (int k = 0; k < parts; k++) s += partial_g[(size_t)k * F + f];  // fixed order
    g[f] = s;
}

// One device allocation and one pinned host allocation, carved into the pieces below.  A device's
// workspace is kept between fits (allocating and freeing the pinned and device memory took longer than
// the fit's kernels) and grows when a fit needs more; aj_lr_release gives it back.
struct Workspace {
    char *dev = nullptr, *host = nullptr;
    size_t dev_bytes = 0, host_bytes = 0;
    cudaEvent_t ev0 = nullptr, ev1 = nullptr;
    size_t head_bytes = 0;         // partial losses, w and the gradient: the part mirrored on the host
    double *partial_ld = nullptr;  // device [2 * grid]: losses, then intercept gradients
    float *w_dev = nullptr, *g_dev = nullptr, *partial_g = nullptr;
    double *ld_host = nullptr;
    float *w_host = nullptr, *g_host = nullptr;
    bool alloc(int F, int grid) {
        const size_t ld = (2 * (size_t)grid * sizeof(double) + 255) & ~(size_t)255;  // every piece starts on a 256-byte boundary
        const size_t vec = ((size_t)F * sizeof(float) + 255) & ~(size_t)255;
        const size_t need_dev = ld + 2 * vec + (size_t)grid * F * sizeof(float), need_host = ld + 2 * vec;
        if (need_dev > dev_bytes || need_host > host_bytes) {
            release();
            if (cudaMalloc(&dev, need_dev) != cudaSuccess || cudaMallocHost(&host, need_host) != cudaSuccess) {
                release();
                return false;
            }
            dev_bytes = need_dev, host_bytes = need_host;
        }
        if (!ev0 && (cudaEventCreate(&ev0) != cudaSuccess || cudaEventCreate(&ev1) != cudaSuccess)) {
            release();
            return false;
        }
        head_bytes = ld + 2 * vec;
        partial_ld = reinterpret_cast<double *>(dev);
        w_dev = reinterpret_cast<float *>(dev + ld);
        g_dev = reinterpret_cast<float *>(reinterpret_cast<char *>(w_dev) + vec);
        partial_g = reinterpret_cast<float *>(reinterpret_cast<char *>(g_dev) + vec);
        ld_host = reinterpret_cast<double *>(host);
        w_host = reinterpret_cast<float *>(host + ld);
        g_host = reinterpret_cast<float *>(reinterpret_cast<char *>(w_host) + vec);
        return true;
    }
    void release() {
        if (dev) cudaFree(dev);
        if (host) cudaFreeHost(host);
        if (ev0) cudaEventDestroy(ev0);
        if (ev1) cudaEventDestroy(ev1);
        dev = host = nullptr;
        ev0 = ev1 = nullptr;
        dev_bytes = host_bytes = 0;
    }
};

constexpr int LR_MAX_DEVICES = 64;
std::mutex g_lr_mutex;  // a fit holds it from start to end: fits in one process take turns
Workspace g_lr_ws[LR_MAX_DEVICES];

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
    // warps per row: the fewest (1, 2, 4, 8 or 16) with at most LR_CPL_MAX chunks per lane
    const int chunks = (int)(row_bytes / 16);
    int G = 1;
    while (G < LR_WARPS && (chunks + 32 * G - 1) / (32 * G) > LR_CPL_MAX) G *= 2;
    const int cpl = (chunks + 32 * G - 1) / (32 * G);
    if (cpl > LR_CPL_MAX) return AJ_ERR_UNSUPPORTED;  // rows wider than 48 KB
    const int groups = LR_WARPS / G;
    const size_t smem = (size_t)F * 4 + 2 * LR_WARPS * sizeof(float) + 2 * LR_WARPS * sizeof(double);

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
    if (device >= LR_MAX_DEVICES) return AJ_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    using Kernel = void (*)(const LrArgs);
    auto pick_g = [&](auto bf, auto cp) -> Kernel {
        constexpr bool B = decltype(bf)::value;
        constexpr int P = decltype(cp)::value;
        switch (G) {
            case 1: return lr_loss_grad_kernel<B, P, 1>;
            case 2: return lr_loss_grad_kernel<B, P, 2>;
            case 4: return lr_loss_grad_kernel<B, P, 4>;
            case 8: return lr_loss_grad_kernel<B, P, 8>;
            default: return lr_loss_grad_kernel<B, P, 16>;
        }
    };
    auto pick_cpl = [&](auto bf) -> Kernel {
        switch (cpl) {
            case 1: return pick_g(bf, std::integral_constant<int, 1>{});
            case 2: return pick_g(bf, std::integral_constant<int, 2>{});
            case 3: return pick_g(bf, std::integral_constant<int, 3>{});
            case 4: return pick_g(bf, std::integral_constant<int, 4>{});
            case 5: return pick_g(bf, std::integral_constant<int, 5>{});
            default: return pick_g(bf, std::integral_constant<int, 6>{});
        }
    };
    Kernel kernel = dtype == AJ_BF16 ? pick_cpl(std::true_type{}) : pick_cpl(std::false_type{});
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return AJ_ERR_CUDA;
    const long long want = (n + groups - 1) / groups;  // CTAs that would have a row for every group
    const int grid = (int)(want < num_sms ? want : num_sms);

    std::lock_guard<std::mutex> lock(g_lr_mutex);
    Workspace &ws = g_lr_ws[device];
    if (!ws.alloc(F, grid)) {
        cudaGetLastError();
        return AJ_ERR_CUDA;
    }

    const int D = F + 1;  // the intercept is the last coordinate
    bool cuda_ok = true;
    cudaEvent_t ev0 = ws.ev0, ev1 = ws.ev1;
    double kernel_ms = 0.0;
    // f and its gradient at v (fp64 on the host, w rounded to fp32 for the device)
    auto eval = [&](const std::vector<double> &v, std::vector<double> &grad) -> double {
        for (int f = 0; f < F; f++) ws.w_host[f] = (float)v[f];
        LrArgs a;
        a.X = static_cast<const char *>(X);
        a.labels = labels;
        a.n = n;
        a.F = F;
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
        // one copy brings back the partial losses and the gradient (and, between them, w as it was sent)
        cuda_ok = cuda_ok && cudaMemcpyAsync(ws.host, ws.dev, ws.head_bytes, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
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

extern "C" aj_status aj_lr_release(int device) {
    using namespace aj;
    if (device >= LR_MAX_DEVICES) return AJ_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_lr_mutex);
    int prev = 0;
    if (cudaGetDevice(&prev) != cudaSuccess) return AJ_ERR_CUDA;
    for (int dev = 0; dev < LR_MAX_DEVICES; dev++) {
        if ((device >= 0 && dev != device) || (!g_lr_ws[dev].dev && !g_lr_ws[dev].ev0)) continue;
        if (cudaSetDevice(dev) != cudaSuccess) {
            cudaGetLastError();
            continue;
        }
        g_lr_ws[dev].release();
    }
    cudaSetDevice(prev);
    return AJ_OK;
}
