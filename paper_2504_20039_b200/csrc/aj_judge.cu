// Mismatch mask, judge at mismatches, accepted-prefix scan: one block per sequence.
//
//   y[j]    = index stored in the row's packed key                    (greedy target tokens)
//   mis[i]  = draft_tok[i] != y[i]
//   p[i]    = sigmoid(b + w . [h_draft[i+1] ; h_target[i+1]])         only where mis[i]
//   stop    = first i with mis[i] and not (p[i] < tau)                ballot + ffs over the window
//   accept_len = stop (K if none), next_tok = y[accept_len]
//
// The judge is latency-bound (a few rows of 8-24 KB each), so the work is cut into
// (position, segment) items: a segment is 1/SEGS of the concatenated feature vector, a warp
// takes one item at a time and issues all of its 128-bit loads before it uses any of them.
// Segment sums are added in a fixed order, so p does not depend on scheduling.
//
// Tree drafts (a.parent given): the K draft tokens are the nodes of a tree in topological order, row
// i + 1 encodes node i, and node i is compared with the target's token of its PARENT's row.  The
// classifier is evaluated at every mismatching node as above; a node is accepted iff its parent is
// (the root always is) and it matches or is forgiven; the result is the deepest accepted node, the
// lowest index among equally deep ones.  A chain (parent[i] = i - 1) is the window case.
//
// When the projection kernel has computed the target half of w . x as three extra rows of the LM head
// (a.fold_parts), only the draft half is read here and the three partial sums are added to it.
//
// The kernel is launched as a programmatic dependent of the projection kernel: its blocks may
// become resident while that kernel still runs and wait at the grid dependency before they
// read the keys.  Each key is cleared right after it is read, so the next cycle finds zeros.
#include "aj_internal.cuh"

#include <cuda_bf16.h>

namespace aj {

namespace {

constexpr int SEGS = 8;
constexpr int THREADS = 512;

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

__device__ inline float dot4_f32(const float4 &a, const float4 &b) {
    float s = a.x * b.x;
    s = fmaf(a.y, b.y, s);
    s = fmaf(a.z, b.z, s);
    s = fmaf(a.w, b.w, s);
    return s;
}

// This lane's share of chunks [c0, c1) of the concatenated feature vector; a chunk is 16 bytes
// of features (8 bf16 or 4 f32).  Chunks below `split` come from the draft row, the rest from
// the target row.  Four chunks are in flight per lane.
template <bool BF16>
__device__ inline float segment_dot(const char *xd, const char *xt, const float *w, int split, int c0, int c1, int lane) {
    constexpr int EPC = BF16 ? 8 : 4;  // elements per chunk
    float acc = 0.0f;
    for (int c = c0 + lane; c < c1; c += 128) {
        uint4 x[4];
        float4 wa[4], wb[4];
#pragma unroll
        for (int u = 0; u < 4; u++) {
            const int cc = c + 32 * u;
            if (cc < c1) {
                const char *src = cc < split ? xd + (size_t)cc * 16 : xt + (size_t)(cc - split) * 16;
                x[u] = __ldg(reinterpret_cast<const uint4 *>(src));
                const float4 *wp = reinterpret_cast<const float4 *>(w + (size_t)cc * EPC);
                wa[u] = __ldg(wp);
                if (BF16) wb[u] = __ldg(wp + 1);
            } else {
                x[u] = make_uint4(0, 0, 0, 0);
                wa[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                wb[u] = wa[u];
            }
        }
#pragma unroll
        for (int u = 0; u < 4; u++) {
            if (BF16)
                acc += dot8_bf16(x[u], wa[u], wb[u]);
            else
                acc += dot4_f32(*reinterpret_cast<const float4 *>(&x[u]), wa[u]);
        }
    }
    return acc;
}

// scalar fallback for widths or addresses that do not allow 16-byte loads
__device__ inline float scalar_dot(const void *x, const float *w, int n, int dtype, int lane) {
    float s = 0.0f;
    if (x == nullptr) return s;
    if (dtype == 0) {
        const __nv_bfloat16 *xs = reinterpret_cast<const __nv_bfloat16 *>(x);
        for (int f = lane; f < n; f += 32) s = fmaf(__bfloat162float(xs[f]), w[f], s);
    } else {
        const float *xs = reinterpret_cast<const float *>(x);
        for (int f = lane; f < n; f += 32) s = fmaf(xs[f], w[f], s);
    }
    return s;
}

__global__ void __maxnreg__(96) judge_scan_kernel(JudgeArgs a) {
    extern __shared__ int smem[];
    const int K = a.K, R = a.K + 1 - a.no_extra_row;  // without the extra row the last draft token is not encoded
    int *y_s = smem;                                          // [K+1]
    int *rej_s = smem + R;                                    // [K]: 1 = mismatch not forgiven
    int *mis_s = rej_s + K;                                   // [K]
    float *part_s = reinterpret_cast<float *>(mis_s + K);     // [K][SEGS]
    int *par_s = reinterpret_cast<int *>(part_s + K * SEGS);  // [K] tree drafts: parent, or below -1 if not valid
    const int b = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const size_t esz = a.dtype == 0 ? 2 : 4;
    const int epc = a.dtype == 0 ? 8 : 4;

    const uintptr_t row_bytes_t = (uintptr_t)a.d * esz, row_bytes_d = (uintptr_t)a.d_draft * esz;

    // ---- before the grid dependency: everything that does not need the projection's result.
    // Let the next kernel in the stream start its own prologue, stage the draft tokens, and pull
    // the judge weights (and, for small batches, the candidate feature rows) into L2.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    for (int i = threadIdx.x; i < K; i += blockDim.x) mis_s[i] = a.draft_tok[(size_t)b * K + i];
    if (a.parent) {
        for (int i = threadIdx.x; i < K; i += blockDim.x) {
            const int q = a.parent[(size_t)b * K + i];
            par_s[i] = (q >= -1 && q < i) ? q : -2;  // a parent must come earlier; anything else is never accepted
        }
    }
    if (a.top_k == 0) {  // the classifier's operands; the top-K rule needs none of them
        const char *wbytes = reinterpret_cast<const char *>(a.judge_w);
        const size_t wlines = ((size_t)(a.d + a.d_draft) * 4 + 127) / 128;
        for (size_t l = threadIdx.x; l < wlines; l += blockDim.x)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(wbytes + l * 128));
        if ((long long)gridDim.x * K <= 256) {
            const size_t lt = a.fold_parts ? 0 : (row_bytes_t + 127) / 128, ld = a.h_draft ? (row_bytes_d + 127) / 128 : 0;
            const size_t per_row = lt + ld;
            for (size_t l = threadIdx.x; l < per_row * (R - 1); l += blockDim.x) {
                const size_t row = (size_t)b * R + 1 + l / per_row, o = l % per_row;
                const char *src = o < lt ? reinterpret_cast<const char *>(a.h_target) + row * row_bytes_t + o * 128
                                         : reinterpret_cast<const char *>(a.h_draft) + row * row_bytes_d + (o - lt) * 128;
                asm volatile("prefetch.global.L2 [%0];" ::"l"(src));
            }
        }
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // ---- the projection kernel has finished and its keys are visible
    if (a.gather.world > 0) {
        // Vocabulary-parallel: every GPU's projection kernel stores its keys into a slot of this
        // GPU's exchange buffer and then the cycle's epoch into a flag.  Wait for all flags.
        if ((int)threadIdx.x < a.gather.world) {
            const unsigned long long *f = a.gather.flags + threadIdx.x;
            unsigned long long seen, t0 = 0;
            for (unsigned spin = 0;; ++spin) {
                asm volatile("ld.acquire.sys.global.u64 %0, [%1];" : "=l"(seen) : "l"(f) : "memory");
                if (seen >= a.gather.epoch) break;
                if ((spin & 0x3F) == 0x3F) {
                    unsigned long long now;
                    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
                    if (t0 == 0) {
                        t0 = now;
                    } else if (now - t0 > 2000000000ull) {  // 2 s: a peer never published
                        atomicCAS(a.status, DEV_OK, DEV_TIMEOUT);
                        break;
                    }
                    __nanosleep(200);
                }
            }
        }
        __syncthreads();
    }
    for (int j = threadIdx.x; j < R; j += blockDim.x) {
        unsigned long long key;
        if (a.gather.world > 0) {
            key = 0ull;
            for (int g = 0; g < a.gather.world; g++) {
                const unsigned long long k = __ldcg(a.gather.slots + (size_t)g * a.gather.stride + (size_t)b * R + j);
                key = k > key ? k : key;  // the same merge the projection kernel's atomic max performs
            }
        } else {
            unsigned long long *kp = a.keys + (size_t)b * R + j;
            key = *kp;
            *kp = 0ull;  // leave the workspace clean for the next cycle
        }
        const int y = key_index(key);
        y_s[j] = y;
        if (a.target_tok) a.target_tok[(size_t)b * R + j] = y;
        if (a.top1_val) a.top1_val[(size_t)b * R + j] = key_value(key);
    }
    __syncthreads();
    if (a.parent) {
        for (int i = threadIdx.x; i < K; i += blockDim.x) mis_s[i] = par_s[i] < -1 || mis_s[i] != y_s[par_s[i] + 1];
    } else {
        for (int i = threadIdx.x; i < K; i += blockDim.x) mis_s[i] = mis_s[i] != y_s[i];  // staged token vs greedy token
    }
    __syncthreads();

    const bool vec = (a.d % epc == 0) && (a.d_draft % epc == 0) && (row_bytes_t % 16 == 0) && (row_bytes_d % 16 == 0) &&
                     ((reinterpret_cast<uintptr_t>(a.h_target) & 15) == 0) &&
                     ((reinterpret_cast<uintptr_t>(a.h_draft) & 15) == 0) &&
                     ((reinterpret_cast<uintptr_t>(a.judge_w) & 15) == 0);
    const int split = a.d_draft / epc;                 // chunks that belong to the draft row
    const int chunks = (a.d_draft + (a.fold_parts ? 0 : a.d)) / epc;  // the target half may come from the projection kernel
    for (int it = warp; it < K * SEGS; it += nwarps) {
        const int i = it / SEGS, seg = it % SEGS;
        if (!mis_s[i] || i + 1 >= R || a.top_k > 0) continue;  // at mismatches only, where the features exist; not under the top-K rule
        if (a.parent && par_s[i] < -1) continue;                // a node without a valid parent is not judged
        const size_t row = (size_t)b * R + (i + 1);     // the hidden states that encode draft token i
        const char *xd = a.h_draft ? reinterpret_cast<const char *>(a.h_draft) + row * row_bytes_d : nullptr;
        const char *xt = reinterpret_cast<const char *>(a.h_target) + row * row_bytes_t;
        float s;
        if (vec) {
            const int c0 = (int)((long long)chunks * seg / SEGS), c1 = (int)((long long)chunks * (seg + 1) / SEGS);
            s = a.dtype == 0 ? segment_dot<true>(xd, xt, a.judge_w, split, c0, c1, lane)
                             : segment_dot<false>(xd, xt, a.judge_w, split, c0, c1, lane);
        } else {
            s = seg == 0 ? scalar_dot(xd, a.judge_w, a.d_draft, a.dtype, lane) +
                               (a.fold_parts ? 0.0f : scalar_dot(xt, a.judge_w + a.d_draft, a.d, a.dtype, lane))
                         : 0.0f;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        if (lane == 0) part_s[it] = s;
    }
    __syncthreads();

    for (int i = threadIdx.x; i < K; i += blockDim.x) {
        float p = __int_as_float(0x7fc00000);  // NaN where the judge is not consulted
        int rej = 0;
        if (a.parent && par_s[i] < -1) {
            rej = 1;
        } else if (mis_s[i] && a.top_k > 0) {
            // top-K rule: accepted iff fewer than top_k entries outrank the draft token; p reports the rank
            const int tk = a.draft_tok[(size_t)b * K + i];
            const bool in_vocab = tk >= 0 && tk < a.V;
            const unsigned ahead = in_vocab ? a.rank_cnt[(size_t)b * R + i] : (unsigned)a.V;
            p = (float)ahead;
            rej = (in_vocab && ahead < (unsigned)a.top_k) ? 0 : 1;
        } else if (mis_s[i] && i + 1 >= R) {
            rej = 1;  // the states that encode the last draft token were not computed: rejected unjudged
        } else if (mis_s[i]) {
            float z = a.judge_b;
#pragma unroll
            for (int seg = 0; seg < SEGS; seg++) z += part_s[i * SEGS + seg];
            if (a.fold_parts) {
                const float *fp = a.fold_parts + (size_t)b * R + (i + 1);  // the row that encodes draft token i
                z += (__ldcg(fp) + __ldcg(fp + a.fold_stride)) + __ldcg(fp + 2 * (size_t)a.fold_stride);
            }
            p = 1.0f / (1.0f + expf(-z));
            const bool forgiven = (a.tau <= 0.0f) ? false : (a.tau >= 1.0f) ? true : (p < a.tau);
            rej = forgiven ? 0 : 1;
        }
        rej_s[i] = rej;
        if (a.judge_p) a.judge_p[(size_t)b * K + i] = p;
    }
    __syncthreads();

    if (a.parent) {
        // Walk the nodes in their (topological) order: rej_s becomes "not accepted", mis_s the depth.
        if (threadIdx.x == 0) {
            int best = -1, best_depth = 0;
            for (int n = 0; n < K; n++) {
                const int q = par_s[n];
                if (q < -1) {
                    rej_s[n] = 1;
                    continue;
                }
                const int depth = (q < 0 ? 0 : mis_s[q]) + 1;
                const int ok = (q < 0 || !rej_s[q]) && !rej_s[n];
                mis_s[n] = depth;
                rej_s[n] = !ok;
                if (ok && depth > best_depth) {  // strict: the lowest index among equally deep nodes
                    best = n;
                    best_depth = depth;
                }
            }
            a.accept_len[b] = best_depth;
            a.next_tok[b] = y_s[best + 1];
            if (a.best_node) a.best_node[b] = best;
        }
    } else if (warp == 0) {
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
            a.next_tok[b] = first < R ? y_s[first] : -1;  // all K accepted and no row K: nothing to predict from
        }
    }
}

// w_target as three bf16 rows whose sum is w_target to fp32 precision, laid out like the LM head:
// [3, d] for a [V, d] head, [d, 8] (entries 0..2) for a [d, V] head.
__global__ void judge_split_kernel(const float *__restrict__ w, int d, int w_layout, __nv_bfloat16 *__restrict__ out) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= d) return;
    float r = w[k];
    __nv_bfloat16 b[JUDGE_FOLD_ROWS];
#pragma unroll
    for (int i = 0; i < JUDGE_FOLD_ROWS; i++) {
        b[i] = __float2bfloat16_rn(r);
        r -= __bfloat162float(b[i]);  // exact: the remainder has fewer significant bits than r
    }
#pragma unroll
    for (int i = 0; i < 8; i++) {
        const __nv_bfloat16 x = i < JUDGE_FOLD_ROWS ? b[i] : __float2bfloat16_rn(0.0f);
        if (w_layout)
            out[(size_t)k * 8 + i] = x;
        else if (i < JUDGE_FOLD_ROWS)
            out[(size_t)i * d + k] = x;
    }
}

}  // namespace

cudaError_t launch_judge_split(const float *w_target, int d, int w_layout, void *rows_out, cudaStream_t stream) {
    judge_split_kernel<<<(d + 255) / 256, 256, 0, stream>>>(w_target, d, w_layout, static_cast<__nv_bfloat16 *>(rows_out));
    return cudaGetLastError();
}

cudaError_t launch_judge_scan(const JudgeArgs &a, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)a.B);
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = (size_t)(4 * a.K + 1) * sizeof(int) + (size_t)a.K * SEGS * sizeof(float);
    if (cfg.dynamicSmemBytes > 48 * 1024) {
        // only the largest window (K = 1024) needs more than the default limit, by four bytes
        const cudaError_t e = cudaFuncSetAttribute(judge_scan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                   (int)cfg.dynamicSmemBytes);
        if (e != cudaSuccess) return e;
    }
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, judge_scan_kernel, a);
}

}  // namespace aj
