// Internal declarations shared by the translation units of the CUDA library.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

namespace aj {

// ---------------------------------------------------------------- packed (max, argmax) key
//
// A row's best (logit, index) so far is one 64-bit word whose unsigned order is
// "larger logit first, then smaller index": the high half is the logit mapped to an
// order-preserving unsigned integer, the low half is ~index.  Merging partial results is
// then an integer max, which is associative and commutative, so the answer does not depend
// on how the vocabulary was split or in which order the pieces arrive.
__host__ __device__ inline uint32_t ordered_from_float(float x) {
    if (x == 0.0f) x = 0.0f;  // -0.0 becomes +0.0: the two zeros tie, the lower index then wins
#ifdef __CUDA_ARCH__
    uint32_t u = __float_as_uint(x);
#else
    uint32_t u;
    memcpy(&u, &x, 4);
#endif
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__host__ __device__ inline unsigned long long pack_key(float val, int idx) {
    return ((unsigned long long)ordered_from_float(val) << 32) | (uint32_t)(~(uint32_t)idx);
}

__device__ inline float key_value(unsigned long long key) {
    uint32_t u = (uint32_t)(key >> 32);
    u = (u & 0x80000000u) ? (u & 0x7FFFFFFFu) : ~u;
    return __uint_as_float(u);
}

__device__ inline int key_index(unsigned long long key) { return (int)(~(uint32_t)key); }

#ifdef __CUDACC__
// The high half of a key, branch-free, for the epilogues: an order-preserving map of a float onto
// unsigned integers in which the two zeros map to one value (equal to ordered_from_float).
__device__ inline uint32_t ordered_image(float x) {
    const uint32_t b = __float_as_uint(x + 0.0f);  // -0.0 + 0.0 = +0.0
    return b ^ ((uint32_t)((int32_t)b >> 31) | 0x80000000u);
}

// Maximum of x over the 32 lanes of the warp.
__device__ inline uint32_t warp_max_u32(uint32_t x) {
    uint32_t r;
    asm volatile("redux.sync.max.u32 %0, %1, 0xffffffff;" : "=r"(r) : "r"(x));
    return r;
}

// Minimum of x over the 32 lanes of the warp.
__device__ inline uint32_t warp_min_u32(uint32_t x) {
    uint32_t r;
    asm volatile("redux.sync.min.u32 %0, %1, 0xffffffff;" : "=r"(r) : "r"(x));
    return r;
}
#endif

// Device status word values (mirrors aj_status where they overlap).
enum : int { DEV_OK = 0, DEV_TIMEOUT = 5 };

// ------------------------------------------------------- vocabulary-parallel exchange of keys
//
// When the LM head is split by vocabulary over several GPUs, each GPU projects its own entries
// and the per-row keys of all GPUs are merged by the same 64-bit max.  The projection kernel does
// the exchange itself: the CTA that finishes last copies this GPU's keys into a slot of every
// GPU's exchange buffer (plain stores, over NVLink for the peers) and then stores the cycle's
// epoch into a flag in each of those buffers with release semantics.  The judge kernel of every
// GPU waits (bounded) until all flags of its own buffer show the epoch and takes the max over
// the slots.  Nothing is multicast and no kernel reads a peer's memory.
constexpr int MAX_SHARD_WORLD = 8;

struct Publish {
    int world = 0;                 // 0: the handle is not sharded, nothing is published
    int M = 0;
    unsigned long long epoch = 0;  // the value stored into the flags
    unsigned *done = nullptr;      // CTAs of this launch that have finished (wraps to zero by itself)
    unsigned long long *slot[MAX_SHARD_WORLD] = {};  // [M] in GPU g's buffer: where it wants this GPU's keys
    unsigned long long *flag[MAX_SHARD_WORLD] = {};  // in GPU g's buffer: where it wants this GPU's epoch
};

struct Gather {
    int world = 0;                              // 0: read and clear the handle's own keys
    int stride = 0;                             // rows per slot
    unsigned long long epoch = 0;
    const unsigned long long *slots = nullptr;  // [world][stride], in this GPU's buffer
    const unsigned long long *flags = nullptr;  // [world], in this GPU's buffer
};

#ifdef __CUDACC__
// Called by every thread of every CTA of a projection kernel once the CTA's own key updates have
// been issued.  The last CTA to arrive publishes the keys and clears them for the next cycle.
__device__ inline void publish_keys(const Publish &p, unsigned long long *keys) {
    if (p.world == 0) return;  // the same for the whole grid
    __shared__ int is_last;
    __threadfence();  // this thread's key updates are performed before its CTA is counted
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned total = gridDim.x * gridDim.y * gridDim.z;
        is_last = atomicInc(p.done, total - 1) == total - 1;
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    for (int j = threadIdx.x; j < p.M; j += blockDim.x) {
        const unsigned long long k = __ldcg(keys + j);
        keys[j] = 0ull;  // every CTA is done with them: leave the workspace clean
        for (int g = 0; g < p.world; g++) p.slot[g][j] = k;
    }
    __threadfence_system();
    __syncthreads();
    if ((int)threadIdx.x < p.world)
        asm volatile("st.release.sys.global.u64 [%0], %1;" ::"l"(p.flag[threadIdx.x]), "l"(p.epoch) : "memory");
}
#endif

// ------------------------------------------------------------------- top-K rule (rank counting)
//
// Under the top-K rule a mismatching draft token is accepted iff fewer than top_k vocabulary
// entries outrank it.  A small kernel first computes, per row, the draft token's own logit (the
// threshold); the projection kernels then also count, per row, the entries that outrank it
// (larger logit, or equal logit and lower index), and the judge kernel compares the count with top_k.
struct RankArgs {
    float *thr = nullptr;        // [M] the draft token's logit; +inf where the row has no draft token, and
                                 //     raised to +inf by the tensor-core kernels once top_k entries outrank it
    const int *tok = nullptr;    // [M] the draft token, -1 where there is none or it is outside the vocabulary
    unsigned *cnt = nullptr;     // [M] entries that outrank it (zeroed by the threshold kernel)
    int top_k = 0;               // the rule asks only whether fewer than top_k entries outrank the token
};

#ifdef __CUDACC__
// Epilogue add-on for the vocabulary-major kernels: the warp holds 32 consecutive vocabulary entries
// (lane = entry v_first + lane) of 32 columns (32 consecutive rows of h) in v[]; lane j is responsible
// for column j: `row` is its row of h, th / tk that row's threshold and draft token (+inf / -1 where the
// column is not a row of the batch), vmax the largest of this lane's 32 logits.
// A row whose count has reached top_k is settled (the rule only asks whether fewer than top_k entries
// outrank the token): its threshold is raised to +inf in global memory, so later tiles read that and leave
// it alone.  And a chunk none of whose logits reaches the lowest of its 32 thresholds is left after one
// reduction and one vote, which is nearly every chunk once the settled rows are out of the way.
__device__ inline float rank_threshold(const RankArgs &rk, int row, bool valid) {
    return valid ? __ldcg(rk.thr + row) : INFINITY;  // from L2: other SMs raise it while this kernel runs
}
__device__ inline void count_outranking(const RankArgs &rk, const float (&v)[32], float vmax, int v_first, bool v_ok, float th,
                                        int tk, int row, bool valid, int lane) {
    const uint32_t tmin = warp_min_u32(ordered_image(th));
    if (!__any_sync(0xffffffffu, v_ok && ordered_image(vmax) >= tmin)) return;
    const int vidx = v_first + lane;
    unsigned mine = 0;
#pragma unroll
    for (int j = 0; j < 32; j++) {
        const float t = __shfl_sync(0xffffffffu, th, j);
        const int k = __shfl_sync(0xffffffffu, tk, j);
        const bool ahead = v_ok && vidx != k && (v[j] > t || (v[j] == t && vidx < k));
        const unsigned b = __ballot_sync(0xffffffffu, ahead);
        if (lane == j) mine = __popc(b);
    }
    if (valid && mine) {
        const unsigned before = atomicAdd(rk.cnt + row, mine);
        if (before < (unsigned)rk.top_k && before + mine >= (unsigned)rk.top_k) rk.thr[row] = INFINITY;
    }
}
#endif

// ------------------------------------------------------- sampling by the Gumbel-max trick
//
// With a temperature T > 0 the target's token of a row is argmax_v (logit[v] + T * g[v]) with g
// standard Gumbel noise, which draws from softmax(logit / T); the noise is a deterministic
// function of (seed, cycle counter, row, vocabulary entry), so that a draw can be reproduced and
// does not depend on how the work was tiled or sharded.  For row j and entry v: x = word (j mod 4)
// of Philox4x32-10 with key (seed low, seed high) and counter (v, j div 4, step low, step high);
// u = ((x >> 9) + 0.5) * 2^-23 (exact in fp32, never 0 or 1); g = -ln(-ln u).
struct Noise {
    float temperature = 0.0f;  // 0: greedy, no noise
    float inv_temperature = 0.0f;
    uint32_t key0 = 0, key1 = 0;    // seed
    uint32_t step0 = 0, step1 = 0;  // cycle counter
};

#ifdef __CUDACC__
__device__ inline void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1,
                                     uint32_t (&out)[4]) {
#pragma unroll
    for (int r = 0; r < 10; r++) {
        const unsigned long long p0 = (unsigned long long)0xD2511F53u * c0;  // one wide multiply gives both halves
        const unsigned long long p1 = (unsigned long long)0xCD9E8D57u * c2;
        c0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        c1 = (uint32_t)p1;
        c2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        c3 = (uint32_t)p0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0;
    out[1] = c1;
    out[2] = c2;
    out[3] = c3;
}

// lg2(-ln u) for u = (k + 0.5) * 2^-23, k = x >> 9; the Gumbel noise is g = -ln 2 * that, to about
// 2e-6 absolute.  Built on the hardware's base-2 logarithm, whose absolute error (about 2e-7 on the
// logarithm of the mantissa) is not enough for -ln u where u is close to 1, which is where the
// largest noise values, the ones that win, come from: for t = 1 - u <= 1/16 (exact in fp32) the
// series t + t^2/2 + ... + t^6/6 is used instead (the first term left out is below 1e-8 relative).
// No integer-to-float conversion, no division, no branch: u is assembled from the bits.
__device__ inline float lg2_approx(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ inline float lg2_neg_ln_uniform(uint32_t x) {
    const float f = __uint_as_float(0x3F800000u | (x >> 9));  // 1 + k 2^-23
    const float u = f - __uint_as_float(0x3F7FFFFFu);         // minus (1 - 2^-24): (k + 0.5) 2^-23, exact
    const float t = 1.0f - u;                                 // exact
    const float near_one =
        t * fmaf(t, fmaf(t, fmaf(t, fmaf(t, fmaf(t, 1.0f / 6.0f, 0.2f), 0.25f), 1.0f / 3.0f), 0.5f), 1.0f);
    const float far = -0.693147180559945f * lg2_approx(u);
    return lg2_approx(t <= 0.0625f ? near_one : far);
}

__device__ inline float gumbel_from_bits(uint32_t x) { return -0.693147180559945f * lg2_neg_ln_uniform(x); }

// The noisy score of one element.
__device__ inline float noisy_score(const Noise &nz, float logit, int row, int v) {
    uint32_t w[4];
    philox4x32_10((uint32_t)v, (uint32_t)(row >> 2), nz.step0, nz.step1, nz.key0, nz.key1, w);
    const uint32_t x = (row & 2) ? ((row & 1) ? w[3] : w[2]) : ((row & 1) ? w[1] : w[0]);
    return fmaf(nz.temperature * -0.693147180559945f, lg2_neg_ln_uniform(x), logit);
}

// Which draws can matter.  A thread holds 32 logits of one vocabulary entry, none above vmax, and the rows
// they belong to have each a best noisy score so far, none below `lowest`: an element can only take its
// row over if its noise is at least need = (lowest - vmax) / T.  The noise grows with the random word, so
// that is a cutoff on the word's upper 23 bits: k >= u(need) 2^23 with u(g) = exp(-exp(-g)), taken with a
// margin (need lowered by 2e-3, 16 counts off) that covers the approximate exponentials.  0: every draw
// may matter (no row has a score yet, or need is small); that is also the answer to a NaN.
__device__ inline float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ inline uint32_t noise_cutoff(float lowest, float vmax, float inv_temperature) {
    const float need = (lowest - vmax) * inv_temperature - 2e-3f;
    if (!(need > -3.0f)) return 0u;
    const float e = ex2_approx(-1.4426950408889634f * need);  // exp(-need) <= e^3
    const float u = ex2_approx(-1.4426950408889634f * e);
    const float k = u * 8388608.0f - 16.0f;
    return k > 0.0f ? (uint32_t)k : 0u;
}

// Epilogue add-on for the vocabulary-major kernels: this thread holds entry v of the 32 rows
// row_first .. + 32 (row_first a multiple of 4) in x[]; one Philox call serves four rows.  Every word
// is drawn (the eight generator calls of a chunk back to back, so that their multiply chains overlap); the
// two logarithms are only taken of the words that reach k_need (see noise_cutoff), the other elements
// cannot take their row over and become -inf.  False: no element of the warp's chunk can matter and x[] is
// left as it was.  The whole warp must call this together.
__device__ inline bool add_gumbel_noise(const Noise &nz, float (&x)[32], int v, int row_first, uint32_t k_need) {
    const float scale = nz.temperature * -0.693147180559945f;
    uint32_t w[32];
#pragma unroll
    for (int q = 0; q < 8; q++) {
        uint32_t o[4];
        philox4x32_10((uint32_t)v, (uint32_t)((row_first >> 2) + q), nz.step0, nz.step1, nz.key0, nz.key1, o);
        w[4 * q + 0] = o[0], w[4 * q + 1] = o[1], w[4 * q + 2] = o[2], w[4 * q + 3] = o[3];
    }
    uint32_t top = w[0];
#pragma unroll
    for (int i = 1; i < 32; i++) top = w[i] > top ? w[i] : top;
    if (!__any_sync(0xffffffffu, (top >> 9) >= k_need)) return false;  // one decision per warp: a real branch
#pragma unroll
    for (int q = 0; q < 8; q++) {
        const bool c0 = (w[4 * q] >> 9) >= k_need, c1 = (w[4 * q + 1] >> 9) >= k_need, c2 = (w[4 * q + 2] >> 9) >= k_need,
                   c3 = (w[4 * q + 3] >> 9) >= k_need;
        if (__any_sync(0xffffffffu, c0 || c1 || c2 || c3)) {
            x[4 * q + 0] = c0 ? fmaf(scale, lg2_neg_ln_uniform(w[4 * q + 0]), x[4 * q + 0]) : -INFINITY;
            x[4 * q + 1] = c1 ? fmaf(scale, lg2_neg_ln_uniform(w[4 * q + 1]), x[4 * q + 1]) : -INFINITY;
            x[4 * q + 2] = c2 ? fmaf(scale, lg2_neg_ln_uniform(w[4 * q + 2]), x[4 * q + 2]) : -INFINITY;
            x[4 * q + 3] = c3 ? fmaf(scale, lg2_neg_ln_uniform(w[4 * q + 3]), x[4 * q + 3]) : -INFINITY;
        } else {
            x[4 * q + 0] = x[4 * q + 1] = x[4 * q + 2] = x[4 * q + 3] = -INFINITY;
        }
    }
    return true;
}
#endif

// ------------------------------------------------ the classifier's target half as rows of the LM head
//
// z = b + w_draft . h_draft[row] + w_target . h_target[row]: the second dot product has the shape of
// one more logit.  When it is folded into the projection, w_target is appended to the vocabulary as
// THREE bf16 rows whose sum is w_target to fp32 precision (w = b0 + b1 + b2, each the bf16 rounding of
// what the previous ones leave), in one extra vocabulary block that follows the real ones.  Its
// entries lie past V, so they never enter the argmax; the epilogue stores the three partial dot
// products of every row to parts[3][stride] and the scan kernel adds them in a fixed order.
struct JudgeFold {
    const void *rows = nullptr;  // bf16, laid out like W_lm: [3, d], or [d, 8] (3 of 8 entries used); nullptr: not folded
    float *parts = nullptr;      // [3][stride]
    int stride = 0;
};
constexpr int JUDGE_FOLD_ROWS = 3;
cudaError_t launch_judge_split(const float *w_target, int d, int w_layout, void *rows_out, cudaStream_t stream);

struct RankPrepArgs {
    const void *h;             // [M, d]
    const void *W;             // LM head
    const int32_t *draft_tok;  // [B, K]
    int B, K, R, d, V, dtype, w_layout;
    float *thr;
    int *tok;
    unsigned *cnt;
};
cudaError_t launch_rank_prepare(const RankPrepArgs &a, cudaStream_t stream);

// ------------------------------------------------------------------------------ launchers

struct GemmArgs {
    const void *h;       // [M, d]
    const void *W;       // [V, d] or [d, V]; V entries starting at vocabulary index v_offset
    int M, d, V;
    int v_offset = 0;    // added to every index stored in a key (vocabulary-parallel shards)
    int dtype;           // 0 bf16, 1 f32
    int w_layout;        // 0 [V,d], 1 [d,V]
    unsigned long long *keys;  // [M], must be zero on entry (the judge kernel clears what it reads)
    int *status;
    Publish pub;
    RankArgs rank;       // thr != nullptr: also count, per row, the entries that outrank the draft token
    Noise noise;         // temperature > 0: the argmax is taken over logit + temperature * Gumbel noise
    JudgeFold fold;      // rows != nullptr: one more vocabulary block computes the classifier's target half
    // Two words, zero between launches, through which the CTA pairs of the two-SM kernel share out their
    // tiles as they become free (a tile counter and a count of the pairs that are done with it);
    // nullptr: every pair takes the tiles pair, pair + pairs, ... in a fixed order.
    unsigned *sched = nullptr;
};

// What a projection kernel's epilogue does besides the argmax.
enum : int { EPI_PLAIN = 0, EPI_COUNT = 1, EPI_SAMPLE = 2 };

// CUDA-core projection + argmax (any dtype / layout).
cudaError_t launch_simt_gemm_argmax(const GemmArgs &a, int num_sms, cudaStream_t stream);

// tcgen05 projection + argmax (bf16), vocabulary on the UMMA M axis, one SM per tile.
struct UmmaPlan {
    CUtensorMap tmap_h;  // rows of h, 128-byte swizzle
    CUtensorMap tmap_w;  // rows of W (or, for [d, V], 64 entries x 64 k-rows)
    CUtensorMap tmap_j;  // the folded classifier rows, same box as tmap_w (only with GemmArgs::fold)
    int bn;              // rows of h per tile
    int grid;
};
// tmap_w has a 64 x 128 box and tmap_h a 64 x vm_box_rows(M, bn) box, bn = vm_choose_bn(M) rows of h per tile.
int vm_choose_bn(int M);
int vm_box_rows(int M, int bn);
cudaError_t umma_vm_prepare();
cudaError_t launch_umma_vm(const GemmArgs &a, const UmmaPlan &p, cudaStream_t stream);
const char *umma_vm_path_name(int bn);

// tcgen05 projection + argmax on CTA pairs (cta_group::2): 256 vocabulary entries x up to 256 rows
// per tile.  tmap_w has a 64 x 128 box, tmap_h a 64 x pair_schedule().box_rows box; p.grid = 2 *
// number of pairs.
struct PairSched {
    int n_v;               // blocks of 256 vocabulary entries, the block of the folded classifier rows included
    int fold;              // 1: the last block holds the classifier rows instead of vocabulary entries
    int n_n;               // row tiles
    int u_base, u_rem;     // row tile i holds u_base + (i < u_rem) units of 16 rows
    int box_rows;          // rows of h each CTA of a pair stages per k-block and accumulator
    int dual;              // 1: every tile uses two accumulators that share the staged block of W
    int stages;            // depth of the shared-memory ring
    int kps;               // k-blocks of 64 per stage (1 or 2)
    int n_groups;          // row tiles are walked in groups ...
    int g_base, g_rem;     // ... group g holds g_base + (g < g_rem) row tiles
};
PairSched pair_schedule(int M, int V, int d, int fold);
cudaError_t umma_pair_prepare(int num_sms);
int umma_pair_max_pairs();
cudaError_t launch_umma_pair(const GemmArgs &a, const UmmaPlan &p, cudaStream_t stream);

struct JudgeArgs {
    unsigned long long *keys;        // [B*(K+1)]; read, then cleared for the next cycle (unless gathered)
    Gather gather;                   // vocabulary-parallel: where the merged keys come from
    int *status = nullptr;           // device status word (set when a bounded wait runs out)
    const void *h_target;            // [B, K+1, d]
    const void *h_draft;             // [B, K+1, d_draft] or nullptr
    const int32_t *draft_tok;        // [B, K]
    const float *judge_w;            // [d_draft + d]
    float judge_b, tau;
    int B, K, d, d_draft, dtype;
    int no_extra_row = 0;            // 1: K rows per sequence instead of K + 1
    int top_k = 0;                   // > 0: the top-K rule replaces the classifier
    int V = 0;                       // vocabulary size (top-K rule: ids outside it are never accepted)
    unsigned *rank_cnt = nullptr;    // [B*R] counts from the projection kernel (top-K rule)
    const float *fold_parts = nullptr;  // [3][fold_stride] the target half of the classifier from the projection kernel, else nullptr
    int fold_stride = 0;
    const int32_t *parent = nullptr; // [B, K] tree drafts: parent node of every node (-1 = the root), else nullptr
    int32_t *best_node = nullptr;    // [B] tree drafts: the deepest accepted node (-1 = the root), optional
    int32_t *accept_len, *next_tok, *target_tok;
    float *top1_val, *judge_p;
};
cudaError_t launch_judge_scan(const JudgeArgs &a, cudaStream_t stream);

}  // namespace aj
