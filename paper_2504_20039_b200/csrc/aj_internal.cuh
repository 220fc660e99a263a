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

// Device status word values (mirrors aj_status where they overlap).
enum : int { DEV_OK = 0, DEV_TIMEOUT = 5 };

// ------------------------------------------------------------------------------ launchers

struct GemmArgs {
    const void *h;       // [M, d]
    const void *W;       // [V, d] or [d, V]
    int M, d, V;
    int dtype;           // 0 bf16, 1 f32
    int w_layout;        // 0 [V,d], 1 [d,V]
    unsigned long long *keys;  // [M], must be zero on entry (the judge kernel clears what it reads)
    int *status;
};

// CUDA-core projection + argmax (any dtype / layout).
cudaError_t launch_simt_gemm_argmax(const GemmArgs &a, int num_sms, cudaStream_t stream);

// tcgen05 projection + argmax (bf16, [V,d]).  `bn` is the vocabulary tile width (64, 128 or 256).
struct UmmaPlan {
    CUtensorMap tmap_h;  // rows of h, box 64 x 128, 128-byte swizzle
    CUtensorMap tmap_w;  // rows of W, box 64 x bn
    int bn;
    int grid;
};
cudaError_t umma_prepare();  // opt-in shared memory attributes; call once per device
cudaError_t launch_umma_gemm_argmax(const GemmArgs &a, const UmmaPlan &p, cudaStream_t stream);
const char *umma_path_name(int bn);

// tcgen05 projection + argmax with the vocabulary on the UMMA M axis (the default path).
// Here tmap_w has a 64 x 128 box and tmap_h a 64 x bn box, bn = vm_choose_bn(M) rows of h per tile.
int vm_choose_bn(int M);
cudaError_t umma_vm_prepare();
cudaError_t launch_umma_vm(const GemmArgs &a, const UmmaPlan &p, cudaStream_t stream);
const char *umma_vm_path_name(int bn);

// tcgen05 projection + argmax on CTA pairs (cta_group::2): 256 vocabulary entries x up to 256 rows
// per tile.  tmap_w has a 64 x 128 box, tmap_h a 64 x pair_schedule().box_rows box; p.grid = 2 *
// number of pairs.
struct PairSched {
    int n_v;               // blocks of 256 vocabulary entries
    int n_n;               // row tiles
    int u_base, u_rem;     // row tile i holds u_base + (i < u_rem) units of 16 rows
    int box_rows;          // rows of h each CTA of a pair stages per k-block
    int n_groups;          // row tiles are walked in groups ...
    int g_base, g_rem;     // ... group g holds g_base + (g < g_rem) row tiles
};
PairSched pair_schedule(int M, int V, int d);
cudaError_t umma_pair_prepare(int num_sms);
int umma_pair_max_pairs();
cudaError_t launch_umma_pair(const GemmArgs &a, const UmmaPlan &p, cudaStream_t stream);

struct JudgeArgs {
    unsigned long long *keys;        // [B*(K+1)]; read, then cleared for the next cycle
    const void *h_target;            // [B, K+1, d]
    const void *h_draft;             // [B, K+1, d_draft] or nullptr
    const int32_t *draft_tok;        // [B, K]
    const float *judge_w;            // [d_draft + d]
    float judge_b, tau;
    int B, K, d, d_draft, dtype;
    int32_t *accept_len, *next_tok, *target_tok;
    float *top1_val, *judge_p;
};
cudaError_t launch_judge_scan(const JudgeArgs &a, cudaStream_t stream);

}  // namespace aj
