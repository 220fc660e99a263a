// Host side of the C-ABI: argument checks, workspace, tensor maps, stream-ordered launches.
// One cycle = projection + argmax kernel, then judge + scan kernel as its programmatic dependent;
// no host synchronisation and no allocation inside aj_verify.  The per-row keys start at zero
// (cleared at creation) and the judge kernel clears each key as it reads it, so a cycle needs no
// separate clearing pass; only after a launch failed half-way are they cleared explicitly.
#include "../../include/aj_verify.h"
#include "aj_internal.cuh"

#include <new>

namespace {

using namespace aj;

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TmapSlot {
    const void *ptr = nullptr;
    long long rows = 0;
    int box_rows = 0;  // -1: a [d, rows] map, W_lm stored [d, V] (64 entries x 64 k-rows per box)
    unsigned long long stamp = 0;
    CUtensorMap map;
};

constexpr int TMAP_SLOTS = 8;
constexpr int EVENT_RING = 512;

}  // namespace

struct aj_handle_s {
    int device = 0;
    int max_B = 0, max_K = 0, d = 0, d_draft = 0, V = 0;
    int dtype = 0, layout = 0;
    unsigned flags = 0;
    int num_sms = 0;
    bool umma_ok = false;
    bool pair_ok = false;  // the two-SM kernel can be launched on this device
    unsigned long long *keys = nullptr;
    bool keys_dirty = false;  // a cycle was started but its judge kernel was not enqueued
    int *status = nullptr;
    // staging for aj_verify_host
    void *st_ht = nullptr, *st_hd = nullptr;
    int32_t *st_tok = nullptr, *st_acc = nullptr, *st_next = nullptr, *st_tt = nullptr;
    EncodeTiledFn encode = nullptr;
    TmapSlot slots[TMAP_SLOTS];
    unsigned long long stamp = 0;
    cudaEvent_t ev0[EVENT_RING] = {}, ev1[EVENT_RING] = {};  // with AJ_FLAG_TIME_KERNELS
    long long n_timed = 0;                                   // calls recorded since the last read-out
    int last_launches = 0;
    const char *last_path = "none";
    // vocabulary-parallel handles (aj_create_sharded)
    int world = 0, rank = 0;         // world == 0: the handle holds the whole LM head
    int v_begin = 0, v_count = 0;    // this GPU's vocabulary entries
    unsigned long long *exchange[MAX_SHARD_WORLD] = {};  // every GPU's exchange buffer, as mapped on this device
    unsigned long long epoch = 0;    // cycles started; the same on every rank, which call in step
    bool projected = false;          // aj_shard_project was enqueued and its aj_shard_finish is still due
    // top-K rule (aj_set_top_k)
    int top_k = 0;                   // 0: the classifier decides
    // sampled verification (aj_set_sampling)
    float temperature = 0.0f;        // 0: greedy
    unsigned long long seed = 0, step = 0;
    float *rk_thr = nullptr;         // [max_M] the draft tokens' own logits
    int *rk_tok = nullptr;           // [max_M]
    unsigned *rk_cnt = nullptr;      // [max_M] entries that outrank them
    // the classifier's target half folded into the projection (aj_fuse_judge)
    bool fold = false;
    void *fold_rows = nullptr;       // three bf16 rows that add up to w_target, laid out like W_lm
    float *fold_parts = nullptr;     // [3][max_M] their dot products with every row of h_target
};

// Exchange buffer of one GPU: 256 bytes of flags (one 8-byte epoch per source GPU), then two slot
// arrays (one per epoch parity) of world x max_M keys.
constexpr size_t EXCHANGE_FLAG_BYTES = 256;

namespace {

size_t elem_size(int dtype) { return dtype == AJ_BF16 ? 2 : 4; }

class DeviceGuard {
   public:
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev_) != cudaSuccess) prev_ = -1;
        if (prev_ != dev) ok_ = cudaSetDevice(dev) == cudaSuccess;
        changed_ = ok_ && prev_ != dev;
    }
    ~DeviceGuard() {
        if (changed_ && prev_ >= 0) cudaSetDevice(prev_);
    }
    bool ok() const { return ok_; }

   private:
    int prev_ = -1;
    bool ok_ = true, changed_ = false;
};

// A tensor map over `rows` rows of `d` bf16 elements, box 64 columns x box_rows rows, 128-byte
// swizzle; rows past the end read as zero.  Cached per (pointer, rows, box).
const CUtensorMap *get_tmap(aj_handle h, const void *ptr, long long rows, int box_rows) {
    TmapSlot *victim = &h->slots[0];
    for (auto &s : h->slots) {
        if (s.ptr == ptr && s.rows == rows && s.box_rows == box_rows) {
            s.stamp = ++h->stamp;
            return &s.map;
        }
        if (s.stamp < victim->stamp) victim = &s;
    }
    cuuint64_t dims[2] = {(cuuint64_t)h->d, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)h->d * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    if (box_rows < 0) {  // W_lm stored [d, V]: `rows` vocabulary entries are the inner dimension
        dims[0] = (cuuint64_t)rows;
        dims[1] = (cuuint64_t)h->d;
        strides[0] = (cuuint64_t)rows * 2;
        box[1] = 64;
    }
    cuuint32_t estr[2] = {1, 1};
    CUresult r = h->encode(&victim->map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box,
                           estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        victim->ptr = nullptr;
        return nullptr;
    }
    victim->ptr = ptr;
    victim->rows = rows;
    victim->box_rows = box_rows;
    victim->stamp = ++h->stamp;
    return &victim->map;
}

// Batches with more rows than this run on the two-SM kernel; smaller ones are bound by the W_lm
// stream from HBM and keep the one-SM kernel, which has more loads in flight per SM.
constexpr int PAIR_MIN_ROWS = 128;

aj_status check_call(aj_handle h, const void *h_target, const void *h_draft, const void *W_lm, const int32_t *draft_tok,
                     const float *judge_w, int B, int K, int d, int V, const int32_t *accept_len,
                     const int32_t *next_tok) {
    if (!h) return AJ_ERR_INVALID_ARG;
    if (!h_target || !W_lm || !draft_tok || !accept_len || !next_tok) return AJ_ERR_INVALID_ARG;
    if (h->top_k == 0) {  // the classifier's operands are needed unless the top-K rule is in force
        if (!judge_w || (h->d_draft > 0) != (h_draft != nullptr)) return AJ_ERR_INVALID_ARG;
    }
    if (B < 1 || K < 1 || d != h->d || V != h->V) return AJ_ERR_INVALID_ARG;
    if (B > h->max_B || K > h->max_K) return AJ_ERR_WORKSPACE;
    return AJ_OK;
}

// rows of hidden states per sequence: the last accepted token and the K draft tokens, or without
// the last draft token when the caller does not encode it
int rows_per_seq(aj_handle h, int K) { return (h->flags & AJ_FLAG_NO_EXTRA_ROW) ? K : K + 1; }

// The address at which the current device can read and write a HOST buffer directly, or nullptr
// if the buffer is ordinary pageable memory (then it has to be copied).
void *device_view(const void *host_ptr) {
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, host_ptr) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    return attr.type == cudaMemoryTypeHost ? attr.devicePointer : nullptr;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// Brings one cycle's hidden states from pinned host memory into the handle's staging buffers: every
// thread fetches 16-byte pieces over PCIe (all of a small batch's pieces are in flight at once).  For the
// few hundred KB of a small batch this takes less than two copy operations do, and the projection
// kernel, launched as a programmatic dependent, sets itself up meanwhile.
__global__ void stage_hidden_kernel(const uint4 *__restrict__ a_src, uint4 *__restrict__ a_dst, unsigned n_a,
                                    const uint4 *__restrict__ b_src, uint4 *__restrict__ b_dst, unsigned n_b) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const unsigned stride = gridDim.x * blockDim.x;
    for (unsigned i = blockIdx.x * blockDim.x + threadIdx.x; i < n_a + n_b; i += stride) {
        // the host rewrites these buffers between cycles: never a cached copy
        if (i < n_a)
            a_dst[i] = __ldcv(a_src + i);
        else
            b_dst[i - n_a] = __ldcv(b_src + (i - n_a));
    }
}
constexpr size_t STAGE_KERNEL_MAX_BYTES = 1u << 20;  // above this the copy engines are at least as fast

}  // namespace

extern "C" {

const char *aj_version(void) { return "aj_verify 0.1 (sm_100a)"; }

const char *aj_status_string(aj_status s) {
    switch (s) {
        case AJ_OK: return "ok";
        case AJ_ERR_INVALID_ARG: return "invalid argument";
        case AJ_ERR_UNSUPPORTED: return "unsupported configuration";
        case AJ_ERR_WORKSPACE: return "batch or window exceeds the handle's workspace";
        case AJ_ERR_CUDA: return "CUDA call failed";
        case AJ_ERR_TIMEOUT: return "a bounded wait in a kernel ran out";
        case AJ_ERR_NOT_SM100: return "device is not compute capability 10.x";
    }
    return "unknown status";
}

aj_status aj_create(aj_handle *out, int device, int max_B, int max_K, int d, int d_draft, int V, aj_dtype dtype,
                    aj_w_layout layout, unsigned flags) {
    if (!out) return AJ_ERR_INVALID_ARG;
    *out = nullptr;
    if (device < 0 || max_B < 1 || max_K < 1 || max_K > 1024 || d < 1 || d_draft < 0 || V < 1) return AJ_ERR_INVALID_ARG;
    if (dtype != AJ_BF16 && dtype != AJ_F32) return AJ_ERR_INVALID_ARG;
    if (layout != AJ_W_VD && layout != AJ_W_DV) return AJ_ERR_INVALID_ARG;
    if (flags & ~(AJ_FLAG_FORCE_SIMT | AJ_FLAG_TIME_KERNELS | AJ_FLAG_ONE_SM | AJ_FLAG_NO_EXTRA_ROW))
        return AJ_ERR_INVALID_ARG;
    if ((long long)max_B * (max_K + 1) > (1ll << 24)) return AJ_ERR_INVALID_ARG;
    if (dtype == AJ_BF16 && (d % 8 != 0 || d_draft % 8 != 0)) return AJ_ERR_UNSUPPORTED;

    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device >= count) {
        cudaGetLastError();
        return AJ_ERR_CUDA;
    }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return AJ_ERR_CUDA;
    if (prop.major != 10) return AJ_ERR_NOT_SM100;
    DeviceGuard guard(device);
    if (!guard.ok()) return AJ_ERR_CUDA;

    aj_handle h = new (std::nothrow) aj_handle_s;
    if (!h) return AJ_ERR_CUDA;
    h->device = device;
    h->max_B = max_B;
    h->max_K = max_K;
    h->d = d;
    h->d_draft = d_draft;
    h->V = V;
    h->dtype = dtype;
    h->layout = layout;
    h->flags = flags;
    h->num_sms = prop.multiProcessorCount;
    // tensor-core path: bf16, d a multiple of 64; W_lm as [V, d], or as [d, V] with a row pitch that
    // TMA accepts (a multiple of 16 bytes) on the vocabulary-major kernels
    h->umma_ok = dtype == AJ_BF16 && d % 64 == 0 && !(flags & AJ_FLAG_FORCE_SIMT) &&
                 (layout == AJ_W_VD || V % 8 == 0);

    const size_t max_M = (size_t)max_B * (max_K + 1);
    const size_t esz = elem_size(dtype);
    bool ok = cudaMalloc(&h->keys, max_M * sizeof(unsigned long long)) == cudaSuccess &&
              cudaMemset(h->keys, 0, max_M * sizeof(unsigned long long)) == cudaSuccess &&
              cudaMalloc(&h->status, 256) == cudaSuccess && cudaMemset(h->status, 0, 256) == cudaSuccess &&
              cudaMalloc(&h->st_ht, max_M * d * esz) == cudaSuccess &&
              (d_draft == 0 || cudaMalloc(&h->st_hd, max_M * d_draft * esz) == cudaSuccess) &&
              cudaMalloc(&h->st_tok, (size_t)max_B * max_K * 4) == cudaSuccess &&
              cudaMalloc(&h->st_acc, (size_t)max_B * 4) == cudaSuccess &&
              cudaMalloc(&h->st_next, (size_t)max_B * 4) == cudaSuccess && cudaMalloc(&h->st_tt, max_M * 4) == cudaSuccess &&
              cudaMalloc(&h->rk_thr, max_M * 4) == cudaSuccess && cudaMalloc(&h->rk_tok, max_M * 4) == cudaSuccess &&
              cudaMalloc(&h->rk_cnt, max_M * 4) == cudaSuccess &&
              cudaMalloc(&h->fold_rows, (size_t)8 * d * 2) == cudaSuccess &&
              cudaMalloc(&h->fold_parts, (size_t)JUDGE_FOLD_ROWS * max_M * 4) == cudaSuccess;
    if (ok && (flags & AJ_FLAG_TIME_KERNELS))
        for (int i = 0; ok && i < EVENT_RING; i++)
            ok = cudaEventCreate(&h->ev0[i]) == cudaSuccess && cudaEventCreate(&h->ev1[i]) == cudaSuccess;
    if (ok && h->umma_ok) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        ok = cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres) == cudaSuccess &&
             qres == cudaDriverEntryPointSuccess && fn != nullptr;
        h->encode = reinterpret_cast<EncodeTiledFn>(fn);
        if (ok) ok = umma_vm_prepare() == cudaSuccess;
        if (ok) h->pair_ok = umma_pair_prepare(h->num_sms) == cudaSuccess && umma_pair_max_pairs() > 0;
        if (!h->pair_ok) cudaGetLastError();  // no room for CTA pairs: the one-SM kernel serves every batch
    }
    if (!ok) {
        cudaGetLastError();
        aj_destroy(h);
        return AJ_ERR_CUDA;
    }
    *out = h;
    return AJ_OK;
}

aj_status aj_destroy(aj_handle h) {
    if (!h) return AJ_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    cudaFree(h->keys);
    cudaFree(h->status);
    cudaFree(h->st_ht);
    cudaFree(h->st_hd);
    cudaFree(h->st_tok);
    cudaFree(h->st_acc);
    cudaFree(h->st_next);
    cudaFree(h->st_tt);
    cudaFree(h->rk_thr);
    cudaFree(h->rk_tok);
    cudaFree(h->rk_cnt);
    cudaFree(h->fold_rows);
    cudaFree(h->fold_parts);
    for (int i = 0; i < EVENT_RING; i++) {
        if (h->ev0[i]) cudaEventDestroy(h->ev0[i]);
        if (h->ev1[i]) cudaEventDestroy(h->ev1[i]);
    }
    delete h;
    return AJ_OK;
}

// Enqueue the projection + argmax kernel of one cycle (and, on a sharded handle, its exchange).
static aj_status enqueue_project(aj_handle h, const void *h_target, const void *W_lm, const int32_t *draft_tok, int B, int K,
                                 cudaStream_t stream) {
    const int M = B * rows_per_seq(h, K);
    const int d = h->d;
    const int V = h->world ? h->v_count : h->V;  // vocabulary entries this GPU projects
    h->last_launches = 0;

    if (h->keys_dirty) {
        const size_t all = (size_t)h->max_B * (h->max_K + 1) * sizeof(unsigned long long);
        if (cudaMemsetAsync(h->keys, 0, all, stream) != cudaSuccess) return AJ_ERR_CUDA;
        // (and the two-SM kernel's tile counter, which a cycle that gave up may not have put back)
        if (cudaMemsetAsync(reinterpret_cast<unsigned *>(h->status) + 32, 0, 2 * sizeof(unsigned), stream) != cudaSuccess) return AJ_ERR_CUDA;
    }
    h->keys_dirty = true;

    GemmArgs g;
    if (h->top_k > 0) {
        // top-K rule: the draft tokens' own logits first; the projection kernel counts against them
        RankPrepArgs r;
        r.h = h_target;
        r.W = W_lm;
        r.draft_tok = draft_tok;
        r.B = B;
        r.K = K;
        r.R = rows_per_seq(h, K);
        r.d = d;
        r.V = V;
        r.dtype = h->dtype;
        r.w_layout = h->layout;
        r.thr = h->rk_thr;
        r.tok = h->rk_tok;
        r.cnt = h->rk_cnt;
        if (launch_rank_prepare(r, stream) != cudaSuccess) return AJ_ERR_CUDA;
        h->last_launches++;
        g.rank.thr = h->rk_thr;
        g.rank.tok = h->rk_tok;
        g.rank.cnt = h->rk_cnt;
        g.rank.top_k = h->top_k;
    }
    if (h->temperature > 0.0f) {
        g.noise.temperature = h->temperature;
        g.noise.inv_temperature = 1.0f / h->temperature;
        g.noise.key0 = (uint32_t)h->seed;
        g.noise.key1 = (uint32_t)(h->seed >> 32);
        g.noise.step0 = (uint32_t)h->step;
        g.noise.step1 = (uint32_t)(h->step >> 32);
        ++h->step;
    }
    g.h = h_target;
    g.W = W_lm;
    g.M = M;
    g.d = d;
    g.V = V;
    g.v_offset = h->world ? h->v_begin : 0;
    g.dtype = h->dtype;
    g.w_layout = h->layout;
    g.keys = h->keys;
    g.status = h->status;
    g.sched = reinterpret_cast<unsigned *>(h->status) + 32;  // zeroed with the status block; the kernel leaves it zero
    const bool fold = h->fold && h->umma_ok && h->top_k == 0;  // the top-K rule does not consult the classifier
    if (fold) {
        g.fold.rows = h->fold_rows;
        g.fold.parts = h->fold_parts;
        g.fold.stride = h->max_B * (h->max_K + 1);
    }
    if (h->world) {
        ++h->epoch;
        const size_t max_M = (size_t)h->max_B * (h->max_K + 1);
        g.pub.world = h->world;
        g.pub.M = M;
        g.pub.epoch = h->epoch;
        g.pub.done = reinterpret_cast<unsigned *>(h->status) + 16;
        for (int r = 0; r < h->world; r++) {
            unsigned long long *buf = h->exchange[r];
            g.pub.flag[r] = buf + h->rank;
            g.pub.slot[r] = buf + EXCHANGE_FLAG_BYTES / 8 + ((h->epoch & 1) * h->world + h->rank) * max_M;
        }
    }

    const bool time_it = (h->flags & AJ_FLAG_TIME_KERNELS) != 0;
    const int slot = (int)(h->n_timed % EVENT_RING);
    if (time_it && cudaEventRecord(h->ev0[slot], stream) != cudaSuccess) return AJ_ERR_CUDA;
    cudaError_t e;
    if (h->umma_ok && h->pair_ok && M > PAIR_MIN_ROWS && !(h->flags & AJ_FLAG_ONE_SM)) {
        // tensor-bound regime: two-SM tiles of 256 vocabulary entries x up to 256 rows
        UmmaPlan p;
        p.bn = 256;
        const PairSched sc = pair_schedule(M, V, d, fold);
        const CUtensorMap *tw = get_tmap(h, W_lm, V, h->layout == AJ_W_DV ? -1 : 128);
        const CUtensorMap *th = get_tmap(h, h_target, M, sc.box_rows);
        const CUtensorMap *tj = fold ? get_tmap(h, h->fold_rows, h->layout == AJ_W_DV ? 8 : JUDGE_FOLD_ROWS, h->layout == AJ_W_DV ? -1 : 128) : tw;
        if (!th || !tw || !tj) return AJ_ERR_CUDA;
        p.tmap_h = *th;
        p.tmap_w = *tw;
        p.tmap_j = *tj;
        const long long tiles = (long long)sc.n_n * sc.n_v;
        const int pairs = umma_pair_max_pairs();
        p.grid = 2 * (int)(tiles < pairs ? tiles : pairs);
        e = launch_umma_pair(g, p, stream);
        h->last_path = "umma_pair_256x256";
    } else if (h->umma_ok) {
        UmmaPlan p;
        p.bn = vm_choose_bn(M);
        const CUtensorMap *tw = get_tmap(h, W_lm, V, h->layout == AJ_W_DV ? -1 : 128);
        const CUtensorMap *th = get_tmap(h, h_target, M, vm_box_rows(M, p.bn));
        const CUtensorMap *tj = fold ? get_tmap(h, h->fold_rows, h->layout == AJ_W_DV ? 8 : JUDGE_FOLD_ROWS, h->layout == AJ_W_DV ? -1 : 128) : tw;
        if (!th || !tw || !tj) return AJ_ERR_CUDA;
        p.tmap_h = *th;
        p.tmap_w = *tw;
        p.tmap_j = *tj;
        const long long tiles = (long long)((M + p.bn - 1) / p.bn) * ((V + 127) / 128 + (fold ? 1 : 0));
        p.grid = (int)(tiles < h->num_sms ? tiles : h->num_sms);
        e = launch_umma_vm(g, p, stream);
        h->last_path = umma_vm_path_name(p.bn);
    } else {
        e = launch_simt_gemm_argmax(g, h->num_sms, stream);
        h->last_path = "simt";
    }
    if (e != cudaSuccess) return AJ_ERR_CUDA;
    h->last_launches++;
    if (time_it) {
        if (cudaEventRecord(h->ev1[slot], stream) != cudaSuccess) return AJ_ERR_CUDA;
        h->n_timed++;
    }

    return AJ_OK;
}

// Enqueue the judge + prefix-scan kernel of the cycle whose projection was enqueued last.
static aj_status enqueue_finish(aj_handle h, const void *h_target, const void *h_draft, const int32_t *draft_tok,
                                const float *judge_w, float judge_b, float tau, int B, int K, int32_t *accept_len,
                                int32_t *next_tok, int32_t *target_tok, float *top1_val, float *judge_p,
                                cudaStream_t stream, const int32_t *parent = nullptr, int32_t *best_node = nullptr) {
    JudgeArgs j;
    j.parent = parent;
    j.best_node = best_node;
    j.keys = h->keys;
    j.status = h->status;
    if (h->world) {
        const size_t max_M = (size_t)h->max_B * (h->max_K + 1);
        const unsigned long long *own = h->exchange[h->rank];
        j.gather.world = h->world;
        j.gather.stride = (int)max_M;
        j.gather.epoch = h->epoch;
        j.gather.flags = own;
        j.gather.slots = own + EXCHANGE_FLAG_BYTES / 8 + (h->epoch & 1) * h->world * max_M;
    }
    j.h_target = h_target;
    j.h_draft = h_draft;
    j.draft_tok = draft_tok;
    j.judge_w = judge_w;
    j.judge_b = judge_b;
    j.tau = tau;
    j.B = B;
    j.K = K;
    j.d = h->d;
    j.d_draft = h->d_draft;
    j.dtype = h->dtype;
    j.no_extra_row = (h->flags & AJ_FLAG_NO_EXTRA_ROW) ? 1 : 0;
    j.top_k = h->top_k;
    j.V = h->V;
    j.rank_cnt = h->rk_cnt;
    if (h->fold && h->umma_ok && h->top_k == 0) {
        j.fold_parts = h->fold_parts;
        j.fold_stride = h->max_B * (h->max_K + 1);
    }
    j.accept_len = accept_len;
    j.next_tok = next_tok;
    j.target_tok = target_tok;
    j.top1_val = top1_val;
    j.judge_p = judge_p;
    if (launch_judge_scan(j, stream) != cudaSuccess) return AJ_ERR_CUDA;
    h->keys_dirty = false;
    h->last_launches++;
    return AJ_OK;
}

aj_status aj_verify(aj_handle h, const void *h_target, const void *h_draft, const void *W_lm, const int32_t *draft_tok,
                    const float *judge_w, float judge_b, float tau, int B, int K, int d, int V, int32_t *accept_len,
                    int32_t *next_tok, int32_t *target_tok, float *top1_val, float *judge_p, void *cuda_stream) {
    aj_status st = check_call(h, h_target, h_draft, W_lm, draft_tok, judge_w, B, K, d, V, accept_len, next_tok);
    if (st != AJ_OK) return st;
    if (h->dtype == AJ_BF16 && (!aligned16(h_target) || !aligned16(W_lm) || (h_draft && !aligned16(h_draft))))
        return AJ_ERR_UNSUPPORTED;
    if (h->projected) return AJ_ERR_INVALID_ARG;  // an aj_shard_project is waiting for its aj_shard_finish
    DeviceGuard guard(h->device);
    if (!guard.ok()) return AJ_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    st = enqueue_project(h, h_target, W_lm, draft_tok, B, K, stream);
    if (st != AJ_OK) return st;
    return enqueue_finish(h, h_target, h_draft, draft_tok, judge_w, judge_b, tau, B, K, accept_len, next_tok, target_tok,
                          top1_val, judge_p, stream);
}

aj_status aj_verify_tree(aj_handle h, const void *h_target, const void *h_draft, const void *W_lm, const int32_t *draft_tok,
                         const int32_t *parent, const float *judge_w, float judge_b, float tau, int B, int N, int d, int V,
                         int32_t *accept_len, int32_t *next_tok, int32_t *best_node, int32_t *target_tok, float *top1_val,
                         float *judge_p, void *cuda_stream) {
    aj_status st = check_call(h, h_target, h_draft, W_lm, draft_tok, judge_w, B, N, d, V, accept_len, next_tok);
    if (st != AJ_OK) return st;
    if (!parent) return AJ_ERR_INVALID_ARG;
    // every node needs its own row, and the top-K rule's thresholds are taken per window position
    if ((h->flags & AJ_FLAG_NO_EXTRA_ROW) || h->top_k > 0) return AJ_ERR_UNSUPPORTED;
    if (h->dtype == AJ_BF16 && (!aligned16(h_target) || !aligned16(W_lm) || (h_draft && !aligned16(h_draft))))
        return AJ_ERR_UNSUPPORTED;
    if (h->projected) return AJ_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok()) return AJ_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    st = enqueue_project(h, h_target, W_lm, draft_tok, B, N, stream);
    if (st != AJ_OK) return st;
    return enqueue_finish(h, h_target, h_draft, draft_tok, judge_w, judge_b, tau, B, N, accept_len, next_tok, target_tok,
                          top1_val, judge_p, stream, parent, best_node);
}

aj_status aj_verify_host(aj_handle h, const void *h_target_host, const void *h_draft_host, const void *W_lm,
                         const int32_t *draft_tok_host, const float *judge_w, float judge_b, float tau, int B, int K,
                         int d, int V, int32_t *accept_len_host, int32_t *next_tok_host, int32_t *target_tok_host,
                         void *cuda_stream) {
    aj_status st = check_call(h, h_target_host, h_draft_host, W_lm, draft_tok_host, judge_w, B, K, d, V, accept_len_host,
                              next_tok_host);
    if (st != AJ_OK) return st;
    DeviceGuard guard(h->device);
    if (!guard.ok()) return AJ_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t M = (size_t)B * rows_per_seq(h, K), esz = elem_size(h->dtype);
    // The hidden states are always copied (the projection kernel reads them a thousand times over), and
    // their copies are enqueued first: everything the host does next runs while they are on their way.
    // A small batch in pinned memory is fetched by a kernel, anything else by the copy engines.
    const size_t ht_bytes = M * d * esz, hd_bytes = M * h->d_draft * esz;
    bool ok = true, staged = false;
    if (ht_bytes + hd_bytes <= STAGE_KERNEL_MAX_BYTES && ht_bytes % 16 == 0 && hd_bytes % 16 == 0) {
        const void *ht_view = device_view(h_target_host);
        const void *hd_view = hd_bytes ? device_view(h_draft_host) : nullptr;
        if (ht_view && aligned16(ht_view) && (hd_bytes == 0 || (hd_view && aligned16(hd_view)))) {
            const unsigned n_a = (unsigned)(ht_bytes / 16), n_b = (unsigned)(hd_bytes / 16);
            const unsigned blocks = (n_a + n_b + 255) / 256;
            stage_hidden_kernel<<<blocks < 1024 ? blocks : 1024, 256, 0, stream>>>(
                static_cast<const uint4 *>(ht_view), static_cast<uint4 *>(h->st_ht), n_a, static_cast<const uint4 *>(hd_view),
                static_cast<uint4 *>(h->st_hd), n_b);
            ok = cudaGetLastError() == cudaSuccess;
            staged = true;
        }
    }
    if (!staged)
        ok = cudaMemcpyAsync(h->st_ht, h_target_host, ht_bytes, cudaMemcpyHostToDevice, stream) == cudaSuccess &&
             (hd_bytes == 0 || cudaMemcpyAsync(h->st_hd, h_draft_host, hd_bytes, cudaMemcpyHostToDevice, stream) == cudaSuccess);
    if (!ok) return AJ_ERR_CUDA;
    // Small host buffers that are pinned (and therefore mapped into the device's address space) are
    // used in place by the judge kernel: it reads the draft tokens and writes the results over PCIe,
    // which saves three copy operations per cycle.
    int32_t *tok_dev = static_cast<int32_t *>(device_view(draft_tok_host));
    int32_t *acc_dev = static_cast<int32_t *>(device_view(accept_len_host));
    int32_t *next_dev = static_cast<int32_t *>(device_view(next_tok_host));
    int32_t *tt_dev = target_tok_host ? static_cast<int32_t *>(device_view(target_tok_host)) : nullptr;
    ok = tok_dev || cudaMemcpyAsync(h->st_tok, draft_tok_host, (size_t)B * K * 4, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    if (!ok) return AJ_ERR_CUDA;
    st = aj_verify(h, h->st_ht, h->d_draft ? h->st_hd : nullptr, W_lm, tok_dev ? tok_dev : h->st_tok, judge_w, judge_b, tau, B, K,
                   d, V, acc_dev ? acc_dev : h->st_acc, next_dev ? next_dev : h->st_next,
                   target_tok_host ? (tt_dev ? tt_dev : h->st_tt) : nullptr, nullptr, nullptr, cuda_stream);
    if (st != AJ_OK) return st;
    const int launches = h->last_launches + (staged ? 1 : 0);
    ok = (acc_dev || cudaMemcpyAsync(accept_len_host, h->st_acc, (size_t)B * 4, cudaMemcpyDeviceToHost, stream) == cudaSuccess) &&
         (next_dev || cudaMemcpyAsync(next_tok_host, h->st_next, (size_t)B * 4, cudaMemcpyDeviceToHost, stream) == cudaSuccess) &&
         (!target_tok_host || tt_dev ||
          cudaMemcpyAsync(target_tok_host, h->st_tt, M * 4, cudaMemcpyDeviceToHost, stream) == cudaSuccess) &&
         cudaStreamSynchronize(stream) == cudaSuccess;
    h->last_launches = launches;
    return ok ? AJ_OK : AJ_ERR_CUDA;
}

aj_status aj_last_status(aj_handle h) {
    if (!h) return AJ_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok()) return AJ_ERR_CUDA;
    int word = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) return AJ_ERR_CUDA;
    if (cudaMemcpy(&word, h->status, sizeof word, cudaMemcpyDeviceToHost) != cudaSuccess) return AJ_ERR_CUDA;
    if (word != 0) {
        if (cudaMemset(h->status, 0, sizeof word) != cudaSuccess) return AJ_ERR_CUDA;
        h->keys_dirty = true;  // a cycle that gave up may have left partial keys behind
    }
    return word == DEV_TIMEOUT ? AJ_ERR_TIMEOUT : (word == 0 ? AJ_OK : AJ_ERR_CUDA);
}

aj_status aj_last_gemm_ms(aj_handle h, float *ms) {
    if (!h || !ms || !(h->flags & AJ_FLAG_TIME_KERNELS) || h->n_timed == 0) return AJ_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    const int slot = (int)((h->n_timed - 1) % EVENT_RING);
    if (cudaEventSynchronize(h->ev1[slot]) != cudaSuccess) return AJ_ERR_CUDA;
    if (cudaEventElapsedTime(ms, h->ev0[slot], h->ev1[slot]) != cudaSuccess) return AJ_ERR_CUDA;
    return AJ_OK;
}

aj_status aj_gemm_ms_stats(aj_handle h, float *mean_ms, float *min_ms, int *count) {
    if (!h || !mean_ms || !count || !(h->flags & AJ_FLAG_TIME_KERNELS)) return AJ_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    const long long n = h->n_timed < EVENT_RING ? h->n_timed : EVENT_RING;
    double sum = 0.0;
    float lo = 0.0f;
    for (long long i = 0; i < n; i++) {
        const int slot = (int)((h->n_timed - 1 - i) % EVENT_RING);
        float ms = 0.0f;
        if (cudaEventSynchronize(h->ev1[slot]) != cudaSuccess) return AJ_ERR_CUDA;
        if (cudaEventElapsedTime(&ms, h->ev0[slot], h->ev1[slot]) != cudaSuccess) return AJ_ERR_CUDA;
        sum += ms;
        if (i == 0 || ms < lo) lo = ms;
    }
    *mean_ms = n ? (float)(sum / n) : 0.0f;
    if (min_ms) *min_ms = lo;
    *count = (int)n;
    h->n_timed = 0;
    return AJ_OK;
}

size_t aj_shard_exchange_bytes(int max_B, int max_K, int world) {
    if (max_B < 1 || max_K < 1 || world < 1 || world > MAX_SHARD_WORLD) return 0;
    return EXCHANGE_FLAG_BYTES + 2 * (size_t)world * ((size_t)max_B * (max_K + 1)) * sizeof(unsigned long long);
}

aj_status aj_shard_range(int V, int world, int rank, int *v_begin, int *v_count) {
    if (!v_begin || !v_count || V < 1 || world < 1 || world > MAX_SHARD_WORLD || rank < 0 || rank >= world)
        return AJ_ERR_INVALID_ARG;
    const int blocks = (V + 255) / 256;  // whole blocks of 256 entries, so that shards start on a tile boundary
    if (blocks < world) return AJ_ERR_INVALID_ARG;  // some GPU would get nothing
    const int base = blocks / world, rem = blocks % world;
    const long long b0 = (long long)rank * base + (rank < rem ? rank : rem);
    const long long b1 = b0 + base + (rank < rem ? 1 : 0);
    const long long lo = b0 * 256 < V ? b0 * 256 : V, hi = b1 * 256 < V ? b1 * 256 : V;
    *v_begin = (int)lo;
    *v_count = (int)(hi - lo);
    return AJ_OK;
}

aj_status aj_create_sharded(aj_handle *out, int device, int max_B, int max_K, int d, int d_draft, int V, aj_dtype dtype,
                            aj_w_layout layout, unsigned flags, int rank, int world, int v_begin, int v_count,
                            void *const *exchange) {
    if (!out) return AJ_ERR_INVALID_ARG;
    *out = nullptr;
    if (!exchange || world < 1 || world > MAX_SHARD_WORLD || rank < 0 || rank >= world) return AJ_ERR_INVALID_ARG;
    if (v_begin < 0 || v_count < 1 || (long long)v_begin + v_count > V) return AJ_ERR_INVALID_ARG;
    for (int r = 0; r < world; r++)
        if (!exchange[r] || (reinterpret_cast<uintptr_t>(exchange[r]) & 255)) return AJ_ERR_INVALID_ARG;
    aj_handle h = nullptr;
    if (layout == AJ_W_DV && v_count % 8 != 0) flags |= AJ_FLAG_FORCE_SIMT;  // the shard's row pitch is not TMA-loadable
    aj_status st = aj_create(&h, device, max_B, max_K, d, d_draft, V, dtype, layout, flags);
    if (st != AJ_OK) return st;
    h->world = world;
    h->rank = rank;
    h->v_begin = v_begin;
    h->v_count = v_count;
    for (int r = 0; r < world; r++) h->exchange[r] = static_cast<unsigned long long *>(exchange[r]);
    // this GPU's own buffer starts from zero flags; peers must not publish before every rank has
    // created its handle (the caller puts a barrier between creation and the first cycle)
    DeviceGuard guard(device);
    if (!guard.ok() || cudaMemset(exchange[rank], 0, aj_shard_exchange_bytes(max_B, max_K, world)) != cudaSuccess ||
        cudaDeviceSynchronize() != cudaSuccess) {
        cudaGetLastError();
        aj_destroy(h);
        return AJ_ERR_CUDA;
    }
    *out = h;
    return AJ_OK;
}

aj_status aj_shard_project(aj_handle h, const void *h_target, const void *W_shard, int B, int K, void *cuda_stream) {
    if (!h || !h->world || !h_target || !W_shard || B < 1 || K < 1) return AJ_ERR_INVALID_ARG;
    if (B > h->max_B || K > h->max_K) return AJ_ERR_WORKSPACE;
    if (h->projected) return AJ_ERR_INVALID_ARG;
    if (h->dtype == AJ_BF16 && (!aligned16(h_target) || !aligned16(W_shard))) return AJ_ERR_UNSUPPORTED;
    DeviceGuard guard(h->device);
    if (!guard.ok()) return AJ_ERR_CUDA;
    aj_status st = enqueue_project(h, h_target, W_shard, nullptr, B, K, static_cast<cudaStream_t>(cuda_stream));
    if (st == AJ_OK) h->projected = true;
    return st;
}

aj_status aj_shard_finish(aj_handle h, const void *h_target, const void *h_draft, const int32_t *draft_tok,
                          const float *judge_w, float judge_b, float tau, int B, int K, int32_t *accept_len,
                          int32_t *next_tok, int32_t *target_tok, float *top1_val, float *judge_p, void *cuda_stream) {
    if (!h || !h->world || !h->projected) return AJ_ERR_INVALID_ARG;
    if (!h_target || !draft_tok || !judge_w || !accept_len || !next_tok) return AJ_ERR_INVALID_ARG;
    if ((h->d_draft > 0) != (h_draft != nullptr) || B < 1 || K < 1) return AJ_ERR_INVALID_ARG;
    if (B > h->max_B || K > h->max_K) return AJ_ERR_WORKSPACE;
    if (h->dtype == AJ_BF16 && (!aligned16(h_target) || (h_draft && !aligned16(h_draft)))) return AJ_ERR_UNSUPPORTED;
    DeviceGuard guard(h->device);
    if (!guard.ok()) return AJ_ERR_CUDA;
    aj_status st = enqueue_finish(h, h_target, h_draft, draft_tok, judge_w, judge_b, tau, B, K, accept_len, next_tok,
                                  target_tok, top1_val, judge_p, static_cast<cudaStream_t>(cuda_stream));
    if (st == AJ_OK) h->projected = false;
    return st;
}

aj_status aj_shard_exchange_alloc(int max_B, int max_K, int world, void **device_ptr_out) {
    if (!device_ptr_out) return AJ_ERR_INVALID_ARG;
    *device_ptr_out = nullptr;
    const size_t n = aj_shard_exchange_bytes(max_B, max_K, world);
    if (n == 0) return AJ_ERR_INVALID_ARG;
    void *p = nullptr;
    if (cudaMalloc(&p, n) != cudaSuccess || cudaMemset(p, 0, n) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) {
        cudaGetLastError();
        if (p) cudaFree(p);
        return AJ_ERR_CUDA;
    }
    *device_ptr_out = p;
    return AJ_OK;
}

aj_status aj_shard_exchange_free(void *device_ptr) {
    if (!device_ptr) return AJ_ERR_INVALID_ARG;
    if (cudaFree(device_ptr) != cudaSuccess) {
        cudaGetLastError();
        return AJ_ERR_CUDA;
    }
    return AJ_OK;
}

aj_status aj_ipc_export(const void *device_ptr, unsigned char handle_out[64]) {
    if (!device_ptr || !handle_out) return AJ_ERR_INVALID_ARG;
    static_assert(sizeof(cudaIpcMemHandle_t) == 64, "IPC handle size");
    cudaIpcMemHandle_t hd;
    if (cudaIpcGetMemHandle(&hd, const_cast<void *>(device_ptr)) != cudaSuccess) {
        cudaGetLastError();
        return AJ_ERR_CUDA;
    }
    memcpy(handle_out, &hd, 64);
    return AJ_OK;
}

aj_status aj_ipc_import(const unsigned char handle_in[64], void **device_ptr_out) {
    if (!handle_in || !device_ptr_out) return AJ_ERR_INVALID_ARG;
    cudaIpcMemHandle_t hd;
    memcpy(&hd, handle_in, 64);
    if (cudaIpcOpenMemHandle(device_ptr_out, hd, cudaIpcMemLazyEnablePeerAccess) != cudaSuccess) {
        cudaGetLastError();
        *device_ptr_out = nullptr;
        return AJ_ERR_CUDA;
    }
    return AJ_OK;
}

aj_status aj_ipc_close(void *device_ptr) {
    if (!device_ptr) return AJ_ERR_INVALID_ARG;
    if (cudaIpcCloseMemHandle(device_ptr) != cudaSuccess) {
        cudaGetLastError();
        return AJ_ERR_CUDA;
    }
    return AJ_OK;
}

aj_status aj_set_top_k(aj_handle h, int top_k) {
    if (!h || top_k < 0) return AJ_ERR_INVALID_ARG;
    // the count is kept per GPU
    if (top_k > 0 && (h->world || (h->flags & AJ_FLAG_NO_EXTRA_ROW))) return AJ_ERR_UNSUPPORTED;
    if (top_k > 0 && h->temperature > 0.0f) return AJ_ERR_UNSUPPORTED;  // the rule ranks the plain logits
    h->top_k = top_k;
    return AJ_OK;
}

aj_status aj_set_sampling(aj_handle h, float temperature, uint64_t seed, uint64_t step) {
    if (!h || !(temperature >= 0.0f) || !(temperature <= 3.0e38f)) return AJ_ERR_INVALID_ARG;
    if (temperature > 0.0f && h->top_k > 0) return AJ_ERR_UNSUPPORTED;
    h->temperature = temperature;
    h->seed = seed;
    h->step = step;
    return AJ_OK;
}

aj_status aj_fuse_judge(aj_handle h, const float *judge_w, void *cuda_stream) {
    if (!h) return AJ_ERR_INVALID_ARG;
    if (!judge_w) {
        h->fold = false;
        return AJ_OK;
    }
    if (!h->umma_ok) return AJ_ERR_UNSUPPORTED;  // the CUDA-core kernel has no extra rows to offer
    DeviceGuard guard(h->device);
    if (!guard.ok()) return AJ_ERR_CUDA;
    if (launch_judge_split(judge_w + h->d_draft, h->d, h->layout, h->fold_rows, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return AJ_ERR_CUDA;
    h->fold = true;
    return AJ_OK;
}

int aj_last_launch_count(aj_handle h) { return h ? h->last_launches : 0; }

aj_status aj_pair_schedule(int M, int d, int V, int32_t out[10]) {
    if (!out || M < 1 || d < 1 || V < 1) return AJ_ERR_INVALID_ARG;
    const PairSched sc = pair_schedule(M, V, d, 0);
    out[0] = sc.n_v;
    out[1] = sc.n_n;
    out[2] = sc.u_base;
    out[3] = sc.u_rem;
    out[4] = sc.box_rows;
    out[5] = sc.n_groups;
    out[6] = sc.g_base;
    out[7] = sc.g_rem;
    out[8] = sc.dual;
    out[9] = sc.stages;
    return AJ_OK;
}

const char *aj_last_gemm_path(aj_handle h) { return h ? h->last_path : "none"; }

}  // extern "C"
