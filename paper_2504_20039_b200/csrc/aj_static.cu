// aj_verify_static: the verify-and-judge cycle for callers that must not allocate.
//
// Some callers cannot call cudaMalloc at the point where they need a cycle verified: an
// inference server that handed all device memory to its own pool at start-up, code running
// under a memory budget that is audited per allocation, or a library loaded late into a
// process whose allocator is frozen.  aj_create allocates a workspace, so those callers cannot
// use the handle API.  This entry point needs no handle: the only scratch memory the cycle
// needs (one packed (max, argmax) key per row of hidden states, plus a status word) lives in a
// fixed array in the library's own device image, below.  Every GPU that loads the library holds
// that array (AJ_STATIC_MAX_ROWS * 8 + 256 bytes) until the process exits.
//
// The array's name is a host-side stand-in in host code, not a device address, so the address
// the kernels receive is looked up with cudaGetSymbolAddress, once per device, with that
// device current, the first time this entry point is called on the device.
#include "../../include/aj_verify.h"
#include "aj_internal.cuh"

#include <mutex>

constexpr int STATIC_MAX_ROWS = AJ_STATIC_MAX_ROWS;
constexpr int STATUS_BYTES = 256;

// keys[STATIC_MAX_ROWS] followed by a status word; shared by every call on this device
static __device__ __align__(256) unsigned char g_static_scratch[(size_t)STATIC_MAX_ROWS * 8 + STATUS_BYTES];

namespace {

using namespace aj;

constexpr int MAX_DEVICES = 64;

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct DeviceSetup {
    bool done = false;
    aj_status error = AJ_OK;
    unsigned char *scratch = nullptr;  // device address of g_static_scratch on this device
    int num_sms = 0;
    bool pair_ok = false;  // the two-SM kernel can be launched on this device
    EncodeTiledFn encode = nullptr;
};

std::mutex g_mutex;
DeviceSetup g_setup[MAX_DEVICES];

// Once per device, with that device current: resolve the scratch array's device address, check
// the architecture, fetch the tensor-map encoder and opt the kernels into large shared memory.
// None of this allocates device memory.
const DeviceSetup *setup_current_device(aj_status *st) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) {
        cudaGetLastError();
        *st = AJ_ERR_CUDA;
        return nullptr;
    }
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceSetup &s = g_setup[dev];
    if (!s.done) {
        s.done = true;
        int major = 0;
        void *ptr = nullptr;
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&s.num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            s.error = AJ_ERR_CUDA;
        } else if (major != 10) {
            s.error = AJ_ERR_NOT_SM100;
        } else if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) {
            s.error = AJ_ERR_CUDA;
        } else if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres) != cudaSuccess ||
                   qres != cudaDriverEntryPointSuccess || fn == nullptr) {
            s.error = AJ_ERR_CUDA;
        } else if (umma_vm_prepare() != cudaSuccess) {
            s.error = AJ_ERR_CUDA;
        } else {
            s.scratch = static_cast<unsigned char *>(ptr);
            s.encode = reinterpret_cast<EncodeTiledFn>(fn);
            s.pair_ok = umma_pair_prepare(s.num_sms) == cudaSuccess && umma_pair_max_pairs() > 0;  // an occupancy query, no allocation
        }
        if (s.error != AJ_OK) cudaGetLastError();
    }
    *st = s.error;
    return s.error == AJ_OK ? &s : nullptr;
}

bool encode_rows(const DeviceSetup *s, CUtensorMap *map, const void *ptr, int d, long long rows, int box_rows) {
    cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)d * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return s->encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace

extern "C" aj_status aj_verify_static(const void *h_target, const void *h_draft, const void *W_lm, const int32_t *draft_tok,
                                      const float *judge_w, float judge_b, float tau, int B, int K, int d, int d_draft, int V,
                                      aj_dtype dtype, aj_w_layout layout, int32_t *accept_len, int32_t *next_tok,
                                      int32_t *target_tok, float *top1_val, float *judge_p, int32_t *dev_status,
                                      void *cuda_stream) {
    if (!h_target || !W_lm || !draft_tok || !judge_w || !accept_len || !next_tok) return AJ_ERR_INVALID_ARG;
    if (B < 1 || K < 1 || K > 1024 || d < 1 || d_draft < 0 || V < 1) return AJ_ERR_INVALID_ARG;
    if ((d_draft > 0) != (h_draft != nullptr)) return AJ_ERR_INVALID_ARG;
    if (dtype != AJ_BF16 && dtype != AJ_F32) return AJ_ERR_INVALID_ARG;
    if (layout != AJ_W_VD && layout != AJ_W_DV) return AJ_ERR_INVALID_ARG;
    if ((long long)B * (K + 1) > STATIC_MAX_ROWS) return AJ_ERR_WORKSPACE;  // more rows than the fixed scratch holds
    if (dtype == AJ_BF16 && (d % 8 != 0 || d_draft % 8 != 0)) return AJ_ERR_UNSUPPORTED;
    if (dtype == AJ_BF16 && (!aligned16(h_target) || !aligned16(W_lm) || (h_draft && !aligned16(h_draft))))
        return AJ_ERR_UNSUPPORTED;

    aj_status st = AJ_OK;
    const DeviceSetup *s = setup_current_device(&st);
    if (!s) return st;

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int M = B * (K + 1);
    unsigned long long *keys = reinterpret_cast<unsigned long long *>(s->scratch);
    int *status = dev_status ? dev_status : reinterpret_cast<int *>(s->scratch + (size_t)STATIC_MAX_ROWS * 8);

    // the array keeps the previous call's contents: the keys of this call's rows must start at zero
    if (cudaMemsetAsync(keys, 0, (size_t)M * sizeof(unsigned long long), stream) != cudaSuccess) return AJ_ERR_CUDA;
    if (cudaMemsetAsync(status, 0, sizeof(int), stream) != cudaSuccess) return AJ_ERR_CUDA;

    GemmArgs g;
    g.h = h_target;
    g.W = W_lm;
    g.M = M;
    g.d = d;
    g.V = V;
    g.dtype = dtype;
    g.w_layout = layout;
    g.keys = keys;
    g.status = status;
    // the tile counter of the two-SM kernel: zero when the library is loaded, put back to zero by every launch
    g.sched = reinterpret_cast<unsigned *>(s->scratch + (size_t)STATIC_MAX_ROWS * 8) + 32;

    // the same choice of projection kernel as aj_verify makes
    cudaError_t e;
    if (dtype == AJ_BF16 && layout == AJ_W_VD && d % 64 == 0 && M > 128 && s->pair_ok) {
        UmmaPlan p;
        p.bn = 256;
        const PairSched sc = pair_schedule(M, V, d, 0);
        if (!encode_rows(s, &p.tmap_w, W_lm, d, V, 128) || !encode_rows(s, &p.tmap_h, h_target, d, M, sc.box_rows)) return AJ_ERR_CUDA;
        const long long tiles = (long long)sc.n_n * sc.n_v;
        const int pairs = umma_pair_max_pairs();
        p.grid = 2 * (int)(tiles < pairs ? tiles : pairs);
        e = launch_umma_pair(g, p, stream);
    } else if (dtype == AJ_BF16 && layout == AJ_W_VD && d % 64 == 0) {
        UmmaPlan p;
        p.bn = vm_choose_bn(M);
        if (!encode_rows(s, &p.tmap_w, W_lm, d, V, 128) || !encode_rows(s, &p.tmap_h, h_target, d, M, vm_box_rows(M, p.bn))) return AJ_ERR_CUDA;
        const long long tiles = (long long)((M + p.bn - 1) / p.bn) * ((V + 127) / 128);
        p.grid = (int)(tiles < s->num_sms ? tiles : s->num_sms);
        e = launch_umma_vm(g, p, stream);
    } else {
        e = launch_simt_gemm_argmax(g, s->num_sms, stream);
    }
    if (e != cudaSuccess) return AJ_ERR_CUDA;

    JudgeArgs j;
    j.keys = keys;
    j.status = status;
    j.h_target = h_target;
    j.h_draft = h_draft;
    j.draft_tok = draft_tok;
    j.judge_w = judge_w;
    j.judge_b = judge_b;
    j.tau = tau;
    j.B = B;
    j.K = K;
    j.d = d;
    j.d_draft = d_draft;
    j.dtype = dtype;
    j.accept_len = accept_len;
    j.next_tok = next_tok;
    j.target_tok = target_tok;
    j.top1_val = top1_val;
    j.judge_p = judge_p;
    return launch_judge_scan(j, stream) == cudaSuccess ? AJ_OK : AJ_ERR_CUDA;
}
