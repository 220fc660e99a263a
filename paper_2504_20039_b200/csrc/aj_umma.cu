// Tensor-core projection + running argmax for sm_100a:
//
//   logit[m, v] = sum_k h[m, k] * W[v, k]        bf16 x bf16 -> fp32 in tensor memory, never stored
//   keys[m]     = max over v of pack(logit[m, v], v)
//
// Persistent CTAs, one per SM, three roles:
//   warp 0      TMA producer: k-blocks of 64 columns of h (128 rows) and of W (BN rows) into a
//               ring of shared-memory stages, 128-byte swizzle, completion on mbarriers;
//   warp 1      MMA issuer: one thread issues tcgen05.mma (M=128, N=BN, K=16) from shared-memory
//               descriptors into one of two accumulator buffers in tensor memory, and commits
//               stage-release and accumulator-ready barriers;
//   warps 2..5  epilogue: each thread owns one row of the tile (one TMEM lane), reads the
//               accumulator 32 columns at a time and keeps a running (max, argmax) in registers
//               across the CTA's vocabulary tiles; it is merged into the row's packed key with
//               a 64-bit atomic max when the CTA moves to another row tile and at the end.
// The two accumulator buffers let the epilogue of one tile run under the MMAs of the next.
//
// There is no split over k: every logit is one fixed-order accumulation, so the result does
// not depend on the tiling, the grid or the batch composition.
//
// Every wait is bounded: a wait that runs out sets the status word to "timeout", raises a
// CTA-wide abort flag that the other roles poll, and the CTA leaves through the normal
// teardown (tensor memory is freed after a pause that lets copies in flight land).
#include "aj_internal.cuh"
#include "aj_ptx.cuh"

namespace aj {

namespace {

constexpr int BM = 128;      // rows of h per tile = UMMA M = TMEM lanes
constexpr int BK = 64;       // bf16 elements per k-block = 128 bytes = one swizzle span
constexpr int UMMA_K = 16;   // k per tcgen05.mma for 16-bit inputs
constexpr int NUM_THREADS = 192;
constexpr int A_BYTES = BM * BK * 2;

template <int BN> struct Cfg {
    static constexpr int B_BYTES = BN * BK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int STAGES = (192 * 1024) / STAGE_BYTES;
    static constexpr int TMEM_COLS = 2 * BN;
    static constexpr int BAR_BYTES = 8 * (2 * STAGES + 4) + 16;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + BAR_BYTES + 1024;  // + alignment slack
};

// ------------------------------------------------------------------------------------ kernel

template <int BN>
__global__ void __launch_bounds__(NUM_THREADS, 1)
umma_gemm_argmax_kernel(const __grid_constant__ CUtensorMap tmap_h, const __grid_constant__ CUtensorMap tmap_w,
                        int M, int V, int d, int n_m, int n_v, int stream_w,
                        unsigned long long *__restrict__ keys, int *__restrict__ status) {
    using C = Cfg<BN>;
    constexpr int STAGES = C::STAGES;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;  // swizzled tiles need 1024-byte alignment
    uint8_t *smem = smem_raw + (base - raw);

    const uint32_t bar_base = base + STAGES * C::STAGE_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto acc_full_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
    auto acc_empty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + STAGES * C::STAGE_BYTES + 8 * (2 * STAGES + 4));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5;  // warp-uniform
    const int lane = threadIdx.x & 31;
    const int num_kb = d / BK;
    const int num_tiles = n_m * n_v;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; s++) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < 2; a++) {
            mbar_init(acc_full_bar(a), 1);
            mbar_init(acc_empty_bar(a), 128);
        }
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_slot)), C::TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // This kernel may be launched as a programmatic dependent of whatever precedes it in the
    // stream, so that the set-up above overlaps that kernel's tail: nothing the caller passed has
    // been read yet, and nothing is before this wait returns (the previous grid has then finished
    // and its writes are visible).  Then let this kernel's own dependent, the judge kernel, become
    // resident; it waits at its grid dependency until this whole grid has finished.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    auto give_up = [&]() {
        *abort_flag = 1;
        atomicCAS(status, DEV_OK, DEV_TIMEOUT);
    };

    if (warp == 0) {
        if (lane == 0) {
            // ------------------------------------------------------------ TMA producer
            const unsigned long long pol_h = policy_evict_last();
            const unsigned long long pol_w = stream_w ? policy_evict_first() : policy_evict_normal();
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int t = blockIdx.x; ok && t < num_tiles; t += gridDim.x) {
                const int m_tile = t % n_m, v_tile = t / n_m;
                for (int kb = 0; kb < num_kb; kb++) {
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) {
                        give_up();
                        ok = false;
                        break;
                    }
                    mbar_expect_tx(full_bar(s), C::STAGE_BYTES);
                    const uint32_t a_dst = base + s * C::STAGE_BYTES;
                    tma_load_2d(a_dst, &tmap_h, kb * BK, m_tile * BM, full_bar(s), pol_h);
                    tma_load_2d(a_dst + A_BYTES, &tmap_w, kb * BK, v_tile * BN, full_bar(s), pol_w);
                    if (++s == STAGES) {
                        s = 0;
                        ph ^= 1u;
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // -------------------------------------------------------------- MMA issuer
            constexpr uint32_t idesc = instr_desc(BM, BN);
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            int it = 0;
            for (int t = blockIdx.x; ok && t < num_tiles; t += gridDim.x, ++it) {
                const int ab = it & 1;
                const uint32_t aph = (uint32_t)(it >> 1) & 1u;
                if (!mbar_wait(acc_empty_bar(ab), aph ^ 1u, abort_flag)) {
                    give_up();
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(ab * BN);
                for (int kb = 0; kb < num_kb; kb++) {
                    if (!mbar_wait(full_bar(s), ph, abort_flag)) {
                        give_up();
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t a_addr = base + s * C::STAGE_BYTES;
                    const unsigned long long adesc = smem_desc_sw128(a_addr);
                    const unsigned long long bdesc = smem_desc_sw128(a_addr + A_BYTES);
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; k++)
                        umma_bf16(d_tmem, adesc + 2ull * k, bdesc + 2ull * k, idesc, (uint32_t)((kb | k) != 0));
                    umma_commit(empty_bar(s));  // the stage is free once these MMAs have read it
                    if (++s == STAGES) {
                        s = 0;
                        ph ^= 1u;
                    }
                }
                if (ok) umma_commit(acc_full_bar(ab));  // the accumulator is complete
            }
        }
    } else {
        // -------------------------------------------------------------------- epilogue
        const int q = warp & 3;  // TMEM lane quadrant this warp may read
        const int row_in_tile = q * 32 + lane;
        float best = -INFINITY;
        int bidx = 0;
        int cur_m = -1;
        auto flush = [&]() {
            if (cur_m >= 0) {
                const int row = cur_m * BM + row_in_tile;
                if (row < M) atomicMax(&keys[row], pack_key(best, bidx));
            }
        };
        int it = 0;
        for (int t = blockIdx.x; t < num_tiles; t += gridDim.x, ++it) {
            const int m_tile = t % n_m, v_tile = t / n_m;
            const int ab = it & 1;
            const uint32_t aph = (uint32_t)(it >> 1) & 1u;
            if (m_tile != cur_m) {
                flush();
                best = -INFINITY;
                bidx = 0;
                cur_m = m_tile;
            }
            // the whole warp takes one decision, so the aligned TMEM loads below stay converged
            if (!__all_sync(0xffffffffu, mbar_wait(acc_full_bar(ab), aph, abort_flag))) {
                give_up();
                break;
            }
            tc_fence_after();
            const int v0 = v_tile * BN;
            const int ncols = min(BN, V - v0);
            const bool warp_has_rows = (m_tile * BM + q * 32) < M;  // warp-uniform
            if (warp_has_rows) {
                const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(ab * BN);
#pragma unroll 1
                for (int c = 0; c < BN / 32; c++) {
                    const int c0 = c * 32;
                    if (c0 >= ncols) break;
                    float v[32];
                    tmem_ld32(taddr + c0, v);
                    if (c0 + 32 <= ncols) {
#pragma unroll
                        for (int j = 0; j < 32; j++)
                            if (v[j] > best) {  // strict: columns ascend, the lowest index keeps a tie
                                best = v[j];
                                bidx = v0 + c0 + j;
                            }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; j++)
                            if (c0 + j < ncols && v[j] > best) {  // columns past V hold zero-filled junk
                                best = v[j];
                                bidx = v0 + c0 + j;
                            }
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(acc_empty_bar(ab));
        }
        flush();
    }

    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        if (*abort_flag) {
            // copies or MMAs may still be in flight after an abort: give them time to land
            const unsigned long long t0 = globaltimer_ns();
            while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
        }
        tc_fence_after();
        tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
}

template <int BN>
cudaError_t launch_one(const GemmArgs &a, const UmmaPlan &p, cudaStream_t stream) {
    const int n_m = (a.M + BM - 1) / BM;
    const int n_v = (a.V + BN - 1) / BN;
    const int stream_w = (n_m == 1) ? 1 : 0;  // W is read by one CTA only: do not keep it in L2
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.grid);
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = Cfg<BN>::SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, umma_gemm_argmax_kernel<BN>, p.tmap_h, p.tmap_w, a.M, a.V, a.d, n_m, n_v, stream_w,
                              a.keys, a.status);
}

}  // namespace

cudaError_t umma_prepare() {
    cudaError_t e;
    e = cudaFuncSetAttribute(umma_gemm_argmax_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<64>::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(umma_gemm_argmax_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<128>::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(umma_gemm_argmax_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<256>::SMEM_BYTES);
    return e;
}

cudaError_t launch_umma_gemm_argmax(const GemmArgs &a, const UmmaPlan &p, cudaStream_t stream) {
    switch (p.bn) {
        case 64: return launch_one<64>(a, p, stream);
        case 128: return launch_one<128>(a, p, stream);
        case 256: return launch_one<256>(a, p, stream);
        default: return cudaErrorInvalidValue;
    }
}

const char *umma_path_name(int bn) {
    switch (bn) {
        case 64: return "umma_128x64";
        case 128: return "umma_128x128";
        case 256: return "umma_128x256";
        default: return "umma_?";
    }
}

}  // namespace aj
