// Tensor-core projection + running argmax for sm_100a, vocabulary-major tiles:
//
//   logit[v, m] = sum_k W[v, k] * h[m, k]        bf16 x bf16 -> fp32 in tensor memory, never stored
//   keys[m]     = max over v of pack(logit[v, m], v)
//
// The vocabulary runs along the UMMA M axis (128 entries per tile = the 128 TMEM lanes) and the
// rows of hidden states along the UMMA N axis, which may be any multiple of 16 up to 256.  So a
// batch of M rows costs ceil16(M) columns of tensor work, not a multiple of 128: a 17-row batch
// issues N = 32 MMAs, and a 2112-row batch splits into 8 tiles of 256 rows plus one of 64.
//
// Persistent CTAs, one per SM, three roles:
//   warp 0      TMA producer: k-blocks of 64 columns of W (128 rows) and of h (BN rows) into a
//               ring of shared-memory stages (one or two k-blocks per stage), 128-byte swizzle,
//               completion on mbarriers;
//   warp 1      MMA issuer: one thread issues tcgen05.mma (M=128, N=rows of the tile, K=16) into
//               one of two accumulator buffers in tensor memory;
//   warps 2..5  epilogue: a thread owns one TMEM lane = one vocabulary entry and reads 32 columns
//               (rows of h) at a time.  Per column the warp takes the maximum over its 32 entries
//               with one redux.sync on the order-preserving integer image of the logit, finds the
//               lowest lane that attains it with a ballot, and lane j keeps the running
//               (max, argmax) of column j.  The running values are merged into the rows' packed
//               keys with 64-bit atomic max when the CTA moves to another block of rows, and at
//               the end.
// No split over k: every logit is one fixed-order accumulation.  Every wait is bounded (see
// aj_ptx.cuh); a wait that runs out sets the status word and the CTA leaves through the normal
// teardown.
#include "aj_internal.cuh"
#include "aj_ptx.cuh"

#include <type_traits>

namespace aj {

namespace {

constexpr int BV = 128;     // vocabulary entries per tile = UMMA M = TMEM lanes
constexpr int BK = 64;      // bf16 elements per k-block = 128 bytes = one swizzle span
constexpr int UMMA_K = 16;  // k per tcgen05.mma for 16-bit inputs
constexpr int NUM_THREADS = 192;
constexpr int A_BYTES = BV * BK * 2;

template <int BN> struct VCfg {
    static constexpr int B_BYTES = BN * BK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    // ring size: 224 of the SM's 227 KB per CTA, except for the narrowest tile, where 9 stages of
    // 20 KB measured faster than 11 (161 vs 168 us on the batch-1 8B shape); with two k-blocks per
    // stage that is four stages of 40 KB (five measured slower again: 163.5 vs 161.6 us)
    static constexpr int STAGES = ((BN <= 32 ? 192 : 224) * 1024) / STAGE_BYTES;
    static constexpr int TMEM_COLS = 2 * BN < 32 ? 32 : 2 * BN;
    static constexpr int NCH = (BN + 31) / 32;  // 32-column chunks per accumulator
    static constexpr int BAR_BYTES = 8 * (2 * STAGES + 4) + 16;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + BAR_BYTES + 1024;  // + alignment slack
};

// WDV: W is stored [d, V].  EPI: EPI_COUNT also counts, per row, the entries that outrank the draft
// token; EPI_SAMPLE adds Gumbel noise to the logits before the argmax.
template <int BN, bool WDV, int EPI>
__global__ void __launch_bounds__(NUM_THREADS, 1)
umma_vm_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_h,
               const __grid_constant__ CUtensorMap tmap_j, int M, int V, int d, int n_n, int n_v, int fold_tile,
               int stream_w, int kps, int box_rows, int v_offset, unsigned long long *__restrict__ keys, int *__restrict__ status, const Publish pub,
               const RankArgs rk, const Noise nz, float *__restrict__ fold_parts, int fold_stride) {
    using C = VCfg<BN>;
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
    const int num_tiles = n_n * n_v;
    // A stage holds kps k-blocks (1 or 2), each [W | h], in the same ring: with two, the issuing thread tests
    // one barrier and commits once per 8 MMAs instead of per 4.
    // (and the rows of h per k-block are the rows of the tensor map's box, box_rows <= BN: a batch that fits one
    // row tile stages only the rows it has, which leaves room for more stages)
    const uint32_t sub_bytes = A_BYTES + (uint32_t)box_rows * BK * 2;
    const uint32_t stage_bytes = (uint32_t)kps * sub_bytes;
    const int fit = (STAGES * C::STAGE_BYTES) / (int)stage_bytes;
    const int stages = fit < STAGES ? fit : STAGES;

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
    // Programmatic dependent launch: the set-up above may overlap the previous kernel's tail.
    // Nothing the caller passed is read before this wait returns.  Then let this kernel's own
    // dependent, the judge kernel, become resident; it waits until this whole grid has finished.
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
                const int n_tile = t % n_n, v_tile = t / n_n;
                const bool fold = v_tile == fold_tile;  // the block after the vocabulary: the classifier rows, entry 0 of their own map
                const CUtensorMap *tw = fold ? &tmap_j : &tmap_w;
                const int w_row = fold ? 0 : v_tile * BV;
                for (int kb = 0; kb < num_kb; kb += kps) {
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) {
                        give_up();
                        ok = false;
                        break;
                    }
                    mbar_expect_tx(full_bar(s), stage_bytes);
                    for (int j = 0; j < kps; j++) {
                        const uint32_t a_dst = base + s * stage_bytes + j * sub_bytes;
                        const int kc = (kb + j) * BK;
                        if (WDV) {  // W stored [d, V]: two boxes of 64 entries x 64 k-rows
                            tma_load_2d(a_dst, tw, w_row, kc, full_bar(s), pol_w);
                            tma_load_2d(a_dst + A_BYTES / 2, tw, w_row + 64, kc, full_bar(s), pol_w);
                        } else {
                            tma_load_2d(a_dst, tw, kc, w_row, full_bar(s), pol_w);
                        }
                        tma_load_2d(a_dst + A_BYTES, &tmap_h, kc, n_tile * BN, full_bar(s), pol_h);
                    }
                    if (++s == stages) {
                        s = 0;
                        ph ^= 1u;
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // -------------------------------------------------------------- MMA issuer
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            int it = 0;
            for (int t = blockIdx.x; ok && t < num_tiles; t += gridDim.x, ++it) {
                const int n_tile = t % n_n;
                const int rows_valid = min(BN, M - n_tile * BN);
                const int n_inst = max(16, (rows_valid + 15) & ~15);  // UMMA N: a multiple of 16
                const uint32_t idesc = instr_desc(BV, n_inst) | (WDV ? IDESC_A_MN_MAJOR : 0u);
                const int ab = it & 1;
                const uint32_t aph = (uint32_t)(it >> 1) & 1u;
                if (!mbar_wait(acc_empty_bar(ab), aph ^ 1u, abort_flag)) {
                    give_up();
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(ab * BN);
                for (int kb = 0; kb < num_kb; kb += kps) {
                    if (!mbar_wait(full_bar(s), ph, abort_flag)) {
                        give_up();
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    for (int j = 0; j < kps; j++) {
                        const uint32_t a_addr = base + s * stage_bytes + j * sub_bytes;
                        const unsigned long long adesc = WDV ? smem_desc_sw128_mn(a_addr) : smem_desc_sw128(a_addr);
                        constexpr unsigned long long a_step = WDV ? MN_KSTEP : 2ull;
                        const unsigned long long bdesc = smem_desc_sw128(a_addr + A_BYTES);
#pragma unroll
                        for (int k = 0; k < BK / UMMA_K; k++)
                            umma_bf16(d_tmem, adesc + a_step * k, bdesc + 2ull * k, idesc, (uint32_t)((kb | j | k) != 0));
                    }
                    umma_commit(empty_bar(s));  // the stage is free once these MMAs have read it
                    if (++s == stages) {
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
        uint32_t rb_u[C::NCH];   // lane j, chunk c: running maximum of column 32c + j (ordered image)
        int rb_i[C::NCH];        //                  and the vocabulary entry that attains it
#pragma unroll
        for (int c = 0; c < C::NCH; c++) {
            rb_u[c] = 0u;
            rb_i[c] = 0;
        }
        auto flush = [&](int n_tile) {
#pragma unroll
            for (int c = 0; c < C::NCH; c++) {
                const int row = n_tile * BN + c * 32 + lane;
                if (row < M && rb_u[c] != 0u)
                    atomicMax(&keys[row], ((unsigned long long)rb_u[c] << 32) | (uint32_t)(~(uint32_t)(rb_i[c] + v_offset)));
                rb_u[c] = 0u;
            }
        };
        int it = 0;
        for (int t = blockIdx.x; t < num_tiles; t += gridDim.x, ++it) {
            const int n_tile = t % n_n, v_tile = t / n_n;
            const int rows_valid = min(BN, M - n_tile * BN);
            const int n_inst = max(16, (rows_valid + 15) & ~15);
            const int ab = it & 1;
            const uint32_t aph = (uint32_t)(it >> 1) & 1u;
            // the whole warp takes one decision, so the aligned TMEM loads below stay converged
            if (!__all_sync(0xffffffffu, mbar_wait(acc_full_bar(ab), aph, abort_flag))) {
                give_up();
                break;
            }
            tc_fence_after();
            const int v_first = v_tile * BV + q * 32;       // vocabulary entry of lane 0 of this warp
            const bool v_ok = v_first + lane < V;           // entries past V hold zero-filled junk
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(ab * BN);
#pragma unroll
            for (int c = 0; c < C::NCH; c++) {
                if (c * 32 < n_inst) {  // warp-uniform
                    float v[32];
                    tmem_ld32(taddr + c * 32, v);
                    if (v_tile == fold_tile) {
                        // the classifier rows: lanes 0..2 of the first quadrant hold the three partial dot
                        // products of 32 rows of h; they are stored, and nothing of this block is a logit
                        if (q == 0 && lane < JUDGE_FOLD_ROWS) {
#pragma unroll
                            for (int j = 0; j < 32; j++) {
                                const int row = n_tile * BN + c * 32 + j;
                                if (c * 32 + j < n_inst && row < M) fold_parts[(size_t)lane * fold_stride + row] = v[j];
                            }
                        }
                        continue;
                    }
                    if (EPI == EPI_COUNT) {
                        const int row = n_tile * BN + c * 32 + lane;
                        const bool valid = c * 32 + lane < n_inst && row < M;
                        float vmax = v[0];
#pragma unroll
                        for (int j = 1; j < 32; j++) vmax = fmaxf(vmax, v[j]);
                        count_outranking(rk, v, vmax, v_first, v_ok, rank_threshold(rk, row, valid), valid ? __ldg(rk.tok + row) : -1, row,
                                         valid, lane);
                    }
                    if (EPI == EPI_SAMPLE) {
                        // the lowest of the chunk's running maxima bounds the noise an element needs to matter
                        const int row = n_tile * BN + c * 32 + lane;
                        const uint32_t tmin = warp_min_u32((c * 32 + lane < n_inst && row < M) ? rb_u[c] : 0xFFFFFFFFu);
                        float pmax = v[0];
#pragma unroll
                        for (int j = 1; j < 32; j++) pmax = fmaxf(pmax, v[j]);
                        const uint32_t k_need = noise_cutoff(key_value((unsigned long long)tmin << 32), pmax, nz.inv_temperature);
                        if (!add_gumbel_noise(nz, v, v_first + lane + v_offset, n_tile * BN + c * 32, k_need)) continue;
                    }
                    // all 32 reductions are issued before any result is used, so that their
                    // latencies overlap instead of adding up
                    uint32_t u[32], m[32];
#pragma unroll
                    for (int j = 0; j < 32; j++) u[j] = v_ok ? ordered_image(v[j]) : 0u;
#pragma unroll
                    for (int j = 0; j < 32; j++) m[j] = warp_max_u32(u[j]);
#pragma unroll
                    for (int j = 0; j < 32; j++) {
                        const uint32_t who = __ballot_sync(0xffffffffu, u[j] == m[j]);
                        if (lane == j && m[j] > rb_u[c]) {  // strict: an earlier (lower) entry keeps a tie
                            rb_u[c] = m[j];
                            rb_i[c] = v_first + __ffs(who) - 1;
                        }
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(acc_empty_bar(ab));
            const int t_next = t + gridDim.x;
            if (t_next >= num_tiles || (t_next % n_n) != n_tile) flush(n_tile);
        }
    }

    __syncwarp();
    tc_fence_before();
    __syncthreads();
    publish_keys(pub, keys);
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
cudaError_t launch_vm(const GemmArgs &a, const UmmaPlan &p, cudaStream_t stream) {
    const int n_n = (a.M + BN - 1) / BN;
    const int fold = a.fold.rows ? 1 : 0;
    const int n_v = (a.V + BV - 1) / BV + fold;  // one more block for the folded classifier rows
    const int stream_w = (n_n == 1) ? 1 : 0;  // W is read by one CTA only: do not keep it in L2
    // two k-blocks per stage where three such stages fit (every width but 256): the issuing thread's barrier
    // test and commit then come once per 8 MMAs
    const int box_rows = vm_box_rows(a.M, BN);
    const int ring = VCfg<BN>::STAGES * VCfg<BN>::STAGE_BYTES, sub = A_BYTES + box_rows * BK * 2;
    const int kps = ((a.d / BK) % 2 == 0 && ring / (2 * sub) >= 3) ? 2 : 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.grid);
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = VCfg<BN>::SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    auto pick = [&](auto epi) {
        constexpr int E = decltype(epi)::value;
        return a.w_layout ? umma_vm_kernel<BN, true, E> : umma_vm_kernel<BN, false, E>;
    };
    auto kernel = a.noise.temperature > 0.0f ? pick(std::integral_constant<int, EPI_SAMPLE>{})
                  : a.rank.thr               ? pick(std::integral_constant<int, EPI_COUNT>{})
                                             : pick(std::integral_constant<int, EPI_PLAIN>{});
    return cudaLaunchKernelEx(&cfg, kernel, p.tmap_w, p.tmap_h, fold ? p.tmap_j : p.tmap_w, a.M, a.V, a.d, n_n, n_v,
                              fold ? n_v - 1 : -1, stream_w, kps, box_rows, a.v_offset, a.keys, a.status, a.pub, a.rank, a.noise, a.fold.parts,
                              a.fold.stride);
}

}  // namespace

int vm_choose_bn(int M) { return M <= 32 ? 32 : M <= 64 ? 64 : M <= 128 ? 128 : 256; }

// Rows of h in the tensor map's box (and per staged k-block): the tile width, or, for a batch of one row
// tile wider than 32, just the batch's rows rounded up to the UMMA N granule of 16.
int vm_box_rows(int M, int bn) { return (bn > 32 && M <= bn) ? ((M + 15) & ~15) : bn; }

template <int BN> static cudaError_t set_smem() {
    const int bytes = VCfg<BN>::SMEM_BYTES;
    const void *kernels[6] = {(const void *)umma_vm_kernel<BN, false, EPI_PLAIN>,  (const void *)umma_vm_kernel<BN, true, EPI_PLAIN>,
                              (const void *)umma_vm_kernel<BN, false, EPI_COUNT>,  (const void *)umma_vm_kernel<BN, true, EPI_COUNT>,
                              (const void *)umma_vm_kernel<BN, false, EPI_SAMPLE>, (const void *)umma_vm_kernel<BN, true, EPI_SAMPLE>};
    for (const void *k : kernels) {
        const cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t umma_vm_prepare() {
    cudaError_t e;
    e = set_smem<32>();
    if (e != cudaSuccess) return e;
    e = set_smem<64>();
    if (e != cudaSuccess) return e;
    e = set_smem<128>();
    if (e != cudaSuccess) return e;
    e = set_smem<256>();
    return e;
}

cudaError_t launch_umma_vm(const GemmArgs &a, const UmmaPlan &p, cudaStream_t stream) {
    switch (p.bn) {
        case 32: return launch_vm<32>(a, p, stream);
        case 64: return launch_vm<64>(a, p, stream);
        case 128: return launch_vm<128>(a, p, stream);
        case 256: return launch_vm<256>(a, p, stream);
        default: return cudaErrorInvalidValue;
    }
}

const char *umma_vm_path_name(int bn) {
    switch (bn) {
        case 32: return "umma_vm_128x32";
        case 64: return "umma_vm_128x64";
        case 128: return "umma_vm_128x128";
        case 256: return "umma_vm_128x256";
        default: return "umma_vm_?";
    }
}

}  // namespace aj
