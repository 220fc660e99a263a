// Tensor-core projection + running argmax for sm_100a on CTA pairs (two SMs per tile), the
// tensor-bound regime (more than 128 rows of hidden states):
//
//   logit[v, m] = sum_k W[v, k] * h[m, k]        bf16 x bf16 -> fp32 in tensor memory, never stored
//   keys[m]     = max over v of pack(logit[v, m], v)
//
// A tile is 256 vocabulary entries (UMMA M = 256, 128 per SM = the 128 TMEM lanes of each SM) by
// up to 256 rows of hidden states (UMMA N, any multiple of 16).  The rows are cut into the fewest
// tiles of at most 256 rows and spread over them evenly in units of 16 rows (2112 rows = 6 tiles of
// 240 + 3 of 224), so no tensor work is spent on padding and all tiles take nearly the same time,
// which keeps the pairs that share a block of W in step and that block in L2.  When h_target
// outgrows L2 the row tiles are walked in groups, each group against the whole vocabulary.
//
// The two CTAs of a cluster sit on one SM pair; the even CTA (the leader) issues
// tcgen05.mma.cta_group::2 for both.  Each CTA stages its own 128 rows of W and HALF of the tile's
// rows of h, so a k-block costs at most 32 KB of L2 -> SM traffic per SM where the one-SM kernel
// needs 48 KB for the same tensor work.  Nothing is multicast: every CTA fetches its own half-tiles
// with ordinary tiled TMA loads, and the follower's loads report their bytes to the leader's barrier.
//
// Roles in each CTA (192 threads):
//   warp 0      TMA producer (one thread): waits for its own stage to be free, then loads
//               W[v0 + 128*rank .. +128, kb] and h[n0 + (N/2)*rank .. , kb] with 128-byte swizzle;
//   warp 1      allocates tensor memory (both CTAs); in the leader one thread issues the MMAs and
//               commits stage-release and accumulator-ready barriers to both CTAs at once;
//   warps 2..5  epilogue: thread = one TMEM lane = one vocabulary entry.  32 columns (rows of h) at a
//               time are compared with the best value each row has so far (read from its key); only
//               a chunk in which some logit reaches that value is reduced (per column the warp
//               maximum by redux.sync on the order-preserving image of the logit, the lowest lane
//               attaining it by ballot) and merged into the row's packed key by a 64-bit atomic max.
// Two accumulator buffers of 256 columns: the epilogue of one tile runs under the MMAs of the next.
// No split over k.  Every wait is bounded; a wait that runs out sets the status word, and both CTAs
// still meet at the cluster barrier before tensor memory is freed.
#include "aj_internal.cuh"
#include "aj_ptx.cuh"

#include <type_traits>

namespace aj {

namespace {

constexpr int BV = 256;       // vocabulary entries per tile (128 per CTA)
constexpr int BV_CTA = 128;
constexpr int BN = 256;       // rows of h per accumulator (half of them staged by each CTA)
constexpr int BK = 64;        // bf16 elements per k-block = 128 bytes = one swizzle span
constexpr int UMMA_K = 16;
// Warp 0 loads, warp 1 issues the MMAs, the rest drain the accumulators: one warp per TMEM lane quadrant,
// or two (which take alternate groups of column chunks) where the epilogue does more than the argmax (the
// noise, or the count of the top-K rule) and, with two accumulators per tile, is not hidden under the next
// tile's MMAs.  Measured on one GPU against four warps: sampled mode 3 % and 4 % faster with two
// accumulators at 2080 x 8192 and 264 x 4096, but 3 % slower with one at 2112 and 528 rows x 4096; top-K
// rule 8 % and 4 % faster at the same two shapes; the plain argmax unchanged at both (3 % faster at 392 rows).
__host__ __device__ constexpr int epilogue_warps(int epi, bool dual) { return epi != EPI_PLAIN && dual ? 8 : 4; }
__host__ __device__ constexpr int num_threads(int epi, bool dual) { return 64 + 32 * epilogue_warps(epi, dual); }
constexpr int A_BYTES = BV_CTA * BK * 2;   // 16 KB: this CTA's 128 rows of W, one k-block
constexpr int RING_BYTES = 224 * 1024;     // shared memory given to the stage ring (the SM has 227 KB per CTA)
constexpr int MAX_STAGES = 8;
constexpr int TMEM_COLS = 2 * BN;
constexpr int BAR_BYTES = 8 * (2 * MAX_STAGES + 4) + 16;
constexpr int SMEM_BYTES = RING_BYTES + BAR_BYTES + 1024;

struct Tile {
    int v_tile;     // block of 256 vocabulary entries
    int row0[2];    // first row of h of each accumulator
    int n_inst[2];  // rows of each accumulator = UMMA N, a multiple of 16 (the second is 0 in single mode)
};

// Tile t of the schedule.  Row tiles come in groups; a group is walked against every vocabulary
// block (row tile fastest) before the next group starts.  Consecutive tiles, which run on
// neighbouring pairs at the same time, share a block of W.  Which row tile of the group a pair gets
// rotates with the vocabulary block, so that pairs whose number is a multiple of the group size
// apart do not always get the larger (or the smaller) row tiles and drift away from the pairs they
// share W with.  In dual mode a row tile is split over the two accumulators.
__device__ inline Tile decode_tile(const PairSched &sc, int t) {
    int g = 0, start = 0, sz = sc.g_base + (0 < sc.g_rem ? 1 : 0);
    while (g + 1 < sc.n_groups && t >= start + sz * sc.n_v) {
        start += sz * sc.n_v;
        ++g;
        sz = sc.g_base + (g < sc.g_rem ? 1 : 0);
    }
    const int first = g * sc.g_base + min(g, sc.g_rem);
    const int local = t - start;
    Tile r;
    r.v_tile = local / sz;
    const int n_tile = first + (local % sz + r.v_tile) % sz;
    const int u0 = n_tile * sc.u_base + min(n_tile, sc.u_rem);
    const int nu = sc.u_base + (n_tile < sc.u_rem ? 1 : 0);
    const int nu0 = sc.dual ? (nu + 1) >> 1 : nu;
    r.row0[0] = 16 * u0;
    r.n_inst[0] = 16 * nu0;
    r.row0[1] = 16 * (u0 + nu0);
    r.n_inst[1] = 16 * (nu - nu0);
    return r;
}

// DUAL: every tile uses two accumulators that share the staged block of W.  WDV: W is stored [d, V].
// EPI: EPI_COUNT also counts, per row, the entries that outrank the draft token (top-K rule);
// EPI_SAMPLE adds Gumbel noise to the logits before the argmax.
template <bool DUAL, bool WDV, int EPI>
__global__ void __launch_bounds__(num_threads(EPI, DUAL), 1)
umma_pair_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_h,
                 int M, int V, int d, PairSched sc, int stream_w, int v_offset,
                 unsigned long long *__restrict__ keys, int *__restrict__ status, const Publish pub, const RankArgs rk,
                 const Noise nz) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;  // the same offset in both CTAs: one descriptor serves both
    uint8_t *smem = smem_raw + (base - raw);

    const uint32_t bar_base = base + RING_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };                                  // used in the leader only
    auto empty_bar = [&](int s) { return bar_base + 8u * (MAX_STAGES + s); };
    auto acc_full_bar = [&](int a) { return bar_base + 8u * (2 * MAX_STAGES + a); };
    auto acc_empty_bar = [&](int a) { return bar_base + 8u * (2 * MAX_STAGES + 2 + a); };      // used in the leader only
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + RING_BYTES + 8 * (2 * MAX_STAGES + 4));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5;  // warp-uniform
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();  // 0 = leader
    const int pair = blockIdx.x >> 1;
    const int num_pairs = gridDim.x >> 1;
    const int num_kb = d / BK;
    const int num_tiles = sc.n_n * sc.n_v;
    constexpr int n_acc = DUAL ? 2 : 1;
    const int stages = sc.stages;
    const uint32_t b_bytes = (uint32_t)sc.box_rows * BK * 2;       // one accumulator's rows of h staged by this CTA
    const uint32_t stage_bytes = A_BYTES + n_acc * b_bytes;         // a multiple of 1024
    const uint32_t stage_tx = 2u * stage_bytes;                     // bytes both CTAs load per stage

    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_STAGES; s++) {
            mbar_init(full_bar(s), 1);   // the leader's producer; bytes arrive from both CTAs
            mbar_init(empty_bar(s), 1);  // one commit from the leader's MMA thread
        }
        for (int a = 0; a < 2; a++) {
            mbar_init(acc_full_bar(a), 1);
            mbar_init(acc_empty_bar(a), 2 * epilogue_warps(EPI, DUAL));  // the epilogue warps of the two CTAs
        }
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc_pair(smem_u32(const_cast<uint32_t *>(tmem_slot)), TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // the peer's barriers exist before anything is sent to them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // Programmatic dependent launch: nothing the caller passed is read before this wait returns.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    auto give_up = [&]() {
        *abort_flag = 1;
        atomicCAS(status, DEV_OK, DEV_TIMEOUT);
    };
    // Accumulator hand-over.  Single mode: the two 256-column buffers alternate from tile to tile
    // (buffer it & 1, each with its own pair of barriers).  Dual mode: every tile uses both buffers
    // as two accumulators that share the staged block of W, and one pair of barriers.
    auto acc_slot = [&](int it) { return DUAL ? 0 : (it & 1); };
    auto acc_phase = [&](int it) { return (uint32_t)(DUAL ? it : (it >> 1)) & 1u; };

    if (warp == 0) {
        if (lane == 0) {
            // ------------------------------------------------------------ TMA producer
            const unsigned long long pol_h = policy_evict_last();
            const unsigned long long pol_w = stream_w ? policy_evict_first() : policy_evict_normal();
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int t = pair; ok && t < num_tiles; t += num_pairs) {
                const Tile tl = decode_tile(sc, t);
                const int w_row = tl.v_tile * BV + (int)rank * BV_CTA;
                const int h_row0 = tl.row0[0] + (int)rank * (tl.n_inst[0] >> 1);
                const int h_row1 = tl.row0[1] + (int)rank * (tl.n_inst[1] >> 1);
                for (int kb = 0; kb < num_kb; kb++) {
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) {
                        give_up();
                        ok = false;
                        break;
                    }
                    const uint32_t leader_full = map_to_cta(full_bar(s), 0);
                    if (rank == 0) mbar_expect_tx(full_bar(s), stage_tx);
                    const uint32_t a_dst = base + s * stage_bytes;
                    if (WDV) {  // W stored [d, V]: two boxes of 64 entries x 64 k-rows
                        tma_load_2d_pair(a_dst, &tmap_w, w_row, kb * BK, leader_full, pol_w);
                        tma_load_2d_pair(a_dst + A_BYTES / 2, &tmap_w, w_row + 64, kb * BK, leader_full, pol_w);
                    } else {
                        tma_load_2d_pair(a_dst, &tmap_w, kb * BK, w_row, leader_full, pol_w);
                    }
                    tma_load_2d_pair(a_dst + A_BYTES, &tmap_h, kb * BK, h_row0, leader_full, pol_h);
                    if (n_acc == 2) tma_load_2d_pair(a_dst + A_BYTES + b_bytes, &tmap_h, kb * BK, h_row1, leader_full, pol_h);
                    if (++s == stages) {
                        s = 0;
                        ph ^= 1u;
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            // ------------------------------------------- MMA issuer (leader CTA only)
            // (rebuilding the descriptors per k-block measured slightly faster than stepping them
            // from stage to stage, which chains every k-block's issue to the previous one)
            const unsigned long long acc_step = b_bytes >> 4;
            constexpr unsigned long long a_step = WDV ? MN_KSTEP : 2ull;
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            int it = 0;
            for (int t = pair; ok && t < num_tiles; t += num_pairs, ++it) {
                const Tile tl = decode_tile(sc, t);
                constexpr uint32_t a_major = WDV ? IDESC_A_MN_MAJOR : 0u;
                const uint32_t idesc0 = instr_desc(BV, tl.n_inst[0]) | a_major;
                const uint32_t idesc1 = instr_desc(BV, tl.n_inst[1]) | a_major;
                const int slot = acc_slot(it);
                if (!mbar_wait(acc_empty_bar(slot), acc_phase(it) ^ 1u, abort_flag)) {
                    give_up();
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem0 = tmem_base + (uint32_t)(slot * BN);
                const uint32_t d_tmem1 = tmem_base + (uint32_t)BN;  // dual mode only
                for (int kb = 0; kb < num_kb; kb++) {
                    if (!mbar_wait(full_bar(s), ph, abort_flag)) {
                        give_up();
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t a_addr = base + s * stage_bytes;
                    const unsigned long long adesc = WDV ? smem_desc_sw128_mn(a_addr) : smem_desc_sw128(a_addr);
                    const unsigned long long bdesc0 = smem_desc_sw128(a_addr + A_BYTES);
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; k++)
                        umma_bf16_pair(d_tmem0, adesc + a_step * k, bdesc0 + 2ull * k, idesc0, (uint32_t)((kb | k) != 0));
                    if (n_acc == 2) {
                        const unsigned long long bdesc1 = bdesc0 + acc_step;
#pragma unroll
                        for (int k = 0; k < BK / UMMA_K; k++)
                            umma_bf16_pair(d_tmem1, adesc + a_step * k, bdesc1 + 2ull * k, idesc1, (uint32_t)((kb | k) != 0));
                    }
                    umma_commit_pair(empty_bar(s));  // frees the stage in both CTAs
                    if (++s == stages) {
                        s = 0;
                        ph ^= 1u;
                    }
                }
                if (ok) umma_commit_pair(acc_full_bar(slot));  // the accumulators in both CTAs are complete
            }
        }
    } else {
        // -------------------------------------------------------------------- epilogue
        // A logit can only matter if it reaches the best value its row has so far.  Lane j reads
        // that value for column 32c + j from the row's key before the tile's accumulators are
        // ready (a stale value is only lower, never wrong).  A chunk of 32 columns is then checked
        // with one comparison per element against the shuffled-in thresholds and one vote; only
        // if some element qualifies does the chunk take the reduction path (warp maximum per
        // column by redux.sync, lowest lane by ballot, 64-bit atomic max into the key).  After the
        // first few vocabulary blocks nearly every chunk is skipped.
        const int q = warp & 3;  // TMEM lane quadrant this warp may read
        constexpr int SPLIT = epilogue_warps(EPI, DUAL) / 4;           // warps per quadrant
        const int part = SPLIT == 1 ? 0 : (warp - 2) >> 2;        // which of them this one is
        const float never = __int_as_float(0x7fc00000);  // NaN: no comparison with it is ever true
        // Chunk g of a tile is columns 32 (g & 7) .. + 32 of accumulator g >> 3.  Its threshold for
        // lane j is the best value the row of column 32 (g & 7) + j has so far, read from the key.
        auto load_thr = [&](const Tile &tl, int g) {
            const int a = g >> 3, col = (g & 7) * 32 + lane;
            const int row = (a ? tl.row0[1] : tl.row0[0]) + col;
            if (a >= n_acc || col >= (a ? tl.n_inst[1] : tl.n_inst[0]) || row >= M) return never;
            const unsigned long long k = __ldcg(keys + row);
            return k == 0ull ? -INFINITY : key_value(k);
        };
        // thresholds are fetched GRP chunks ahead of their use, an L2 round trip: four chunks, or one
        // where the noise makes a chunk take that long by itself (and one copy of its code, not four,
        // then stays within the instruction cache)
        constexpr int GRP = EPI == EPI_SAMPLE ? 1 : 4;
        int it = 0;
        for (int t = pair; t < num_tiles; t += num_pairs, ++it) {
            const Tile tl = decode_tile(sc, t);
            const int slot = acc_slot(it);
            float cur[GRP], nxt[GRP];
#pragma unroll
            for (int u = 0; u < GRP; u++) cur[u] = load_thr(tl, part * GRP + u);  // in flight while the accumulators are being computed
            // the whole warp takes one decision, so the aligned TMEM loads below stay converged
            if (!__all_sync(0xffffffffu, mbar_wait(acc_full_bar(slot), acc_phase(it), abort_flag))) {
                give_up();
                break;
            }
            tc_fence_after();
            const int v_first = tl.v_tile * BV + (int)rank * BV_CTA + q * 32;  // vocabulary entry of lane 0
            const bool v_ok = v_first + lane < V;                            // entries past V hold zero-filled junk
            const uint32_t tbase = tmem_base + ((uint32_t)(q * 32) << 16);
            // the group loop is kept rolled: one copy of the code stays in the instruction cache
#pragma unroll 1
            for (int g0 = part * GRP; g0 < 8 * n_acc; g0 += GRP * SPLIT) {
#pragma unroll
                for (int u = 0; u < GRP; u++) nxt[u] = (g0 + GRP * SPLIT < 8 * n_acc) ? load_thr(tl, g0 + GRP * SPLIT + u) : never;
#pragma unroll
                for (int u = 0; u < GRP; u++) {
                    const int g = g0 + u, a = g >> 3, c = g & 7;
                    const int n_inst = a ? tl.n_inst[1] : tl.n_inst[0];
                    if (c * 32 < n_inst) {  // warp-uniform
                        const float thr = cur[u];
                        float v[32];
                        tmem_ld32(tbase + (uint32_t)((DUAL ? a : slot) * BN + c * 32), v);
                        if (EPI == EPI_COUNT)
                            count_outranking(rk, v, v_first, v_ok, (a ? tl.row0[1] : tl.row0[0]) + c * 32, n_inst - c * 32, M, lane);
                        if (EPI == EPI_SAMPLE) add_gumbel_noise(nz, v, v_first + lane + v_offset, (a ? tl.row0[1] : tl.row0[0]) + c * 32);
                        bool hit = false;
#pragma unroll
                        for (int j = 0; j < 32; j++) hit |= v[j] >= __shfl_sync(0xffffffffu, thr, j);
                        if (__any_sync(0xffffffffu, hit && v_ok)) {
                            uint32_t best_u = 0u;  // lane j: maximum of column 32c + j over this warp's 32 entries
                            int best_i = 0;
#pragma unroll
                            for (int j = 0; j < 32; j++) {
                                const uint32_t x = v_ok ? ordered_image(v[j]) : 0u;
                                const uint32_t m = warp_max_u32(x);
                                const uint32_t who = __ballot_sync(0xffffffffu, x == m);
                                if (lane == j) {
                                    best_u = m;
                                    best_i = v_first + __ffs(who) - 1;  // the lowest entry that attains the maximum
                                }
                            }
                            const int row = (a ? tl.row0[1] : tl.row0[0]) + c * 32 + lane;
                            if (c * 32 + lane < n_inst && row < M && best_u != 0u) {
                                const unsigned long long key =
                                    ((unsigned long long)best_u << 32) | (uint32_t)(~(uint32_t)(best_i + v_offset));
                                if (key > *reinterpret_cast<volatile unsigned long long *>(&keys[row])) atomicMax(&keys[row], key);
                            }
                        }
                    }
                }
#pragma unroll
                for (int u = 0; u < GRP; u++) cur[u] = nxt[u];
            }
            // the accumulators are drained: hand them back to the leader's MMA thread
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(acc_empty_bar(slot), 0));
        }
    }

    __syncwarp();
    tc_fence_before();
    __syncthreads();
    publish_keys(pub, keys);
    if (warp == 1 && *abort_flag) {
        // copies or MMAs may still be in flight after an abort: give them time to land
        const unsigned long long t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    cluster_sync_all();  // neither CTA leaves, or frees tensor memory, while the other may still signal it
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

int g_max_pairs = 0;

}  // namespace

cudaError_t umma_pair_prepare(int num_sms) {
    cudaError_t e = cudaSuccess;
    const void *kernels[12] = {
        (const void *)umma_pair_kernel<false, false, EPI_PLAIN>,  (const void *)umma_pair_kernel<true, false, EPI_PLAIN>,
        (const void *)umma_pair_kernel<false, true, EPI_PLAIN>,   (const void *)umma_pair_kernel<true, true, EPI_PLAIN>,
        (const void *)umma_pair_kernel<false, false, EPI_COUNT>,  (const void *)umma_pair_kernel<true, false, EPI_COUNT>,
        (const void *)umma_pair_kernel<false, true, EPI_COUNT>,   (const void *)umma_pair_kernel<true, true, EPI_COUNT>,
        (const void *)umma_pair_kernel<false, false, EPI_SAMPLE>, (const void *)umma_pair_kernel<true, false, EPI_SAMPLE>,
        (const void *)umma_pair_kernel<false, true, EPI_SAMPLE>,  (const void *)umma_pair_kernel<true, true, EPI_SAMPLE>};
    for (const void *k : kernels) {
        e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e != cudaSuccess) return e;
    }
    // how many CTA pairs can be resident at once (pairs need both SMs of a pair free)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(num_sms & ~1));
    cfg.blockDim = dim3(num_threads(EPI_SAMPLE, true));  // the largest block: residency is the same, one CTA per SM
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int clusters = 0;
    e = cudaOccupancyMaxActiveClusters(&clusters, umma_pair_kernel<true, false, EPI_SAMPLE>, &cfg);
    if (e != cudaSuccess) return e;
    if (clusters < 1) return cudaErrorInvalidConfiguration;
    g_max_pairs = clusters < num_sms / 2 ? clusters : num_sms / 2;
    return cudaSuccess;
}

int umma_pair_max_pairs() { return g_max_pairs; }

PairSched pair_schedule(int M, int V, int d) {
    PairSched sc;
    const int units = (M + 15) / 16;  // rows in units of 16 (the UMMA N granule)
    // Two accumulators per tile (up to 512 rows share each staged block of W; 25 % less operand
    // traffic, but the epilogue is no longer hidden under the next tile's MMAs) or one (at most 256
    // rows, double-buffered)?  Measured on the same GPU: two win from 257 to about 450 rows, where
    // they save a second pass over W (-10 % at 264 and 400 rows, +4 % at 512), and for deep
    // contractions with many rows, where the exposed epilogue is a small share of a tile and the
    // operand traffic weighs most (d = 8192: -1.5 % at 1056 rows, -6 % at 2080, -9 % at 4160; but
    // +1.5 % at 528, and +3 ... +8 % for every batch at d = 4096).
    sc.dual = (units > 16 && (units <= 28 || (d >= 8192 && units >= 64))) ? 1 : 0;
    const int cap = sc.dual ? 32 : 16;
    sc.n_n = (units + cap - 1) / cap;
    sc.u_base = units / sc.n_n;
    sc.u_rem = units % sc.n_n;
    sc.n_v = (V + BV - 1) / BV;
    const int u_max = sc.u_base + (sc.u_rem ? 1 : 0);
    // rows of h each CTA stages per accumulator: half of the largest accumulator
    sc.box_rows = 8 * (sc.dual ? (u_max + 1) / 2 : u_max);
    const int stage_bytes = A_BYTES + (sc.dual ? 2 : 1) * sc.box_rows * BK * 2;
    sc.stages = RING_BYTES / stage_bytes < MAX_STAGES ? RING_BYTES / stage_bytes : MAX_STAGES;
    // row tiles per group: keep a group's rows of h (tile rows x d x 2 bytes) within about 40 MB of L2
    const long long tile_bytes = 256ll * d * 2;
    int g_max = (int)((40ll << 20) / tile_bytes);
    if (g_max < 1) g_max = 1;
    sc.n_groups = (sc.n_n + g_max - 1) / g_max;
    sc.g_base = sc.n_n / sc.n_groups;
    sc.g_rem = sc.n_n % sc.n_groups;
    return sc;
}

cudaError_t launch_umma_pair(const GemmArgs &a, const UmmaPlan &p, cudaStream_t stream) {
    const PairSched sc = pair_schedule(a.M, a.V, a.d);
    const int stream_w = (sc.n_n == 1) ? 1 : 0;  // W is read by one pair only: do not keep it in L2
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.grid);  // 2 CTAs per pair
    const int epi = a.noise.temperature > 0.0f ? EPI_SAMPLE : a.rank.thr ? EPI_COUNT : EPI_PLAIN;
    cfg.blockDim = dim3(num_threads(epi, sc.dual != 0));
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    auto pick = [&](auto epi) {
        constexpr int E = decltype(epi)::value;
        return sc.dual ? (a.w_layout ? umma_pair_kernel<true, true, E> : umma_pair_kernel<true, false, E>)
                       : (a.w_layout ? umma_pair_kernel<false, true, E> : umma_pair_kernel<false, false, E>);
    };
    auto kernel = a.noise.temperature > 0.0f ? pick(std::integral_constant<int, EPI_SAMPLE>{})
                  : a.rank.thr               ? pick(std::integral_constant<int, EPI_COUNT>{})
                                             : pick(std::integral_constant<int, EPI_PLAIN>{});
    return cudaLaunchKernelEx(&cfg, kernel, p.tmap_w, p.tmap_h, a.M, a.V, a.d, sc, stream_w, a.v_offset, a.keys, a.status,
                              a.pub, a.rank, a.noise);
}

}  // namespace aj
