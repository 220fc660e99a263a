// Tensor-core projection + running argmax for sm_100a on CTA pairs (two SMs per tile), for batches
// of more than 128 rows of hidden states:
//
//   logit[v, m] = sum_k W[v, k] * h[m, k]        bf16 x bf16 -> fp32 in tensor memory, never stored
//   keys[m]     = max over v of pack(logit[v, m], v)
//
// A tile is 256 vocabulary entries (UMMA M = 256, 128 per SM = the 128 TMEM lanes of each SM) by a
// block of rows of hidden states (UMMA N, any multiple of 16).  The rows are cut into the fewest
// tiles and spread over them evenly in units of 16 rows, so no tensor work is spent on padding and
// all tiles take nearly the same time.  When h_target outgrows L2 the row tiles are walked in groups,
// each group against the whole vocabulary.
//
// Tiles are numbered so that consecutive tiles share a block of W, and the pairs take them in that
// order from a counter in global memory as they become free.  A fixed assignment (pair p takes tiles
// p, p + pairs, ...) loses the sharing: SM pairs do not run at one speed (measured on one GPU: some
// pairs, the same ones in every launch, take 3 % longer per tile), after thirty tiles neighbouring
// pairs are a whole tile apart, and a block of W has left L2 before its last reader asks for it.  With
// the counter the readers of a block start within microseconds of one another at every point of the
// launch, W can be marked evict-first, h_target stays in L2, and a slower pair simply takes fewer tiles.
//
// Two forms (512 columns of tensor memory either way):
//   narrow tiles (DUAL = false, batches of at most 256 rows): one accumulator of up to 256 columns in
//     one of two buffers that alternate from tile to tile, so the epilogue of one tile runs under the
//     MMAs of the next; one issuing thread;
//   wide tiles (DUAL = true): up to 512 rows on TWO accumulators of up to 256 columns that share each
//     staged block of W, each with its own issuing warp and its own pair of barriers.
// Why two issuing warps: a tcgen05.mma holds the thread that issues it for about 100 cycles whatever
// its N (measured: one thread issuing 128 x N x 16 MMAs back to back gets one through per 104 cycles
// for every N <= 208; two warps issuing on two accumulators get one through per max(52, N/2) cycles,
// the tensor pipe's own rate).  With one issuing thread a k-block of two accumulators costs 8 x 104
// cycles plus the waits whatever the tensor work; with two, each accumulator's 4 MMAs per k-block are
// issued in parallel and the tensor pipe is the limit from about 140 rows per accumulator on.  The
// price of the wide form is that an accumulator has to be drained before its next tile can start
// (about 7,000 cycles per tile between the last MMA of one tile and the first of the next, against
// 55,000 cycles of MMAs at d = 4096); measured on one GPU it is the faster form for every batch of
// more than 256 rows (520 rows: 466 vs 562 us, 2112 rows: 1.57 vs 1.75 ms, 2080 x 8192: 3.13 vs 3.52 ms).
//
// The two CTAs of a cluster sit on one SM pair; the even CTA (the leader) issues
// tcgen05.mma.cta_group::2 for both.  Each CTA stages its own 128 rows of W and HALF of each
// accumulator's rows of h.  Nothing is multicast: every CTA fetches its own half-tiles with ordinary
// tiled TMA loads, and the follower's loads report their bytes to the leader's barrier.
//
// Roles in each CTA:
//   warp 0      TMA producer (one thread).  The leader's draws the pair's next tile from the counter and
//               announces it, through a small ring of slots in shared memory with their own barriers,
//               to every other warp of both CTAs (-1: no more tiles).  Both wait for a free stage (one or two
//               k-blocks of 64, see pair_schedule) and load
//               W[v0 + 128*rank .. +128, kb] and, per accumulator a, h[row0[a] + (N[a]/2)*rank .. , kb];
//   warp 1, 2   warp 1 allocates tensor memory (both CTAs); in the leader one thread of each issues
//               the MMAs of accumulator 0 / 1 (warp 2 only for wide tiles) and commits stage-release
//               and accumulator-ready barriers to both CTAs at once;
//   warps 3..   epilogue, one warp per TMEM lane quadrant and accumulator:
//               thread = one TMEM lane = one vocabulary entry.  32 columns (rows of h) at a time are
//               compared with the best value each row has so far (read from its key); only a chunk
//               in which some logit reaches that value is reduced (per column the warp maximum by
//               redux.sync on the order-preserving image of the logit, the lowest lane attaining it
//               by ballot) and merged into the row's packed key by a 64-bit atomic max.
// No split over k.  Every wait is bounded; a wait that runs out sets the status word, and both CTAs
// still meet at the cluster barrier before tensor memory is freed.
#include "aj_internal.cuh"
#include "aj_ptx.cuh"

#include <type_traits>

namespace aj {

namespace {

constexpr int BV = 256;       // vocabulary entries per tile (128 per CTA)
constexpr int BV_CTA = 128;
constexpr int BN = 256;       // columns of one tensor-memory buffer
constexpr int BK = 64;        // bf16 elements per k-block = 128 bytes = one swizzle span
constexpr int UMMA_K = 16;
// Warp 0 loads, warps 1 and 2 issue the MMAs of accumulator 0 and 1, the rest drain the accumulators:
// one warp per TMEM lane quadrant and accumulator.
__host__ __device__ constexpr int epilogue_warps(bool dual) { return dual ? 8 : 4; }  // four per accumulator
__host__ __device__ constexpr int num_threads(bool dual) { return 96 + 32 * epilogue_warps(dual); }
constexpr int FIRST_EPI_WARP = 3;
constexpr int A_BYTES = BV_CTA * BK * 2;   // 16 KB: this CTA's 128 rows of W, one k-block
constexpr int RING_BYTES = 224 * 1024;     // shared memory given to the stage ring (the SM has 227 KB per CTA)
constexpr int MAX_STAGES = 8;
constexpr int TMEM_COLS = 2 * BN;
constexpr int SCHED_SLOTS = 4;  // tiles a pair may have announced to its warps and not yet retired
constexpr int BAR_BYTES = 8 * (2 * MAX_STAGES + 8) + 16 + 8 * 2 * SCHED_SLOTS + 4 * SCHED_SLOTS;
constexpr int SMEM_BYTES = RING_BYTES + BAR_BYTES + 1024;

struct Tile {
    int v_tile;     // block of 256 vocabulary entries
    int row0[2];    // first row of h of each accumulator
    int n_inst[2];  // rows of each accumulator = UMMA N, a multiple of 16 (the second is 0 for narrow tiles)
    // (selected, not indexed: the struct stays in registers)
    __device__ int first_row(int a) const { return a ? row0[1] : row0[0]; }
    __device__ int rows(int a) const { return a ? n_inst[1] : n_inst[0]; }
};

// Tile t of the schedule.  Row tiles come in groups; a group is walked against every vocabulary
// block (row tile fastest) before the next group starts.  Consecutive tiles, which are taken at
// nearly the same time, share a block of W.  Which row tile of the group comes first rotates with the
// vocabulary block (with a fixed assignment of tiles to pairs this keeps a pair from always getting the
// larger, or the smaller, row tiles).  A wide tile's units of 16 rows are split over the two accumulators,
// the larger half first.
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

// DUAL: wide tiles (two accumulators, two issuing warps) instead of narrow ones.  WDV: W is stored
// [d, V].  EPI: EPI_COUNT also counts, per row, the entries that outrank the draft token (top-K
// rule); EPI_SAMPLE adds Gumbel noise to the logits before the argmax.
template <bool DUAL, bool WDV, int EPI>
__global__ void __launch_bounds__(num_threads(DUAL), 1)
umma_pair_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_h,
                 const __grid_constant__ CUtensorMap tmap_j, int M, int V, int d, PairSched sc, int stream_w, int v_offset,
                 unsigned long long *__restrict__ keys, int *__restrict__ status, const Publish pub, const RankArgs rk,
                 const Noise nz, float *__restrict__ fold_parts, int fold_stride, unsigned *__restrict__ sched) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;  // the same offset in both CTAs: one descriptor serves both
    uint8_t *smem = smem_raw + (base - raw);

    const uint32_t bar_base = base + RING_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };                                  // used in the leader only
    auto empty_bar = [&](int s) { return bar_base + 8u * (MAX_STAGES + s); };
    auto acc_full_bar = [&](int a) { return bar_base + 8u * (2 * MAX_STAGES + a); };           // a = 2 * buffer + accumulator
    auto acc_empty_bar = [&](int a) { return bar_base + 8u * (2 * MAX_STAGES + 4 + a); };      // used in the leader only
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + RING_BYTES + 8 * (2 * MAX_STAGES + 8));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    // The tiles of this pair, announced one by one by the leader's producer to every warp of both CTAs.
    const uint32_t sched_base = bar_base + 8u * (2 * MAX_STAGES + 8) + 16u;
    auto sched_full_bar = [&](int i) { return sched_base + 8u * i; };                   // one in each CTA
    auto sched_empty_bar = [&](int i) { return sched_base + 8u * (SCHED_SLOTS + i); };  // used in the leader only
    auto sched_tile_addr = [&](int i) { return sched_base + 8u * (2 * SCHED_SLOTS) + 4u * i; };
    volatile int *sched_tile = reinterpret_cast<volatile int *>(smem + RING_BYTES + 8 * (2 * MAX_STAGES + 8) + 16 + 8 * 2 * SCHED_SLOTS);

    const int warp = threadIdx.x >> 5;  // warp-uniform
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();  // 0 = leader
    const int pair = blockIdx.x >> 1;
    const int num_pairs = gridDim.x >> 1;
    const int num_kb = d / BK;
    const int num_tiles = sc.n_n * sc.n_v;
    const int fold_tile = sc.fold ? sc.n_v - 1 : -1;  // the vocabulary block that holds the classifier rows
    const int stages = sc.stages;
    const uint32_t b_bytes = (uint32_t)sc.box_rows * BK * 2;       // one accumulator's rows of h staged by this CTA
    constexpr int n_acc = DUAL ? 2 : 1;
    // A stage holds kps k-blocks (1 or 2), each [W | h of accumulator 0 | h of accumulator 1]: with two, the
    // issuing thread tests one barrier and commits once per 8 MMAs instead of per 4.
    const int kps = sc.kps;
    const uint32_t sub_bytes = A_BYTES + n_acc * b_bytes;           // one k-block of a stage: a multiple of 1024
    const uint32_t stage_bytes = (uint32_t)kps * sub_bytes;
    const uint32_t stage_tx = 2u * stage_bytes;                     // bytes both CTAs load per stage

    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_STAGES; s++) {
            mbar_init(full_bar(s), 1);   // the leader's producer; bytes arrive from both CTAs
            mbar_init(empty_bar(s), n_acc);  // one commit from each of the leader's issuing threads
        }
        for (int a = 0; a < 4; a++) {
            mbar_init(acc_full_bar(a), 1);   // the accumulator's issuing thread
            mbar_init(acc_empty_bar(a), 8);  // the four warps that drain it, in both CTAs
        }
        for (int i = 0; i < SCHED_SLOTS; i++) {
            mbar_init(sched_full_bar(i), 1);  // the leader's producer
            // every reader of the slot: the issuing threads and the follower's producer, and the epilogue warps of both CTAs
            mbar_init(sched_empty_bar(i), (DUAL ? 2 : 1) * 9 + 1);
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
    // Accumulator hand-over.  Narrow tiles: the two 256-column buffers alternate from tile to tile.
    // Wide tiles: accumulator a in buffer a.  Every buffer has its own full / empty barriers.
    auto acc_id = [&](int it, int a) { return DUAL ? a : (it & 1); };
    auto acc_col = [&](int it, int a) { return (uint32_t)(acc_id(it, a) * BN); };
    auto acc_phase = [&](int it) { return (uint32_t)(DUAL ? it : (it >> 1)) & 1u; };
    // A reader's side of the tile announcements: the it-th tile of this pair, -1 after the last one
    // (or when the wait ran out); the slot is given back once the caller's warp has read it.
    auto announced_tile = [&](int it) {
        const int slot = it & (SCHED_SLOTS - 1);
        return mbar_wait_cluster(sched_full_bar(slot), (uint32_t)(it / SCHED_SLOTS) & 1u, abort_flag) ? sched_tile[slot] : -2;
    };
    auto retire_slot = [&](int it) { mbar_arrive_cluster(map_to_cta(sched_empty_bar(it & (SCHED_SLOTS - 1)), 0)); };

    if (warp == 0) {
        if (lane == 0) {
            // ------------------------------------------------------------ TMA producer
            const unsigned long long pol_h = policy_evict_last();
            const unsigned long long pol_w = stream_w ? policy_evict_first() : policy_evict_normal();
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            // The leader's producer decides which tile comes next.  With a tile counter the pairs take
            // tiles in order as they become free: the tiles that share a block of W are then taken within
            // a short time of one another however far the pairs have drifted apart (some SM pairs run a
            // few percent slower than others), and a slower pair ends up with fewer tiles.  The first
            // tile of a pair is its own number; the counter hands out the rest.  The next tile is
            // asked for some k-blocks before the current one has been loaded, so that the answer is
            // there when it is needed.
            const int kb_ask = num_kb > 16 ? num_kb - 16 : 0;
            int t = pair < num_tiles ? pair : -1;
            for (int it = 0; ok; ++it) {
                const int slot = it & (SCHED_SLOTS - 1);
                if (rank == 0) {
                    if (it >= SCHED_SLOTS &&
                        !mbar_wait_cluster(sched_empty_bar(slot), (uint32_t)(it / SCHED_SLOTS - 1) & 1u, abort_flag)) {
                        give_up();
                        t = -1;  // still announced below: the other warps must not wait for a tile that never comes
                    }
                    sched_tile[slot] = t;
                    st_shared_cluster_u32(map_to_cta(sched_tile_addr(slot), 1), (uint32_t)t);
                    mbar_arrive_cluster(map_to_cta(sched_full_bar(slot), 0));
                    mbar_arrive_cluster(map_to_cta(sched_full_bar(slot), 1));
                } else {
                    t = announced_tile(it);
                    if (t == -2) give_up();
                    retire_slot(it);
                }
                if (t < 0) break;
                const Tile tl = decode_tile(sc, t);
                const bool fold = tl.v_tile == fold_tile;
                const CUtensorMap *tw = fold ? &tmap_j : &tmap_w;  // the classifier rows start at entry 0 of their own map
                const int w_row = (fold ? 0 : tl.v_tile * BV) + (int)rank * BV_CTA;
                const int h_row0 = tl.row0[0] + (int)rank * (tl.n_inst[0] >> 1);
                const int h_row1 = tl.row0[1] + (int)rank * (tl.n_inst[1] >> 1);
                int next = -1;
                for (int kb = 0; kb < num_kb; kb += kps) {
                    // (the answer is not looked at before the loop ends: the thread does not wait for it here)
                    if (rank == 0 && kb <= kb_ask && kb_ask < kb + kps) next = sched ? (int)atomicAdd(sched, 1u) + num_pairs : t + num_pairs;
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) {
                        give_up();
                        ok = false;
                        break;
                    }
                    const uint32_t leader_full = map_to_cta(full_bar(s), 0);
                    if (rank == 0) mbar_expect_tx(full_bar(s), stage_tx);
                    for (int j = 0; j < kps; j++) {
                        const uint32_t a_dst = base + s * stage_bytes + j * sub_bytes;
                        const int kc = (kb + j) * BK;
                        if (WDV) {  // W stored [d, V]: two boxes of 64 entries x 64 k-rows
                            tma_load_2d_pair(a_dst, tw, w_row, kc, leader_full, pol_w);
                            tma_load_2d_pair(a_dst + A_BYTES / 2, tw, w_row + 64, kc, leader_full, pol_w);
                        } else {
                            tma_load_2d_pair(a_dst, tw, kc, w_row, leader_full, pol_w);
                        }
                        tma_load_2d_pair(a_dst + A_BYTES, &tmap_h, kc, h_row0, leader_full, pol_h);
                        if (n_acc == 2) tma_load_2d_pair(a_dst + A_BYTES + b_bytes, &tmap_h, kc, h_row1, leader_full, pol_h);
                    }
                    if (++s == stages) {
                        s = 0;
                        ph ^= 1u;
                    }
                }
                t = next < num_tiles ? next : -1;
            }
            if (rank == 0) {
                // The pair that leaves last puts the counter back to zero for the next launch; each pair has
                // drawn its last number from it before it is counted here.
                if (sched) {
                    __threadfence();
                    if (atomicInc(sched + 1, (unsigned)num_pairs - 1u) == (unsigned)num_pairs - 1u) atomicExch(sched, 0u);
                }
            }
        }
    } else if (warp <= 2) {
        if (lane == 0 && rank == 0 && warp <= n_acc) {
            // --------------------- MMA issuer of accumulator a = warp - 1 (leader CTA only)
            // (rebuilding the descriptors per k-block measured slightly faster than stepping them
            // from stage to stage, which chains every k-block's issue to the previous one)
            const int a = warp - 1;
            constexpr unsigned long long a_step = WDV ? MN_KSTEP : 2ull;
            constexpr uint32_t a_major = WDV ? IDESC_A_MN_MAJOR : 0u;
            const uint32_t b_off = A_BYTES + (uint32_t)a * b_bytes;
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int it = 0; ok; ++it) {
                const int t = announced_tile(it);
                if (t == -2) give_up();
                retire_slot(it);
                if (t < 0) break;
                const Tile tl = decode_tile(sc, t);
                const int n_inst = tl.rows(a);  // 0: this accumulator has no rows in this tile (one unit of 16); the barriers still turn
                const uint32_t idesc = instr_desc(BV, n_inst) | a_major;
                if (!mbar_wait(acc_empty_bar(acc_id(it, a)), acc_phase(it) ^ 1u, abort_flag)) {
                    give_up();
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc_col(it, a);
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
                        const unsigned long long bdesc = smem_desc_sw128(a_addr + b_off);
                        if (n_inst) {
#pragma unroll
                            for (int k = 0; k < BK / UMMA_K; k++)
                                umma_bf16_pair(d_tmem, adesc + a_step * k, bdesc + 2ull * k, idesc, (uint32_t)((kb | j | k) != 0));
                        }
                    }
                    umma_commit_pair(empty_bar(s));  // this accumulator is done with the stage, in both CTAs
                    if (++s == stages) {
                        s = 0;
                        ph ^= 1u;
                    }
                }
                if (ok) umma_commit_pair(acc_full_bar(acc_id(it, a)));  // the accumulator is complete in both CTAs
            }
        }
    } else {
        // -------------------------------------------------------------------- epilogue
        // A logit can only matter if it reaches the best value its row has so far.  Lane j reads
        // the key of the row of column 32c + j before the accumulator is ready (a stale key is only
        // lower, never wrong); its high half is that value as an ordered integer.  A chunk of 32
        // columns is first tested against the LOWEST of its 32 thresholds (one redux.sync.min, and
        // per lane the maximum of its 32 logits): nearly every chunk ends there.  Otherwise the
        // elements are compared one by one with the shuffled-in thresholds, and only if some
        // element qualifies does the chunk take the reduction path (warp maximum per column by
        // redux.sync, lowest lane by ballot, 64-bit atomic max into the key).
        const int q = warp & 3;  // TMEM lane quadrant this warp may read
        const int a = DUAL ? (warp - FIRST_EPI_WARP) >> 2 : 0;              // the accumulator this warp drains
        constexpr int CH = BN / 32;                                         // 32-column chunks per accumulator
        constexpr uint32_t NO_ROW = 0xFFFFFFFFu;  // above every value: nothing qualifies
        // Chunk c is columns 32 c .. + 32 of the accumulator.  Only the high half of the key is read,
        // the best value as an ordered integer; 0 = the row has no key yet.
        auto load_key = [&](const Tile &tl, int c) {
            const int col = c * 32 + lane;
            const int row = tl.first_row(a) + col;
            if (col >= tl.rows(a) || row >= M) return NO_ROW;
            return __ldcg(reinterpret_cast<const uint32_t *>(keys + row) + 1);
        };
        // All of the accumulator's keys are fetched before it is ready, so no chunk waits for an L2
        // round trip.  The chunk loop is kept rolled, one copy of its code stays in the instruction
        // cache: the keys rotate through kk[0].
        for (int it = 0;; ++it) {
            int t = announced_tile(it);
            if (__any_sync(0xffffffffu, t == -2)) {  // the whole warp takes one decision
                give_up();
                t = -2;
            }
            __syncwarp();
            if (lane == 0) retire_slot(it);
            if (t < 0) break;
            const Tile tl = decode_tile(sc, t);
            uint32_t kk[CH];
#pragma unroll
            for (int i = 0; i < CH; i++) kk[i] = load_key(tl, i);
            // top-K rule: the thresholds and draft tokens of the accumulator's rows, fetched ahead like the keys
            float thp[EPI == EPI_COUNT ? CH : 1];
            int tkp[EPI == EPI_COUNT ? CH : 1];
            if (EPI == EPI_COUNT) {
#pragma unroll
                for (int i = 0; i < CH; i++) {
                    const int col = i * 32 + lane, row = tl.first_row(a) + col;
                    const bool valid = col < tl.rows(a) && row < M;
                    thp[i] = rank_threshold(rk, row, valid);
                    tkp[i] = valid ? __ldg(rk.tok + row) : -1;
                }
            }
            const int v_first = tl.v_tile * BV + (int)rank * BV_CTA + q * 32;  // vocabulary entry of lane 0
            const bool v_ok = v_first + lane < V;                            // entries past V hold zero-filled junk
            const uint32_t tbase = tmem_base + ((uint32_t)(q * 32) << 16);
            // the whole warp takes one decision, so the aligned TMEM loads below stay converged
            if (!__all_sync(0xffffffffu, mbar_wait(acc_full_bar(acc_id(it, a)), acc_phase(it), abort_flag))) {
                give_up();
                break;
            }
            tc_fence_after();
            const int n_inst = tl.rows(a), row_a = tl.first_row(a);
#pragma unroll 1
            for (int c = 0; c * 32 < n_inst; c++) {
                const uint32_t kthr = kk[0];
#pragma unroll
                for (int i = 0; i + 1 < CH; i++) kk[i] = kk[i + 1];
                const float th_c = thp[0];
                const int tk_c = tkp[0];
                if (EPI == EPI_COUNT) {
#pragma unroll
                    for (int i = 0; i + 1 < CH; i++) thp[i] = thp[i + 1], tkp[i] = tkp[i + 1];
                }
                {
                    float v[32];
                    tmem_ld32(tbase + acc_col(it, a) + (uint32_t)(c * 32), v);
                    if (tl.v_tile == fold_tile) {
                        // the classifier rows: lanes 0..2 of the leader's first quadrant hold the three partial
                        // dot products of 32 rows of h; they are stored, and nothing of this block is a logit
                        if (rank == 0 && q == 0 && lane < JUDGE_FOLD_ROWS) {
#pragma unroll
                            for (int j = 0; j < 32; j++) {
                                const int row = row_a + c * 32 + j;
                                if (c * 32 + j < n_inst && row < M) fold_parts[(size_t)lane * fold_stride + row] = v[j];
                            }
                        }
                        continue;
                    }
                    // the lowest threshold of the chunk (a row without a key yet: everything qualifies)
                    const uint32_t tmin = warp_min_u32(kthr);
                    if (EPI == EPI_SAMPLE) {
                        float pmax = v[0];  // of the plain logits
#pragma unroll
                        for (int j = 1; j < 32; j++) pmax = fmaxf(pmax, v[j]);
                        const uint32_t k_need = noise_cutoff(key_value((unsigned long long)tmin << 32), pmax, nz.inv_temperature);
                        if (!add_gumbel_noise(nz, v, v_first + lane + v_offset, row_a + c * 32, k_need)) continue;
                    }
                    float vmax = v[0];
#pragma unroll
                    for (int j = 1; j < 32; j++) vmax = fmaxf(vmax, v[j]);
                    if (EPI == EPI_COUNT) {
                        const int row = row_a + c * 32 + lane;
                        count_outranking(rk, v, vmax, v_first, v_ok, th_c, tk_c, row, c * 32 + lane < n_inst && row < M, lane);
                    }
                    if (__any_sync(0xffffffffu, v_ok && ordered_image(vmax) >= tmin)) {
                        const float thr = kthr == NO_ROW ? __int_as_float(0x7fc00000)  // NaN: no comparison with it is ever true
                                          : kthr == 0u  ? -INFINITY
                                                        : key_value((unsigned long long)kthr << 32);
                        bool hit = false;
#pragma unroll
                        for (int j = 0; j < 32; j++) hit |= v[j] >= __shfl_sync(0xffffffffu, thr, j);
                        if (__any_sync(0xffffffffu, hit && v_ok)) {
                            // all 32 reductions are issued before any result is used, so that their
                            // latencies overlap instead of adding up
                            uint32_t x[32], m[32];
#pragma unroll
                            for (int j = 0; j < 32; j++) x[j] = v_ok ? ordered_image(v[j]) : 0u;
#pragma unroll
                            for (int j = 0; j < 32; j++) m[j] = warp_max_u32(x[j]);
                            uint32_t best_u = 0u;  // lane j: maximum of column 32c + j over this warp's 32 entries
                            int best_i = 0;
#pragma unroll
                            for (int j = 0; j < 32; j++) {
                                const uint32_t who = __ballot_sync(0xffffffffu, x[j] == m[j]);
                                if (lane == j) {
                                    best_u = m[j];
                                    best_i = v_first + __ffs(who) - 1;  // the lowest entry that attains the maximum
                                }
                            }
                            const int row = row_a + c * 32 + lane;
                            if (c * 32 + lane < n_inst && row < M && best_u != 0u) {
                                const unsigned long long key =
                                    ((unsigned long long)best_u << 32) | (uint32_t)(~(uint32_t)(best_i + v_offset));
                                if (key > *reinterpret_cast<volatile unsigned long long *>(&keys[row])) atomicMax(&keys[row], key);
                            }
                        }
                    }
                }
            }
            // the accumulator is drained: hand it back to its issuing thread in the leader
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(acc_empty_bar(acc_id(it, a)), 0));
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
    cfg.blockDim = dim3(num_threads(true));  // the largest block: residency is the same, one CTA per SM
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

PairSched pair_schedule(int M, int V, int d, int fold) {
    PairSched sc;
    sc.fold = fold ? 1 : 0;
    const int units = (M + 15) / 16;  // rows in units of 16 (the UMMA N granule)
    // Wide tiles (up to 512 rows on two accumulators with an issuing warp each) for every batch of more
    // than 256 rows; up to 256 rows one narrow tile per vocabulary block, double-buffered.
    sc.dual = units > 16 ? 1 : 0;
    const int cap = sc.dual ? 32 : 16;
    sc.n_n = (units + cap - 1) / cap;
    sc.u_base = units / sc.n_n;
    sc.u_rem = units % sc.n_n;
    sc.n_v = (V + BV - 1) / BV + sc.fold;
    const int u_max = sc.u_base + (sc.u_rem ? 1 : 0);
    // rows of h each CTA stages per accumulator: half of the largest accumulator
    sc.box_rows = 8 * (sc.dual ? (u_max + 1) / 2 : u_max);
    // An issuing thread spends about 546 cycles on a k-block, 130 of them on the barrier test and the commit,
    // and up to some 160 rows per accumulator that, not the tensor pipe, is what a tile waits for.  Two
    // k-blocks per stage halve that share; taken where three such stages still fit (tiles of up to 320 rows:
    // 136 rows 220 -> 191 us, 264 rows 267 -> 247, 520 rows 483 -> 436, 576 rows 503 -> 469; with two stages
    // left, or on the tiles the pipe bounds, it costs 2 ... 8 % instead).
    const int sub_bytes = A_BYTES + (sc.dual ? 2 : 1) * sc.box_rows * BK * 2;
    sc.kps = ((d / BK) % 2 == 0 && RING_BYTES / (2 * sub_bytes) >= 3) ? 2 : 1;
    const int stage_bytes = sc.kps * sub_bytes;
    sc.stages = RING_BYTES / stage_bytes < MAX_STAGES ? RING_BYTES / stage_bytes : MAX_STAGES;
    // row tiles per group: keep a group's rows of h (tile rows x d x 2 bytes) within about 40 MB of L2
    const long long tile_bytes = (sc.dual ? 512ll : 256ll) * d * 2;
    int g_max = (int)((40ll << 20) / tile_bytes);
    if (g_max < 1) g_max = 1;
    sc.n_groups = (sc.n_n + g_max - 1) / g_max;
    sc.g_base = sc.n_n / sc.n_groups;
    sc.g_rem = sc.n_n % sc.n_groups;
    return sc;
}

cudaError_t launch_umma_pair(const GemmArgs &a, const UmmaPlan &p, cudaStream_t stream) {
    const PairSched sc = pair_schedule(a.M, a.V, a.d, a.fold.rows != nullptr);
    // W is not kept in L2 when one pair reads each block, nor when the tiles are shared out by the counter:
    // the pairs that share a block then read it within microseconds of one another, and a block of W that
    // lingers only pushes h_target out (2080 x 8192 rows against 128256 entries: 2.21 GB of DRAM reads per
    // launch instead of 2.80, and 3.9 with the fixed order, against 2.14 GB of operands)
    const int stream_w = (sc.n_n == 1 || a.sched) ? 1 : 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.grid);  // 2 CTAs per pair
    cfg.blockDim = dim3(num_threads(sc.dual != 0));
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
    return cudaLaunchKernelEx(&cfg, kernel, p.tmap_w, p.tmap_h, a.fold.rows ? p.tmap_j : p.tmap_w, a.M, a.V, a.d, sc, stream_w,
                              a.v_offset, a.keys, a.status, a.pub, a.rank, a.noise, a.fold.parts, a.fold.stride, a.sched);
}

}  // namespace aj
