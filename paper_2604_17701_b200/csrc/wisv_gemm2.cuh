// LM-head GEMM + row reduction with the operands swapped: the VOCABULARY on the M side of a CTA-pair MMA
// (tcgen05 cta_group::2, M = 256: 128 weight rows per CTA) and the WINDOW ROWS on the N side, for batches of
// more than 128 window rows.
//
// Why: one tcgen05.mma (K = 16) occupies the tensor pipe for N / 2 SM clocks per CTA whatever its M once N >= 128
// (measured: 128 x N and 64 x N cost the same).  With the window rows on the 128-row M side a batch pays for its
// row count rounded up to 128 (256 for a pair): 144 rows cost as much as 256, 288 rows as much as 384, 576 as
// much as 640.  On the N side the granularity is 16 rows: the batch is cut into ceil(R / 256) row blocks of equal
// width N (a multiple of 16, at most 256) and an MMA costs N / 2 clocks, so the tensor pipe is busy in proportion to
// the rows that exist.  Each CTA also loads only half of a block's activation rows per K block (the pair MMA takes
// the two halves of its B operand from the two CTAs).
//
// D[vocabulary row (TMEM lane), window row (TMEM column)].  A window row's statistics therefore run ACROSS lanes:
// each epilogue warp moves 32 lanes x 32 columns at a time through a padded shared-memory buffer, after which
// lane L owns column L of the chunk and scans that window row's 32 logits in ascending vocabulary order (strict
// '>' keeps the lowest token id).  The running (max, argidx, sum exp) of a window row lives in the registers of
// the lane that owns its column, per warp; the four warps of a CTA are then merged in vocabulary order.
//
// Three ways of dealing out the work:
//  * one row block (up to 256 rows, bound by HBM): every pair owns one contiguous range of the vocabulary (units of
//    32 rows, tiles of tile_m or tile_m - 32 rows, balanced to one unit), carries its running row state across its
//    tiles and writes one partial per (row, CTA) at the end;
//  * a few row blocks (2-4 in practice): the pairs form one team per row block and every team deals out the
//    vocabulary as above, so a row still gets one partial per CTA of its team (48 instead of 1002 at 576 rows and 8B
//    shapes) and nothing is merged or written between tiles; the k-th pairs of all teams stream the same range at the
//    same time and share its weight tiles through L2.  Chosen when the teams need no more tiles per pair than the
//    round-robin below needs rounds;
//  * many row blocks (bound by the tensor pipe at N = 256): work items (vocabulary tile of 256 rows, row block) are dealt
//    out round-robin, row blocks of a group fastest, so the pairs that run at the same time share a weight tile
//    through L2 and a group's activation rows stay resident there; one partial per (row, vocabulary tile, CTA).
//
// Barriers: full[s] in the leader counts both CTAs' bytes, empty[s] / acc_full[a] are signalled
// in both CTAs by a multicast tcgen05.commit, acc_empty[a] in the leader collects the epilogue warps of both CTAs.
// No load uses multicast; every wait is bounded.
#pragma once

#include "wisv_gemm.cuh"

namespace wisv {

constexpr int kPairTileM = 256;              // vocabulary rows of a pair tile (the M of the MMA): 128 per CTA
constexpr int kPairTileN = kPairTileM;       // (the same number where it counts rows of the weight matrix)
constexpr int kPairMaxCols = 256;            // window rows per row block (the N of the MMA)
constexpr int kPairChunk = 32;               // columns moved through shared memory at a time
constexpr int kPairPitch = 36;               // floats per column in the transposition buffer (16-byte rows, no bank conflicts)
constexpr int kPairMaxChunks = kPairMaxCols / kPairChunk;

struct PairParams {
    int32_t rows;        // valid window rows
    int32_t n_cols;      // N of the MMA = width of a row block: a multiple of 16, at most 256
    int32_t row_blocks;  // ceil(rows / n_cols)
    int32_t n_total;     // vocabulary size
    int32_t k_blocks;
    int32_t stages;
    int32_t kbs;         // K blocks per stage (1, 2 or 4): one barrier round trip, on both sides of the ring, serves kbs K blocks
    int32_t box3d;       // 1: the tensor maps are 3-D (column in a K block, row, K block) with boxes of kbs K blocks, so one
                         // TMA instruction per operand fills a stage (each instruction costs the producer about 80 clocks
                         // on top of about 440 per stage); needs H % 64 == 0.  A weight block then takes its real height
                         // in shared memory, not a 128-row slot.
    // one row block (carry = 1): vocabulary ranges in units of 32 rows per pair - units_base units, one more for the
    // first units_rem pairs - cut into tiles_per_pair tiles of tile_m or tile_m - 32 rows
    int32_t carry, units_base, units_rem, tiles_per_pair, tile_m;
    // carry with several row blocks: the pairs form row_blocks teams of team_pairs pairs; team j streams the whole
    // vocabulary for row block j, its k-th pair the k-th range, so the pairs that work on one range at the same time
    // (one per team) share its weight tiles through L2.  One row block: one team of all pairs.
    int32_t team_pairs;
    // several row blocks (carry = 0): n_tiles vocabulary tiles of 256 rows; items run group by group (all vocabulary
    // tiles of a group of b_group row blocks before the next group)
    int32_t n_tiles, b_group;
    int32_t part_stride; // partials per row: 2 per pair of a team (carry) or 2 per vocabulary tile
    int32_t* err;
    float4* lm_part;
    const int32_t* row_tok;
    float* tok_logit;
};

__host__ __device__ inline uint32_t pair_stage_bytes(int n_cols, int kbs = 1) {
    return static_cast<uint32_t>(kbs) * static_cast<uint32_t>(kTileM * kBlockK * 2 + (n_cols / 2) * kBlockK * 2);
}
// alignment slack + barriers, then the four warps' transposition buffers
__host__ __device__ inline uint32_t pair_fixed_bytes() {
    return 1024u + 1024u + 4u * kPairChunk * kPairPitch * 4u;
}

// 2^x for x <= 0 by the hardware approximation alone (relative error 2^-22; results below 2^-126 become 0):
// exp2f() wraps the same instruction in a range fix-up that a sum of exponentials of non-positive numbers does not need.
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ void pair_merge(float& mx, int& arg, float& sum, float omx, int oarg, float osum) {
    if (omx == -CUDART_INF_F && osum == 0.0f) return;
    if (omx > mx) {
        sum = sum * exp2f((mx - omx) * 1.4426950408889634f) + osum;      // exp2(-inf) = 0 covers an empty left side
        mx = omx; arg = oarg;
    } else {
        sum += osum * exp2f((omx - mx) * 1.4426950408889634f);
        if (omx == mx && oarg < arg) arg = oarg;
    }
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1)
lmhead_pair_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW,
                   const __grid_constant__ CUtensorMap tmW2, const PairParams p,
                   const __grid_constant__ CUtensorMap tmZ, const __grid_constant__ CUtensorMap tmW1,
                   const __grid_constant__ CUtensorMap tmW1_2, const GemmParams hd, const int lm_ctas,
                   const int head_ctas)
{
    if (static_cast<int>(blockIdx.x) >= lm_ctas) {
        // whole clusters beyond the pairs evaluate the decision head with the single-CTA GEMM body
        // (the grid is a whole number of clusters: with an odd head_ctas the last CTA has nothing to do)
        const int hc = static_cast<int>(blockIdx.x) - lm_ctas;
        if (hc < head_ctas) gemm_rowreduce_body<EPI_HEAD, false>(tmZ, tmW1, tmW1_2, hd, hc, head_ctas);
        return;
    }
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t pad = ((raw_addr + 1023u) & ~1023u) - raw_addr;
    uint8_t* smem = smem_raw + pad;
    const uint32_t smem_base = raw_addr + pad;

    const uint32_t rank = cluster_ctarank();
    const bool leader = rank == 0;
    const int pair_id = blockIdx.x >> 1;
    const int n_pairs = lm_ctas >> 1;
    const uint32_t a_bytes = kTileM * kBlockK * 2;                                   // weight slot: 128 rows
    const uint32_t b_bytes = static_cast<uint32_t>(p.n_cols / 2) * kBlockK * 2;     // this CTA's half of a row block
    // a stage holds kbs K blocks: [weights of block 0 .. kbs-1][window rows of block 0 .. kbs-1]
    const uint32_t stage_bytes = static_cast<uint32_t>(p.kbs) * (a_bytes + b_bytes);
    const uint32_t x_off = static_cast<uint32_t>(p.kbs) * a_bytes;
    const uint32_t ring_bytes = stage_bytes * static_cast<uint32_t>(p.stages);

    const uint32_t bar_base = smem_base + ring_bytes;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kMaxStages + s); };
    auto acc_full_bar = [&](int s) { return bar_base + 8u * (2 * kMaxStages + s); };
    auto acc_empty_bar = [&](int s) { return bar_base + 8u * (2 * kMaxStages + 2 + s); };
    const uint32_t drain_bar = bar_base + 8u * (2 * kMaxStages + 4);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + ring_bytes + 8 * (2 * kMaxStages + 5));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);   // [0] abort, [1] drain scratch
    float* trans_base = reinterpret_cast<float*>(smem + ring_bytes + 1024);      // 4 x [32 columns][36]

    const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0);   // the same in all lanes, and the compiler knows it
    const int lane = threadIdx.x & 31;
    // carry: this pair's team (row block) and place in it, its contiguous range of 32-row units and how that is cut
    // into tiles
    const int team = p.carry ? pair_id / p.team_pairs : 0;
    const int team_k = p.carry ? pair_id - team * p.team_pairs : 0;
    const int my_units = p.units_base + (team_k < p.units_rem ? 1 : 0);
    const int my_unit0 = team_k * p.units_base + (team_k < p.units_rem ? team_k : p.units_rem);
    const int my_tiles = p.carry ? (my_units < p.tiles_per_pair ? my_units : p.tiles_per_pair) : 0;
    const int my_hq = p.carry ? my_units / p.tiles_per_pair : 0;
    const int my_hr = p.carry ? my_units % p.tiles_per_pair : 0;
    const int total_items = p.n_tiles * p.row_blocks;
    // the i-th work item of this pair: vocabulary tile (index n, first row n0, height h, a multiple of 32) x row block j
    struct Item { int n, n0, h, j; };
    auto item_at = [&](int i, Item& w) -> bool {
        if (p.carry) {
            if (i >= my_tiles) return false;
            w.n = team_k; w.j = team;
            w.h = (my_hq + (i < my_hr ? 1 : 0)) * 32;
            w.n0 = (my_unit0 + i * my_hq + (i < my_hr ? i : my_hr)) * 32;
            return true;
        }
        const int t = pair_id + i * n_pairs;
        if (t >= total_items) return false;
        // groups of b_group row blocks; inside a group the row block runs fastest
        const int per_group = p.b_group * p.n_tiles;
        const int g = t / per_group;
        const int j0 = g * p.b_group;
        const int gsize = min(p.b_group, p.row_blocks - j0);
        const int idx = t - g * per_group;
        w.n = idx / gsize;
        w.j = j0 + idx % gsize;
        w.n0 = w.n * kPairTileN;
        w.h = kPairTileN;
        return true;
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(acc_full_bar(s), 1); mbar_init(acc_empty_bar(s), 8); }
        mbar_init(drain_bar, 1);
        abort_flag[0] = 0;
        abort_flag[1] = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmX);
        tma_prefetch_desc(&tmW);
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(tmem_slot), kTmemCols);
        tmem_relinquish_pair();
    }
    // both CTAs' barriers and TMEM must exist before either touches the other's
    tc_fence_before();
    __syncwarp();
    cluster_arrive();
    cluster_wait();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // The pack kernel wrote the bf16 rows this kernel loads: everyone waits for it here, except the producer warp,
    // which first puts one ring-full of weight tiles in flight (they depend on nothing) and waits then.
    if (warp != 0) {
        griddep_wait();
        griddep_launch_dependents();
    }

    // producer warp: stages issued so far, the same in all its lanes (read again by the drain before the kernel ends)
    long long prod_issued = 0;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (each CTA)
        // The WHOLE warp runs these loops and one elected lane issues: tcgen05.mma, tcgen05.commit and the TMA
        // instructions take their operands from uniform registers, which the compiler can only use in code that the
        // warp runs together.  Written as the work of one thread inside `if (lane == 0)`, the same loops cost 470
        // clocks per stage plus 75 per TMA issue here and 57-74 clocks per MMA in the warp below (measured), more
        // than the tensor pipe needs for the MMAs of a narrow row block.  Plain counters and nested loops only: a
        // 64-bit division per K block in this loop doubled the kernel's time.
        Item w;
        int pre = 0;                               // stages whose weight half-tiles were requested before the wait
        for (int i = 0; pre < p.stages && item_at(i, w); ++i) {
            const int half_h = w.h >> 1;
            const int w_row0 = w.n0 + static_cast<int>(rank) * half_h;
            const CUtensorMap* mapW = (w.h == p.tile_m) ? &tmW : &tmW2;
            for (int kb = 0; kb < p.k_blocks && pre < p.stages; kb += p.kbs, ++pre) {
                const int nb = min(p.kbs, p.k_blocks - kb);
                const uint32_t dst = smem_base + stage_bytes * static_cast<uint32_t>(pre);
                // a 3-D box always brings kbs K blocks (zeros past the end of K)
                const uint32_t tx = 2u * static_cast<uint32_t>(p.box3d ? p.kbs : nb) *
                                    (static_cast<uint32_t>(half_h) * kBlockK * 2u + b_bytes);
                if (elect_one()) {
                    if (leader) mbar_expect_tx(full_bar(pre), tx);          // both CTAs' bytes
                    if (p.box3d) {
                        tma_load_3d_pair(dst, mapW, 0, w_row0, kb, full_bar(pre));
                    } else {
                        for (int u = 0; u < nb; ++u)
                            tma_load_2d_pair(dst + static_cast<uint32_t>(u) * a_bytes, mapW, (kb + u) * kBlockK, w_row0, full_bar(pre));
                    }
                }
                __syncwarp();
            }
        }
        griddep_wait();
        griddep_launch_dependents();
        {
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int i = 0; ok && item_at(i, w); ++i) {
                const int half_h = w.h >> 1;                                   // weight rows this CTA loads
                const int w_row0 = w.n0 + static_cast<int>(rank) * half_h;
                const int x_row0 = w.j * p.n_cols + static_cast<int>(rank) * (p.n_cols / 2);   // its half of the row block
                const CUtensorMap* mapW = (w.h == p.tile_m) ? &tmW : &tmW2;
                const uint32_t tx_w = static_cast<uint32_t>(half_h) * kBlockK * 2u + b_bytes;
                for (int kb = 0; kb < p.k_blocks; kb += p.kbs) {
                    const int nb = min(p.kbs, p.k_blocks - kb);
                    const uint32_t dst = smem_base + stage_bytes * static_cast<uint32_t>(s);
                    const bool fresh = prod_issued >= pre;    // else: first pass over the ring, the stage is free and
                                                              // its weight half-tiles are on their way
                    if (fresh) {
                        ok = __all_sync(0xffffffffu, mbar_wait_bounded(empty_bar(s), ph ^ 1u, abort_flag, kWaitLimitClocks));
                        if (!ok) break;
                    }
                    if (elect_one()) {
                        if (p.box3d) {
                            if (fresh) {
                                if (leader) mbar_expect_tx(full_bar(s), 2u * static_cast<uint32_t>(p.kbs) * tx_w);
                                tma_load_3d_pair(dst, mapW, 0, w_row0, kb, full_bar(s));
                            }
                            tma_load_3d_pair(dst + x_off, &tmX, 0, x_row0, kb, full_bar(s));
                        } else {
                            if (fresh) {
                                if (leader) mbar_expect_tx(full_bar(s), 2u * static_cast<uint32_t>(nb) * tx_w);
                                for (int u = 0; u < nb; ++u)
                                    tma_load_2d_pair(dst + static_cast<uint32_t>(u) * a_bytes, mapW, (kb + u) * kBlockK, w_row0, full_bar(s));
                            }
                            for (int u = 0; u < nb; ++u)
                                tma_load_2d_pair(dst + x_off + static_cast<uint32_t>(u) * b_bytes, &tmX, (kb + u) * kBlockK, x_row0, full_bar(s));
                        }
                    }
                    __syncwarp();
                    ++prod_issued;
                    if (++s == p.stages) { s = 0; ph ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader CTA only; see the producer
        // for why the whole warp runs the loop)
        if (leader) {
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            Item w;
            // M = 256 whatever the tile height: weight rows that were not loaded feed lanes nobody reads
            const uint32_t idesc = idesc_bf16_f32(kPairTileM, static_cast<uint32_t>(p.n_cols));
            for (int local = 0; ok && item_at(local, w); ++local) {
                const int as = local & 1;
                const uint32_t aph = (local >> 1) & 1u;
                ok = __all_sync(0xffffffffu, mbar_wait_bounded(acc_empty_bar(as), aph ^ 1u, abort_flag, kWaitLimitClocks));
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(as * kAccCols);
                // bytes between the weight blocks of a stage
                const uint32_t a_blk = p.box3d ? static_cast<uint32_t>(w.h >> 1) * kBlockK * 2u : a_bytes;
                for (int kb = 0; kb < p.k_blocks; kb += p.kbs) {
                    const int nb = min(p.kbs, p.k_blocks - kb);
                    ok = __all_sync(0xffffffffu, mbar_wait_bounded(full_bar(s), ph, abort_flag, kWaitLimitClocks));
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t st_addr = smem_base + stage_bytes * s;
                    const uint64_t a_desc0 = smem_desc_k128(st_addr);             // weights: the M side
                    const uint64_t b_desc0 = smem_desc_k128(st_addr + x_off);     // window rows: the N side
                    const bool last = kb + nb >= p.k_blocks;
                    if (elect_one()) {
                        for (int u = 0; u < nb; ++u) {
                            const uint64_t a_desc = a_desc0 + static_cast<uint64_t>((static_cast<uint32_t>(u) * a_blk) >> 4);
                            const uint64_t b_desc = b_desc0 + static_cast<uint64_t>((static_cast<uint32_t>(u) * b_bytes) >> 4);
#pragma unroll
                            for (int k = 0; k < kBlockK / kUmmaK; ++k)
                                umma_bf16_pair(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, (kb | u | k) != 0 ? 1u : 0u);
                        }
                        umma_commit_pair(empty_bar(s));                    // frees the stage in both CTAs
                        if (last) umma_commit_pair(acc_full_bar(as));      // accumulator ready in both CTAs
                    }
                    __syncwarp();
                    if (++s == p.stages) { s = 0; ph ^= 1u; }
                }
            }
            if (!ok) {
                if (elect_one()) umma_commit_pair(drain_bar);
                __syncwarp();
                mbar_wait_bounded(drain_bar, 0, abort_flag + 1, kWaitLimitClocks);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..5 of each CTA)
        const int q = warp & 3;                                  // TMEM lane quadrant of this warp
        const int ew = warp - 2;                                 // buffer of this warp
        const int et = threadIdx.x - 64;                         // 0..127 among the epilogue threads
        float* tbuf = trans_base + ew * (kPairChunk * kPairPitch);
        // merge buffer [quadrant][column] (float4): 4 * 256 * 16 B = 16 KB, laid over the transposition buffers
        float4* comb = reinterpret_cast<float4*>(trans_base);
        bool ok = true;
        const uint32_t leader_acc_empty0 = mapa_u32(acc_empty_bar(0), 0);
        const uint32_t leader_acc_empty1 = mapa_u32(acc_empty_bar(1), 0);
        const int n_chunks = (p.n_cols + kPairChunk - 1) / kPairChunk;
        // lane L owns columns L, L + 32, ... of the row block: running state and draft token of each
        float mx[kPairMaxChunks], sum[kPairMaxChunks];
        int arg[kPairMaxChunks], tokc[kPairMaxChunks];
        auto reset_state = [&](int j) {
#pragma unroll
            for (int u = 0; u < kPairMaxChunks; ++u) {
                mx[u] = -CUDART_INF_F; sum[u] = 0.0f; arg[u] = 0x7fffffff;
                const int r = j * p.n_cols + u * kPairChunk + lane;
                tokc[u] = (u < n_chunks && u * kPairChunk + lane < p.n_cols && r < p.rows) ? p.row_tok[r] : -1;
            }
        };
        // merge the four warps of this CTA in vocabulary order (warp q covers TMEM lanes 32q..) and write one
        // partial per row of row block j to slot `slot` of the row's partials
        auto flush_state = [&](int j, int slot) {
            asm volatile("bar.sync 1, 128;" ::: "memory");        // every warp is done with its transposition buffer
#pragma unroll
            for (int u = 0; u < kPairMaxChunks; ++u) {
                const int c = u * kPairChunk + lane;
                if (u < n_chunks && c < p.n_cols)
                    comb[q * kPairMaxCols + c] = make_float4(mx[u], __int_as_float(arg[u]), sum[u], 0.0f);
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");
            for (int c = et; c < p.n_cols; c += kEpiThreads) {
                const int r = j * p.n_cols + c;
                if (r >= p.rows) break;
                float m = -CUDART_INF_F, sm = 0.0f;
                int a = 0x7fffffff;
#pragma unroll
                for (int qq = 0; qq < 4; ++qq) {
                    const float4 f = comb[qq * kPairMaxCols + c];
                    pair_merge(m, a, sm, f.x, __float_as_int(f.y), f.z);
                }
                p.lm_part[(size_t)r * p.part_stride + slot] = make_float4(m, __int_as_float(a), sm, 0.0f);
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");        // the buffer goes back to the transposition
        };
        if (p.carry) reset_state(team);
        Item w;
        for (int local = 0; ok && item_at(local, w); ++local) {
            const int as = local & 1;
            const uint32_t aph = (local >> 1) & 1u;
            const int half_h = w.h >> 1;
            const int warp_v0 = w.n0 + static_cast<int>(rank) * half_h + q * 32;    // token of this warp's first lane
            const bool lane_valid = (q * 32 + lane < half_h) && (warp_v0 + lane < p.n_total);
            const int row0 = w.j * p.n_cols;                                         // first window row of the block
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + static_cast<uint32_t>(as * kAccCols);
            if (!p.carry) reset_state(w.j);

            bool got = mbar_wait_bounded(acc_full_bar(as), aph, abort_flag, kWaitLimitClocks);
            {
                // The four warps must agree on `got`: they meet at barriers inside flush_state, and after a time-out
                // one warp may have seen the abort flag while another still saw the accumulator arrive.
                uint32_t all;
                asm volatile(
                    "{\n\t"
                    ".reg .pred pi, po;\n\t"
                    "setp.ne.u32 pi, %1, 0;\n\t"
                    "barrier.cta.red.and.pred po, 1, 128, pi;\n\t"
                    "selp.u32 %0, 1, 0, po;\n\t"
                    "}\n"
                    : "=r"(all) : "r"(got ? 1u : 0u) : "memory");
                got = all != 0;
            }
            if (!got) { ok = false; break; }
            tc_fence_after();

            const bool warp_has_rows = (q * 32 < half_h) && (warp_v0 < p.n_total);   // uniform over the warp
#pragma unroll
            for (int u = 0; u < kPairMaxChunks; ++u) {
                if (u >= n_chunks || !warp_has_rows) continue;
                const int c0 = u * kPairChunk;
                const int cols_here = min(kPairChunk, p.n_cols - c0);               // 16 or 32
                if (row0 + c0 >= p.rows) continue;                                   // the block's padding columns
                // ---- TMEM -> shared memory, transposed: tbuf[column][lane] (both halves requested before the one wait)
                {
                    uint32_t va[16], vb[16];
                    tmem_ld16(taddr + static_cast<uint32_t>(c0), va);
                    if (cols_here > 16) tmem_ld16(taddr + static_cast<uint32_t>(c0 + 16), vb);
                    tmem_wait_ld();
#pragma unroll
                    for (int t = 0; t < 16; ++t)
                        tbuf[t * kPairPitch + lane] = lane_valid ? __uint_as_float(va[t]) : -CUDART_INF_F;
                    if (cols_here > 16) {
#pragma unroll
                        for (int t = 0; t < 16; ++t)
                            tbuf[(16 + t) * kPairPitch + lane] = lane_valid ? __uint_as_float(vb[t]) : -CUDART_INF_F;
                    }
                }
                __syncwarp();
                // ---- lane L: window row row0 + c0 + L against this warp's 32 vocabulary rows.  Few warps share a
                // scheduler here, so the chains are kept short: the maximum by a tree (the right operand of every
                // merge holds the higher tokens, so strict '>' keeps the lowest token id of a tie), the sum in four
                // independent accumulators.
                const int r = row0 + c0 + lane;
                if (lane < cols_here && r < p.rows) {
                    float x[32];
                    const float4* src = reinterpret_cast<const float4*>(tbuf + lane * kPairPitch);
#pragma unroll
                    for (int t = 0; t < 8; ++t) {
                        const float4 f = src[t];
                        x[4 * t] = f.x; x[4 * t + 1] = f.y; x[4 * t + 2] = f.z; x[4 * t + 3] = f.w;
                    }
                    float tm[16];
                    int ti[16];
#pragma unroll
                    for (int t = 0; t < 16; ++t) {
                        const bool g = x[2 * t + 1] > x[2 * t];
                        tm[t] = g ? x[2 * t + 1] : x[2 * t];
                        ti[t] = g ? 2 * t + 1 : 2 * t;
                    }
#pragma unroll
                    for (int w2 = 8; w2 >= 1; w2 >>= 1) {
#pragma unroll
                        for (int t = 0; t < w2; ++t) {
                            const bool g = tm[2 * t + 1] > tm[2 * t];
                            const float m2 = g ? tm[2 * t + 1] : tm[2 * t];
                            const int i2 = g ? ti[2 * t + 1] : ti[2 * t];
                            tm[t] = m2; ti[t] = i2;
                        }
                    }
                    const float cm = tm[0];
                    const int ci = ti[0];
                    if (cm != -CUDART_INF_F) {
                        if (cm > mx[u]) {                     // strict: an earlier (lower) token keeps a tie
                            sum[u] *= exp2f((mx[u] - cm) * 1.4426950408889634f);
                            mx[u] = cm;
                            arg[u] = warp_v0 + ci;
                        }
                        const float base = mx[u] * 1.4426950408889634f;
                        float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
                        for (int t = 0; t < 32; ++t) acc[t & 3] += ex2_approx(fmaf(x[t], 1.4426950408889634f, -base));
                        sum[u] += (acc[0] + acc[1]) + (acc[2] + acc[3]);
                        const int d = tokc[u] - warp_v0;
                        if (static_cast<unsigned>(d) < 32u && warp_v0 + d < p.n_total && q * 32 + d < half_h)
                            p.tok_logit[r] = tbuf[lane * kPairPitch + d];
                    }
                }
                __syncwarp();                                  // the buffer is rewritten by the next chunk
            }
            // accumulator drained: hand it back to the MMA warp of the leader
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(as ? leader_acc_empty1 : leader_acc_empty0);
            if (!p.carry) flush_state(w.j, w.n * 2 + static_cast<int>(rank));
        }
        // carry: the tiles of a pair ascend through the vocabulary, so the strict '>' of the update kept the lowest
        // index; a pair without tiles is never launched.  (`ok` is the same in all four warps, see above.)
        if (p.carry && ok) flush_state(team, team_k * 2 + static_cast<int>(rank));
    }

    // After a time-out copies may still be heading for the shared memory of either CTA.  Their bytes are counted on
    // the leader's full barriers, so one lane of the leader's producer warp waits (bounded) for the stages it issued last
    // before it arrives at the closing cluster barrier, which in turn keeps the partner from retiring earlier.
    __syncthreads();
    if (leader && warp == 0 && lane == 0 && abort_flag[0] != 0) {
        // K block i went to slot i % stages and completes phase (i / stages) & 1 of its full barrier
        for (long long i = prod_issued > p.stages ? prod_issued - p.stages : 0; i < prod_issued; ++i)
            mbar_wait_bounded(full_bar(static_cast<int>(i % p.stages)), static_cast<uint32_t>((i / p.stages) & 1),
                              abort_flag + 1, kWaitLimitClocks);
    }
    // neither CTA may retire (or release TMEM) while its partner can still signal or read it
    tc_fence_before();
    __syncwarp();
    cluster_arrive();
    cluster_wait();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, kTmemCols);
    }
    if (threadIdx.x == 0 && abort_flag[0] != 0) atomicOr(p.err, 1);
}

}  // namespace wisv
