// LM-head GEMM + row reduction on CTA pairs (tcgen05 cta_group::2), used when the batch has more
// than one row tile.  Two CTAs of a cluster share one 256 x 256 output tile: CTA r holds rows
// r*128 .. r*128+127 of the tile in its own TMEM and loads, per K block, its own 128 activation rows
// and its half (128 rows) of the 256 weight rows - so every weight tile enters shared memory once
// per pair instead of once per CTA, which is what limits the single-CTA kernel (shared-memory fill
// and L2 -> SM traffic, and with it power).  One thread of the even CTA issues the MMAs for both.
//
// Barriers: full[s] lives in the leader and counts the bytes of both CTAs' loads; empty[s] and
// acc_full[a] exist in both CTAs and are signalled by a multicast tcgen05.commit; acc_empty[a] lives in
// the leader and is arrived on by the epilogue warps of both CTAs.  No load uses multicast.  Every
// wait is bounded; both CTAs meet at a cluster barrier before TMEM is released.
#pragma once

#include "wisv_gemm.cuh"

namespace wisv {

constexpr int kPairTileM = 256;
constexpr int kPairTileN = 256;
constexpr uint32_t kPairStageBytes = 2u * kTileM * kBlockK * 2u;   // 128 activation rows + 128 weight rows

struct PairParams {
    int32_t rows;        // valid window rows
    int32_t n_total;     // vocabulary size
    int32_t k_blocks;
    int32_t mp_tiles;    // row tiles of 256
    int32_t m_group;     // row tiles per raster group: tiles run group by group (all vocabulary tiles of a
                         // group of row tiles before the next group) so that the activation rows of a group
                         // stay resident in L2 while the weights stream past them
    int32_t n_tiles;     // vocabulary tiles of 256
    int32_t stages;
    // One row tile of 256 (carry = 1): the vocabulary is dealt out in units of 32 rows as one contiguous range per
    // pair - units_base units, one more for the first units_rem pairs - cut into tiles_per_pair tiles of tile_n or
    // tile_n - 32 rows; a pair carries its running row state across its tiles and writes one partial per (row, pair).
    // The pairs then finish together for any vocabulary size and any number of pairs.
    int32_t carry, units_base, units_rem, tiles_per_pair, tile_n;
    int32_t part_stride; // partials per row (n_tiles, or the number of pairs when carry)
    int32_t* err;
    float4* lm_part;
    const int32_t* row_tok;
    float* tok_logit;
};

__host__ __device__ inline uint32_t pair_fixed_bytes() { return 1024u + 1024u; }   // alignment slack + barriers

// CTAs from lm_ctas on (whole clusters) do not belong to a pair: they evaluate the decision head with the
// single-CTA GEMM body while the pairs stream the LM head (batches of at most 256 window rows, where the
// LM head is bound by HBM and the head would otherwise add its whole latency to the round).
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1)
lmhead_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                   const __grid_constant__ CUtensorMap tmB2, const PairParams p,
                   const __grid_constant__ CUtensorMap tmZ, const __grid_constant__ CUtensorMap tmW1,
                   const __grid_constant__ CUtensorMap tmW1_2, const GemmParams hd, const int lm_ctas,
                   const int head_ctas)
{
    if (static_cast<int>(blockIdx.x) >= lm_ctas) {
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
    const uint32_t half_bytes = kTileM * kBlockK * 2;                 // 16 KB
    const uint32_t ring_bytes = kPairStageBytes * static_cast<uint32_t>(p.stages);

    const uint32_t bar_base = smem_base + ring_bytes;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kMaxStages + s); };
    auto acc_full_bar = [&](int s) { return bar_base + 8u * (2 * kMaxStages + s); };
    auto acc_empty_bar = [&](int s) { return bar_base + 8u * (2 * kMaxStages + 2 + s); };
    const uint32_t drain_bar = bar_base + 8u * (2 * kMaxStages + 4);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + ring_bytes + 8 * (2 * kMaxStages + 5));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);   // [0] abort, [1] drain scratch

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int total_tiles = p.mp_tiles * p.n_tiles;
    // tile t -> (row tile mp, vocabulary tile n): groups of m_group row tiles, row tile fastest inside a group
    auto tile_mp_n = [&](int t, int* mp, int* n) {
        const int per_group = p.m_group * p.n_tiles;
        const int g = t / per_group;
        const int mp0 = g * p.m_group;
        const int gsize = min(p.m_group, p.mp_tiles - mp0);
        const int idx = t - g * per_group;
        *n = idx / gsize;
        *mp = mp0 + idx % gsize;
    };
    // carry: this pair's contiguous range of 32-row units and how it is cut into tiles
    const int my_units = p.units_base + (pair_id < p.units_rem ? 1 : 0);
    const int my_unit0 = pair_id * p.units_base + (pair_id < p.units_rem ? pair_id : p.units_rem);
    const int my_tiles = p.carry ? (my_units < p.tiles_per_pair ? my_units : p.tiles_per_pair) : 0;
    const int my_hq = p.carry ? my_units / p.tiles_per_pair : 0;
    const int my_hr = p.carry ? my_units % p.tiles_per_pair : 0;
    // the i-th tile of this pair: row tile mp, first vocabulary row n0, height h (a multiple of 32), tile index n
    struct PTile { int mp, n, n0, h; };
    auto tile_at = [&](int i, PTile& w) -> bool {
        if (p.carry) {
            if (i >= my_tiles) return false;
            w.mp = 0; w.n = pair_id;
            w.h = (my_hq + (i < my_hr ? 1 : 0)) * 32;
            w.n0 = (my_unit0 + i * my_hq + (i < my_hr ? i : my_hr)) * 32;
            return true;
        }
        const int t = pair_id + i * n_pairs;
        if (t >= total_tiles) return false;
        tile_mp_n(t, &w.mp, &w.n);
        w.n0 = w.n * kPairTileN; w.h = kPairTileN;
        return true;
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(acc_full_bar(s), 1); mbar_init(acc_empty_bar(s), 8); }
        mbar_init(drain_bar, 1);
        abort_flag[0] = 0;
        abort_flag[1] = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
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

    // The pack kernel wrote the bf16 rows this kernel loads: everyone waits for it here, except the producer
    // thread, which first puts one ring-full of weight tiles in flight (they depend on nothing) and waits then.
    const bool producer_thread = warp == 0 && lane == 0;
    if (!producer_thread) {
        griddep_wait();
        griddep_launch_dependents();
    }

    // producer thread only: ring position and stages issued so far (read again by the drain before the kernel ends)
    int prod_s = 0;
    uint32_t prod_ph = 0;
    long long prod_issued = 0;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (each CTA)
        if (lane == 0) {
            int& s = prod_s;
            uint32_t& ph = prod_ph;
            long long& issued = prod_issued;
            bool ok = true;
            PTile w;
            long long pre = 0;                 // stages whose weight half-tile was requested before the wait
            for (int i = 0; pre < p.stages && tile_at(i, w); ++i) {
                const int half_h = w.h >> 1;
                const int col0 = w.n0 + static_cast<int>(rank) * half_h;
                const CUtensorMap* mapB = (w.h == p.tile_n) ? &tmB : &tmB2;
                const uint32_t tx = 2u * (half_bytes + static_cast<uint32_t>(half_h) * kBlockK * 2u);
                for (int kb = 0; kb < p.k_blocks && pre < p.stages; ++kb, ++pre) {
                    const uint32_t a_dst = smem_base + kPairStageBytes * static_cast<uint32_t>(pre);
                    if (leader) mbar_expect_tx(full_bar(static_cast<int>(pre)), tx);
                    tma_load_2d_pair(a_dst + half_bytes, mapB, kb * kBlockK, col0, full_bar(static_cast<int>(pre)));
                }
            }
            griddep_wait();
            griddep_launch_dependents();
            for (int i = 0; ok && tile_at(i, w); ++i) {
                const int row0 = w.mp * kPairTileM + static_cast<int>(rank) * kTileM;
                const int half_h = w.h >> 1;                                   // weight rows this CTA loads
                const int col0 = w.n0 + static_cast<int>(rank) * half_h;
                const CUtensorMap* mapB = (w.h == p.tile_n) ? &tmB : &tmB2;
                const uint32_t tx = 2u * (half_bytes + static_cast<uint32_t>(half_h) * kBlockK * 2u);
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    const uint32_t a_dst = smem_base + kPairStageBytes * s;
                    if (issued < pre) {
                        // first pass over the ring: the stage is free, its bytes are expected and its weight
                        // half-tile is already on its way
                        tma_load_2d_pair(a_dst, &tmA, kb * kBlockK, row0, full_bar(s));
                    } else {
                        if (!mbar_wait_bounded(empty_bar(s), ph ^ 1u, abort_flag, kWaitLimitClocks)) { ok = false; break; }
                        if (leader) mbar_expect_tx(full_bar(s), tx);             // both CTAs' bytes
                        tma_load_2d_pair(a_dst, &tmA, kb * kBlockK, row0, full_bar(s));
                        tma_load_2d_pair(a_dst + half_bytes, mapB, kb * kBlockK, col0, full_bar(s));
                    }
                    ++issued;
                    if (++s == p.stages) { s = 0; ph ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader CTA only)
        if (lane == 0 && leader) {
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            PTile w;
            for (int local = 0; ok && tile_at(local, w); ++local) {
                const uint32_t idesc = idesc_bf16_f32(kPairTileM, static_cast<uint32_t>(w.h));
                const int as = local & 1;
                const uint32_t aph = (local >> 1) & 1u;
                if (!mbar_wait_bounded(acc_empty_bar(as), aph ^ 1u, abort_flag, kWaitLimitClocks)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(as * kAccCols);
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    if (!mbar_wait_bounded(full_bar(s), ph, abort_flag, kWaitLimitClocks)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = smem_base + kPairStageBytes * s;
                    const uint64_t a_desc = smem_desc_k128(a_addr);
                    const uint64_t b_desc = smem_desc_k128(a_addr + half_bytes);
#pragma unroll
                    for (int k = 0; k < kBlockK / kUmmaK; ++k)
                        umma_bf16_pair(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, (kb | k) != 0 ? 1u : 0u);
                    umma_commit_pair(empty_bar(s));          // frees the stage in both CTAs
                    if (++s == p.stages) { s = 0; ph ^= 1u; }
                }
                if (ok) umma_commit_pair(acc_full_bar(as));  // accumulator ready in both CTAs
            }
            if (!ok) {
                umma_commit_pair(drain_bar);
                mbar_wait_bounded(drain_bar, 0, abort_flag + 1, kWaitLimitClocks);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..5 of each CTA)
        const int q = warp & 3;
        bool ok = true;
        const uint32_t leader_acc_empty0 = mapa_u32(acc_empty_bar(0), 0);
        const uint32_t leader_acc_empty1 = mapa_u32(acc_empty_bar(1), 0);
        float mx = -CUDART_INF_F, sum = 0.0f;      // running row state: per tile, or per pair when carry
        int arg = 0;
        PTile w;
        int last_row = -1;
        for (int local = 0; ok && tile_at(local, w); ++local) {
            const int as = local & 1;
            const uint32_t aph = (local >> 1) & 1u;
            const int row = w.mp * kPairTileM + static_cast<int>(rank) * kTileM + q * 32 + lane;
            const bool valid = row < p.rows;
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + static_cast<uint32_t>(as * kAccCols);

            bool got = mbar_wait_bounded(acc_full_bar(as), aph, abort_flag, kWaitLimitClocks);
            got = __all_sync(0xffffffffu, got);
            if (!got) { ok = false; break; }
            tc_fence_after();

            if (!p.carry) { mx = -CUDART_INF_F; sum = 0.0f; arg = 0; }
            const int tok = valid ? p.row_tok[row] : -1;
            for (int c0 = 0; c0 < w.h; c0 += 16) {
                uint32_t v[16];
                __syncwarp();
                tmem_ld16(taddr + static_cast<uint32_t>(c0), v);
                tmem_wait_ld();
                if (!valid) continue;
                lm_update_chunk(v, w.n0 + c0, p.n_total, tok, mx, arg, sum, p.tok_logit + row);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(as ? leader_acc_empty1 : leader_acc_empty0);
            if (valid && !p.carry)
                p.lm_part[(size_t)row * p.part_stride + w.n] = make_float4(mx, __int_as_float(arg), sum, 0.0f);
            last_row = valid ? row : -1;
        }
        // carry: the tiles of a pair ascend through the vocabulary, so the strict '>' of the update kept the
        // lowest index; a pair without tiles is never launched
        if (p.carry && ok && last_row >= 0)
            p.lm_part[(size_t)last_row * p.part_stride + pair_id] = make_float4(mx, __int_as_float(arg), sum, 0.0f);
    }

    // After a time-out copies may still be heading for the shared memory of either CTA.  Their bytes are counted on
    // the leader's full barriers, so the leader's producer thread waits (bounded) for the stages it issued last
    // before it arrives at the closing cluster barrier, which in turn keeps the partner from retiring earlier.
    __syncthreads();
    if (leader && producer_thread && abort_flag[0] != 0) {
        const int inflight = prod_issued < p.stages ? static_cast<int>(prod_issued) : p.stages;
        int ws = prod_s;
        uint32_t wph = prod_ph;
        for (int i = 0; i < inflight; ++i) {
            if (--ws < 0) { ws = p.stages - 1; wph ^= 1u; }
            mbar_wait_bounded(full_bar(ws), wph, abort_flag + 1, kWaitLimitClocks);
        }
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
