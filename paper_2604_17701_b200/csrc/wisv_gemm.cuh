// Persistent, warp-specialised bf16 GEMM for sm_100a whose epilogue reduces each
// output row over the N dimension instead of storing it:
//
//   D[row, n] = sum_k A[row, k] * Bw[n, k]      A: activations (rows x K), Bw: weights (N x K)
//
// * LM-head epilogue: per (row, N-tile) the running max, its lowest column index
//   and sum exp(D - max) (the pieces of argmax / log-sum-exp), plus the one logit
//   at the row's draft token.  The logits never leave TMEM / registers.
// * Decision-head epilogue: per (row, N-tile) the partial dot product
//   sum_n w2[n] * act(D[row, n] + b1[n] + W1c[n, :] . csi[row]).
// * Raw epilogue (bring-up / tests): D written to global memory.
//
// One CTA per SM loops over (m, n) tiles.  Warp 0 streams A and Bw tiles with TMA
// into a ring of shared-memory stages, warp 1 issues tcgen05.mma (M = 128,
// N = tile_n, K = 16) into one of two TMEM accumulators, warps 2-5 drain the other
// accumulator with tcgen05.ld and run the epilogue, so the epilogue of tile i
// overlaps the main loop of tile i+1.  Every wait is bounded.
#pragma once

#include <math_constants.h>

#include "wisv_ptx.cuh"

namespace wisv {

constexpr int kTileM = 128;          // rows per tile = TMEM lanes
constexpr int kBlockK = 64;          // bf16 elements per 128-byte swizzled row
constexpr int kUmmaK = 16;
constexpr int kMaxTileN = 256;
constexpr int kAccCols = 256;        // TMEM columns per accumulator stage
constexpr int kTmemCols = 512;
constexpr int kGemmThreads = 192;
constexpr int kEpiThreads = 128;
constexpr int kMaxStages = 32;
constexpr uint64_t kWaitLimitClocks = 4000000000ull;   // SM clocks: 2 s at 2 GHz, 3.3 s at 1.2 GHz
constexpr int kMaxDc = 16;
constexpr int kMaxKSplits = 16;      // split-K work items per tile (their partial loads are issued together)

enum { EPI_LMHEAD = 0, EPI_HEAD = 1, EPI_RAW = 2 };

struct GemmParams {
    int32_t rows;        // valid rows of A
    int32_t n_total;     // rows of Bw (vocabulary size or d_J)
    int32_t k_blocks;    // ceil(K / 64)
    int32_t tile_n;      // Bw rows per tile: multiple of 16, <= 256
    int32_t m_tiles, n_tiles;
    int32_t stages;
    int32_t a_rows;      // rows of A actually loaded per tile (multiple of 8, <= 128); the MMA still spans
                         // 128 rows, the rest of its A operand is whatever follows in shared memory and only
                         // feeds accumulator rows that are never read
    int32_t mma_m;       // 128: every MMA spans 128 rows (accumulator row i in TMEM lane i).  64: a row tile with at
                         // most 64 valid rows is computed with MMAs of 64 rows (row i in lane (i / 16) * 32 + i % 16:
                         // sixteen lanes of each quadrant) - half the tensor work for that tile, which under the
                         // power cap means higher clocks
    int32_t carry;       // 1: one row tile, each CTA keeps its running row state across its tiles and
                         //    writes one partial per (row, CTA); 0: one partial per (row, N-tile)
    // carry only: the rows of Bw are dealt out in units of 16 as one contiguous range per CTA - CTA c gets
    // units_base units, one more if c < units_rem - and each CTA cuts its range into tiles_per_cta tiles
    // whose heights differ by at most one unit (tile_n is the larger height, tile_n - 16 the smaller).
    // No CTA then has more than 16 rows more than another, whatever n_total and the number of CTAs.
    int32_t units_base, units_rem, tiles_per_cta;
    int32_t part_stride; // partials per row (CTAs when carry, else n_tiles)
    int32_t k_splits;    // decision head only: the K range is cut into k_splits work items per (m, n) tile;
                         // each item stores its raw fp32 tile, the last one to finish adds them up in
                         // split order and applies the epilogue (no CTA ever waits for another)
    int32_t kb_per_split;
    float* splitk_buf;        // [items][tile_n][128] raw partial pre-activations, column-major per item
    int32_t* splitk_count;    // [m_tiles * n_tiles], zero between calls (the last item resets it)
    int32_t* err;        // device error word (bit 0: a bounded wait gave up)
    // LM-head epilogue
    float4* lm_part;          // [rows][part_stride] = {max, bits(argidx), sumexp, 0}
    const int32_t* row_tok;   // [rows] draft token of the row or -1
    float* tok_logit;         // [rows]
    // decision-head epilogue
    float* head_part;         // [rows][part_stride]
    const float* b1;          // [n_total]
    const float* w2;          // [n_total]
    const float* w1c;         // [n_total][d_c] fp32 CSI columns of W1
    const float* csi;         // [B][d_c]
    const int32_t* pos_req;   // [rows] request of each position
    int32_t d_c;
    int32_t act;              // 0 ReLU, 1 exact GELU
    // raw epilogue
    float* raw_out;           // [rows][n_total]
};

__host__ __device__ inline uint32_t gemm_stage_bytes(int tile_n, int a_rows = kTileM) {
    return static_cast<uint32_t>(a_rows * kBlockK * 2 + tile_n * kBlockK * 2);
}
// bytes the MMA may read past the last stage's A slot when fewer than 128 rows are loaded
__host__ __device__ inline uint32_t gemm_overread_bytes(int a_rows) {
    return static_cast<uint32_t>((kTileM - a_rows) * kBlockK * 2);
}
// bytes after the stage ring: barriers + tmem slot + abort flag, then epilogue constants
__host__ __device__ inline uint32_t gemm_tail_bytes(int tile_n, int d_c) {
    return 1024u + 2u * (static_cast<uint32_t>(tile_n) * static_cast<uint32_t>(2 + d_c) +
                        static_cast<uint32_t>(kEpiThreads * d_c)) * 4u;
}

__device__ __forceinline__ float act_apply(float x, int act) {
    if (act == 0) return fmaxf(x, 0.0f);
    return 0.5f * x * (1.0f + erff(x * 0.70710678118654752440f));
}

// Online update of one row's (max, lowest argidx, sum exp) with 16 consecutive logits starting at
// column col0 (columns >= n_total are padding), and capture of the logit at the row's draft token.
__device__ __forceinline__ void lm_update_chunk(const uint32_t (&v)[16], int col0, int n_total, int tok,
                                                float& mx, int& arg, float& sum, float* tok_logit_row)
{
    float f[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) f[j] = (col0 + j < n_total) ? __uint_as_float(v[j]) : -CUDART_INF_F;
    float cm = f[0];
    int ci = 0;
#pragma unroll
    for (int j = 1; j < 16; ++j) { if (f[j] > cm) { cm = f[j]; ci = j; } }
    if (cm > mx) {                           // strict: earlier (lower) index wins ties
        sum *= exp2f((mx - cm) * 1.4426950408889634f);
        mx = cm;
        arg = col0 + ci;
    }
    const float base = mx * 1.4426950408889634f;
    float acc = 0.0f;
#pragma unroll
    for (int j = 0; j < 16; ++j) acc += exp2f(fmaf(f[j], 1.4426950408889634f, -base));
    sum += acc;
    if (static_cast<unsigned>(tok - col0) < 16u) {
        float tl = 0.0f;
#pragma unroll
        for (int j = 0; j < 16; ++j) tl = (tok - col0 == j) ? f[j] : tl;
        *tok_logit_row = tl;
    }
}

// The work of CTA `cta` of `ncta` CTAs that share the tiles of one GEMM.  HEAD_WAITS_LAST selects where
// the decision-head CTAs synchronise with the preceding kernels of the stream (see below).
template <int EPI, bool HEAD_WAITS_LAST>
__device__ __forceinline__ void gemm_rowreduce_body(const CUtensorMap& tmA, const CUtensorMap& tmB,
                                                    const CUtensorMap& tmB2, const GemmParams& p,
                                                    const int cta, const int ncta)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t pad = ((raw_addr + 1023u) & ~1023u) - raw_addr;
    uint8_t* smem = smem_raw + pad;                       // 1024-byte aligned: swizzle atoms need it
    const uint32_t smem_base = raw_addr + pad;

    const uint32_t a_bytes = static_cast<uint32_t>(p.a_rows) * kBlockK * 2;
    const uint32_t b_bytes = static_cast<uint32_t>(p.tile_n) * kBlockK * 2;
    const uint32_t stage_bytes = a_bytes + b_bytes;
    const uint32_t ring_bytes = stage_bytes * static_cast<uint32_t>(p.stages);

    // barriers: full[S], empty[S], acc_full[2], acc_empty[2], drain
    const uint32_t bar_base = smem_base + ring_bytes;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kMaxStages + s); };
    auto acc_full_bar = [&](int s) { return bar_base + 8u * (2 * kMaxStages + s); };
    auto acc_empty_bar = [&](int s) { return bar_base + 8u * (2 * kMaxStages + 2 + s); };
    const uint32_t drain_bar = bar_base + 8u * (2 * kMaxStages + 4);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + ring_bytes + 8 * (2 * kMaxStages + 5));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);   // [0] abort, [1] drain scratch
    volatile int* last_flag = abort_flag + 2;                                    // split-K: this CTA finishes the tile
    float* epi_const = reinterpret_cast<float*>(smem + ring_bytes + 1024);

    const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0);   // the same in all lanes, and the compiler knows it
    const int lane = threadIdx.x & 31;
    const int total_tiles = p.m_tiles * p.n_tiles * p.k_splits;      // work items
    // item t -> row tile m (fastest), K split ks, column tile n
    auto item_m = [&](int t) { return t % p.m_tiles; };
    auto item_ks = [&](int t) { return (t / p.m_tiles) % p.k_splits; };
    auto item_n = [&](int t) { return (t / p.m_tiles) / p.k_splits; };
    auto item_kb0 = [&](int t) { return item_ks(t) * p.kb_per_split; };
    auto item_kb1 = [&](int t) { const int e = (item_ks(t) + 1) * p.kb_per_split; return e < p.k_blocks ? e : p.k_blocks; };
    // carry: this CTA's contiguous range of 16-row units and how it is cut into tiles
    const int my_units = p.units_base + (cta < p.units_rem ? 1 : 0);
    const int my_unit0 = cta * p.units_base + (cta < p.units_rem ? cta : p.units_rem);
    const int my_tiles = my_units < p.tiles_per_cta ? my_units : p.tiles_per_cta;     // tiles that are not empty
    const int my_hq = p.carry ? my_units / p.tiles_per_cta : 0;
    const int my_hr = p.carry ? my_units % p.tiles_per_cta : 0;
    // The i-th work item of this CTA: row tile m, first row n0 and height h of its block of Bw, column tile
    // index n and global item number t (both used only without carry), K blocks [kb0, kb1).
    struct Item { int t, m, n, n0, h, kb0, kb1; };
    auto item_at = [&](int i, Item& w) -> bool {
        if (p.carry) {
            if (i >= my_tiles) return false;
            w.t = i; w.m = 0; w.n = 0;
            w.h = (my_hq + (i < my_hr ? 1 : 0)) * 16;
            w.n0 = (my_unit0 + i * my_hq + (i < my_hr ? i : my_hr)) * 16;
            w.kb0 = 0; w.kb1 = p.k_blocks;
            return true;
        }
        const int t = cta + i * ncta;
        if (t >= total_tiles) return false;
        w.t = t; w.m = item_m(t); w.n = item_n(t); w.n0 = w.n * p.tile_n; w.h = p.tile_n;
        w.kb0 = item_kb0(t); w.kb1 = item_kb1(t);
        return true;
    };
    auto b_map = [&](int h) -> const CUtensorMap* { return h == p.tile_n ? &tmB : &tmB2; };
    // rows of the MMAs of row tile m (see GemmParams::mma_m)
    auto tile_mma_m = [&](int m) { return (p.mma_m == 64 && p.rows - m * kTileM <= 64) ? 64 : kTileM; };

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(acc_full_bar(s), 1); mbar_init(acc_empty_bar(s), 4); }
        mbar_init(drain_bar, 1);
        abort_flag[0] = 0;
        abort_flag[1] = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // Everything above overlaps the previous kernel in the stream.  The LM-head and raw kernels read
    // what the pack kernel wrote, so they wait for it here.  A decision-head kernel launched after the
    // LM-head kernel (HEAD_WAITS_LAST) also reads only pack output, which is complete by the time it can
    // be scheduled (the LM-head kernel releases its dependents only after its own wait); it waits at its
    // end instead, so that "head kernel complete" implies "LM-head kernel complete" for the merge/scan
    // kernel that follows.  Decision-head CTAs that share a launch with the LM head follow the pack
    // kernel directly and wait here like the others.
    // The producer warp of the early waiters waits a little later: weight tiles do not depend on the
    // pack kernel, so it first puts one ring-full of them in flight.
    // (The whole producer warp waits later, not just its issuing lane: lanes of one warp that sit in
    // griddepcontrol.wait hold back the lane that diverged from them.)
    constexpr bool kWaitLast = (EPI == EPI_HEAD) && HEAD_WAITS_LAST;
    const bool producer_warp = warp == 0;
    if (!kWaitLast && !producer_warp) griddep_wait();
    // no thread of an early waiter lets the next kernel start before it has passed its own wait
    if (kWaitLast || !producer_warp) griddep_launch_dependents();

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        // The whole warp runs the loops and one elected lane issues.  The TMA, tcgen05.mma and tcgen05.commit
        // instructions take their operands from uniform registers, which exist only for code the warp runs
        // together: the same loops written as one thread's work (`if (lane == 0)`) cost about twice the clocks
        // per stage here and 57-74 clocks per MMA in the warp below (measured), more than narrow MMAs take.
        long long pre = 0;                     // stages whose weight tile was requested before the wait
        Item w;
        if (!kWaitLast) {
            for (int i = 0; pre < p.stages && item_at(i, w); ++i) {
                const uint32_t tx = a_bytes + static_cast<uint32_t>(w.h) * kBlockK * 2;
                for (int kb = w.kb0; kb < w.kb1 && pre < p.stages; ++kb, ++pre) {
                    const uint32_t a_dst = smem_base + stage_bytes * static_cast<uint32_t>(pre);
                    if (elect_one()) {
                        mbar_expect_tx(full_bar(static_cast<int>(pre)), tx);
                        tma_load_2d(a_dst + a_bytes, b_map(w.h), kb * kBlockK, w.n0, full_bar(static_cast<int>(pre)));
                    }
                    __syncwarp();
                }
            }
            griddep_wait();                    // from here on the activation rows may be read
            griddep_launch_dependents();
        }
        int s = 0;
        uint32_t ph = 0;
        long long issued = 0;
        bool ok = true;
        for (int i = 0; ok && item_at(i, w); ++i) {
            const uint32_t tx = a_bytes + static_cast<uint32_t>(w.h) * kBlockK * 2;
            const CUtensorMap* mapB = b_map(w.h);
            for (int kb = w.kb0; kb < w.kb1; ++kb) {
                const uint32_t a_dst = smem_base + stage_bytes * s;
                // not fresh: first pass over the ring, the stage is free and its weight tile is already on its way
                const bool fresh = issued >= pre;
                if (fresh) {
                    ok = __all_sync(0xffffffffu, mbar_wait_bounded(empty_bar(s), ph ^ 1u, abort_flag, kWaitLimitClocks));
                    if (!ok) break;
                }
                if (elect_one()) {
                    if (fresh) mbar_expect_tx(full_bar(s), tx);
                    tma_load_2d(a_dst, &tmA, kb * kBlockK, w.m * kTileM, full_bar(s));
                    if (fresh) tma_load_2d(a_dst + a_bytes, mapB, kb * kBlockK, w.n0, full_bar(s));
                }
                __syncwarp();
                ++issued;
                if (++s == p.stages) { s = 0; ph ^= 1u; }
            }
        }
        if (!ok) {
            // let copies already in flight land before the CTA retires
            const int inflight = issued < p.stages ? static_cast<int>(issued) : p.stages;
            int ws = s;
            uint32_t wph = ph;
            for (int i = 0; i < inflight; ++i) {
                if (--ws < 0) { ws = p.stages - 1; wph ^= 1u; }
                mbar_wait_bounded(full_bar(ws), wph, abort_flag + 1, kWaitLimitClocks);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (whole warp, one elected lane: see
        // the producer)
        int s = 0;
        uint32_t ph = 0;
        bool ok = true;
        Item w;
        for (int local = 0; ok && item_at(local, w); ++local) {
            const uint32_t idesc = idesc_bf16_f32(static_cast<uint32_t>(tile_mma_m(w.m)), static_cast<uint32_t>(w.h));
            const int as = local & 1;
            const uint32_t aph = (local >> 1) & 1u;
            ok = __all_sync(0xffffffffu, mbar_wait_bounded(acc_empty_bar(as), aph ^ 1u, abort_flag, kWaitLimitClocks));
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(as * kAccCols);
            const int kb0 = w.kb0, kb1 = w.kb1;
            for (int kb = kb0; kb < kb1; ++kb) {
                ok = __all_sync(0xffffffffu, mbar_wait_bounded(full_bar(s), ph, abort_flag, kWaitLimitClocks));
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_addr = smem_base + stage_bytes * s;
                const uint64_t a_desc = smem_desc_k128(a_addr);
                const uint64_t b_desc = smem_desc_k128(a_addr + a_bytes);
                if (elect_one()) {
#pragma unroll
                    for (int k = 0; k < kBlockK / kUmmaK; ++k) {
                        // advancing K by 16 bf16 = 32 bytes = 2 descriptor units inside the swizzle atom
                        umma_bf16(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, ((kb - kb0) | k) != 0 ? 1u : 0u);
                    }
                    umma_commit(empty_bar(s));       // stage is free once these MMAs have read it
                    if (kb + 1 == kb1) umma_commit(acc_full_bar(as));
                }
                __syncwarp();
                if (++s == p.stages) { s = 0; ph ^= 1u; }
            }
        }
        if (!ok) {
            // drain whatever was issued before TMEM is released
            if (elect_one()) umma_commit(drain_bar);
            __syncwarp();
            mbar_wait_bounded(drain_bar, 0, abort_flag + 1, kWaitLimitClocks);
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..5)
        const int q = warp & 3;                            // TMEM lane quadrant this warp may read
        const int et = threadIdx.x - 64;                   // 0..127 among epilogue threads
        bool ok = true;
        float mx = -CUDART_INF_F, sum = 0.0f, hs = 0.0f;   // running row state (per tile, or per CTA when carry)
        int arg = 0;
        Item w;
        for (int local = 0; ok && item_at(local, w); ++local) {
            const int t = w.t, m = w.m, n = w.n;
            const int as = local & 1;
            const uint32_t aph = (local >> 1) & 1u;
            // row of the tile held by this thread's TMEM lane
            const bool m64 = tile_mma_m(m) == 64;
            const int rit = m64 ? q * 16 + (lane & 15) : q * 32 + lane;
            const bool lane_used = m64 ? lane < 16 : true;
            const int row = m * kTileM + rit;
            const bool valid = lane_used && row < p.rows;
            const int n0 = w.n0;
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + static_cast<uint32_t>(as * kAccCols);

            const float* cb1 = nullptr; const float* cw2 = nullptr; const float* cwc = nullptr; const float* ccs = nullptr;
            if (EPI == EPI_HEAD) {
                // stage this tile's b1 / w2 / CSI weights and each row's CSI vector
                // (double-buffered by accumulator stage, so one barrier per tile suffices)
                float* buf = epi_const + as * (p.tile_n * (2 + p.d_c) + kEpiThreads * p.d_c);
                float* wb1 = buf; float* ww2 = buf + p.tile_n; float* wwc = buf + 2 * p.tile_n;
                float* wcs = buf + (2 + p.d_c) * p.tile_n;
                for (int j = et; j < p.tile_n; j += kEpiThreads) {
                    const bool in = (n0 + j) < p.n_total;
                    wb1[j] = in ? p.b1[n0 + j] : 0.0f;
                    ww2[j] = in ? p.w2[n0 + j] : 0.0f;
                    for (int c = 0; c < p.d_c; ++c)
                        wwc[c * p.tile_n + j] = in ? p.w1c[(size_t)(n0 + j) * p.d_c + c] : 0.0f;
                }
                // (read through L2: a late-waiting head kernel may share an SM, and its L1, with earlier rounds)
                const int rq = valid ? __ldcg(p.pos_req + row) : 0;
                // indexed by row within the tile (this thread's TMEM lane), not by thread number
                if (lane_used)
                    for (int c = 0; c < p.d_c; ++c)
                        wcs[c * kEpiThreads + rit] = valid ? __ldcg(p.csi + (size_t)rq * p.d_c + c) : 0.0f;
                cb1 = wb1; cw2 = ww2; cwc = wwc; ccs = wcs;
            }

            bool got = mbar_wait_bounded(acc_full_bar(as), aph, abort_flag, kWaitLimitClocks);
            if (EPI == EPI_HEAD) {
                // barrier over the 128 epilogue threads that also agrees on `got`
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
            } else {
                got = __all_sync(0xffffffffu, got);
            }
            if (!got) { ok = false; break; }
            tc_fence_after();

            if (!p.carry) { mx = -CUDART_INF_F; sum = 0.0f; hs = 0.0f; arg = 0; }
            const int tok = (EPI == EPI_LMHEAD && valid) ? p.row_tok[row] : -1;

            for (int c0 = 0; c0 < w.h; c0 += 16) {
                uint32_t v[16];
                __syncwarp();                                // tcgen05.ld is warp-collective
                tmem_ld16(taddr + static_cast<uint32_t>(c0), v);
                tmem_wait_ld();
                if (!valid) continue;
                const int col0 = n0 + c0;
                if (EPI == EPI_LMHEAD) {
                    lm_update_chunk(v, col0, p.n_total, tok, mx, arg, sum, p.tok_logit + row);
                } else if (EPI == EPI_HEAD && p.k_splits > 1) {
                    // split K: park the raw partial tile, column-major ([tile_n][128]: consecutive lanes hold
                    // consecutive rows, so these stores and the finisher's loads are coalesced); the last item of
                    // this (m, n) tile finishes it
                    float* dst = p.splitk_buf + ((size_t)t * p.tile_n + c0) * kTileM + rit;
#pragma unroll
                    for (int j = 0; j < 16; ++j) dst[(size_t)j * kTileM] = __uint_as_float(v[j]);
                } else if (EPI == EPI_HEAD) {
                    float pre[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) pre[j] = __uint_as_float(v[j]) + cb1[c0 + j];
                    for (int c = 0; c < p.d_c; ++c) {
                        const float x = ccs[c * kEpiThreads + rit];
#pragma unroll
                        for (int j = 0; j < 16; ++j) pre[j] = fmaf(x, cwc[c * p.tile_n + c0 + j], pre[j]);
                    }
#pragma unroll
                    for (int j = 0; j < 16; ++j) hs = fmaf(cw2[c0 + j], act_apply(pre[j], p.act), hs);
                } else {
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (col0 + j < p.n_total) p.raw_out[(size_t)row * p.n_total + col0 + j] = __uint_as_float(v[j]);
                }
            }
            // accumulator drained: hand it back to the MMA warp
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty_bar(as));

            if (EPI == EPI_HEAD && p.k_splits > 1) {
                // publish this item's partial tile, then find out whether it was the last of its tile
                __threadfence();
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (et == 0) {
                    const int old = atomicAdd(p.splitk_count + (m * p.n_tiles + n), 1);
                    const int last = old == p.k_splits - 1;
                    if (last) atomicExch(p.splitk_count + (m * p.n_tiles + n), 0);   // ready for the next call
                    *last_flag = last;
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
                const bool finisher = *last_flag != 0;
                if (finisher) {
                    // Every epilogue thread finishes one row of the tile: per 16 columns it fetches the partial
                    // sums of all splits (all loads in flight together), adds them in split order and then runs
                    // the same 16-wide epilogue as the unsplit path, so the long dependent chain of the exact
                    // GELU is overlapped sixteen-fold.  (A first version gave a warp 32 columns of one row at a
                    // time and reduced with shuffles: one GELU chain per lane at a time, 60 us for a full tile.)
                    __threadfence();
                    const int rows_here = min(kTileM, p.rows - m * kTileM);
                    const int r = et;
                    if (r < rows_here) {
                        float tot = 0.0f;
                        for (int c0 = 0; c0 < p.tile_n; c0 += 16) {
                            float pre[16];
#pragma unroll
                            for (int jj = 0; jj < 16; ++jj) pre[jj] = 0.0f;
                            for (int ks0 = 0; ks0 < p.k_splits; ks0 += 4) {             // four splits' loads at a time
                                float x[4][16];
#pragma unroll
                                for (int u = 0; u < 4; ++u) {
                                    const int ks = ks0 + u;
                                    const int it = (n * p.k_splits + ks) * p.m_tiles + m;
                                    const float* src = p.splitk_buf + ((size_t)it * p.tile_n + c0) * kTileM + r;
#pragma unroll
                                    for (int jj = 0; jj < 16; ++jj)
                                        x[u][jj] = ks < p.k_splits ? __ldcg(src + (size_t)jj * kTileM) : 0.0f;
                                }
#pragma unroll
                                for (int u = 0; u < 4; ++u)                              // split order
#pragma unroll
                                    for (int jj = 0; jj < 16; ++jj) pre[jj] += x[u][jj];
                            }
#pragma unroll
                            for (int jj = 0; jj < 16; ++jj) pre[jj] += cb1[c0 + jj];
                            for (int c = 0; c < p.d_c; ++c) {
                                const float xc = ccs[c * kEpiThreads + r];
#pragma unroll
                                for (int jj = 0; jj < 16; ++jj) pre[jj] = fmaf(xc, cwc[c * p.tile_n + c0 + jj], pre[jj]);
                            }
#pragma unroll
                            for (int jj = 0; jj < 16; ++jj) tot = fmaf(cw2[c0 + jj], act_apply(pre[jj], p.act), tot);
                        }
                        p.head_part[(size_t)(m * kTileM + r) * p.part_stride + n] = tot;
                    }
                }
            } else if (valid && !p.carry) {
                if (EPI == EPI_LMHEAD)
                    p.lm_part[(size_t)row * p.part_stride + n] = make_float4(mx, __int_as_float(arg), sum, 0.0f);
                else if (EPI == EPI_HEAD)
                    p.head_part[(size_t)row * p.part_stride + n] = hs;
            }
        }
        if (p.carry && ok) {
            // one row tile: tiles of this CTA ascend through the vocabulary, so the strict '>' above
            // already kept the lowest index; a CTA without tiles is never launched
            const bool m64 = tile_mma_m(0) == 64;
            const int row = m64 ? q * 16 + (lane & 15) : q * 32 + lane;
            if ((m64 ? lane < 16 : true) && row < p.rows) {
                if (EPI == EPI_LMHEAD)
                    p.lm_part[(size_t)row * p.part_stride + cta] = make_float4(mx, __int_as_float(arg), sum, 0.0f);
                else if (EPI == EPI_HEAD)
                    p.head_part[(size_t)row * p.part_stride + cta] = hs;
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
    if (kWaitLast) griddep_wait();
    if (threadIdx.x == 0 && (abort_flag[0] != 0)) atomicOr(p.err, 1);
}

// HEAD_WAITS_LAST (decision-head epilogue only): true when an LM-head launch that waited for the pack kernel sits
// between the pack kernel and this launch in the stream; false when this launch follows the pack kernel directly
// (the decide and gathered phases), where the head must wait before its first read like every other consumer.
template <int EPI, bool HEAD_WAITS_LAST = true>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_rowreduce_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                      const __grid_constant__ CUtensorMap tmB2, const GemmParams p)
{
    gemm_rowreduce_body<EPI, HEAD_WAITS_LAST>(tmA, tmB, tmB2, p, static_cast<int>(blockIdx.x),
                                              static_cast<int>(gridDim.x));
}

// One row tile of window rows and one of head positions (small batches, where the LM head streams the
// weights at HBM speed and the decision head is a latency-bound 12 MB side stream): both GEMMs in one
// launch.  The first lm_ctas CTAs reduce the LM head, the others evaluate the decision head at the
// same time, so the round no longer pays for the head after the LM head has finished.
static __global__ void __launch_bounds__(kGemmThreads, 1)
round_small_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW,
                   const __grid_constant__ CUtensorMap tmW_2, const __grid_constant__ CUtensorMap tmZ,
                   const __grid_constant__ CUtensorMap tmW1, const __grid_constant__ CUtensorMap tmW1_2,
                   const GemmParams lm, const GemmParams hd, const int lm_ctas)
{
    const int cta = static_cast<int>(blockIdx.x);
    if (cta < lm_ctas)
        gemm_rowreduce_body<EPI_LMHEAD, false>(tmX, tmW, tmW_2, lm, cta, lm_ctas);
    else
        gemm_rowreduce_body<EPI_HEAD, false>(tmZ, tmW1, tmW1_2, hd, cta - lm_ctas,
                                             static_cast<int>(gridDim.x) - lm_ctas);
}

}  // namespace wisv
