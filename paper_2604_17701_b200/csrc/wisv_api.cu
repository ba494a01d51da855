// Host side of the WISV verifier library: context, argument validation, launch
// plan and the C ABI declared in include/wisv.h.  One verification round is three
// or four stream-ordered launches: pack -> LM-head GEMM+reduce (with the decision
// head on CTAs of the same launch where the plan allows, else -> decision-head
// GEMM+reduce) -> merge/localize/scan, chained by programmatic dependent launch.
// Control never returns to the host between them and nothing is synchronised.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <utility>

#include "../../include/wisv.h"
#include "wisv_aux.cuh"
#include "wisv_gemm.cuh"
#include "wisv_gemm2.cuh"

using namespace wisv;

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr int kNumTileVariants = kMaxTileN / 16;   // tile_n = 16, 32, ..., 256
constexpr int kNumRowVariants = kTileM / 8;        // a_rows = 8, 16, ..., 128
constexpr int kStages = 4;                         // profiled stages per call
constexpr int kSplitTileN = 64;                    // head tile height when K is split over CTAs
constexpr int kSplitMaxRowTiles = 4;               // K is split for decision heads of up to this many row tiles
constexpr long long kTeamRowBytes = 32ll << 20;    // CTA-pair LM head: teams only while all bf16 window rows fit in this
constexpr int kPairKbPerStage = 2;                 // CTA-pair LM head: K blocks per shared-memory stage

struct Plan {
    int tile_n, m_tiles, n_tiles, ctas, stages;
    int a_rows;      // activation rows loaded per tile (8..128)
    int carry;       // one partial per (row, CTA) instead of per (row, N-tile)
    int parts;       // partials per row
    int pair;        // LM head on CTA pairs (vocabulary on the M side, window rows on the N side): m_tiles = row blocks
    int n_cols;      // pairs: N of the MMA = width of a row block (a multiple of 16)
    int n_blocks;    // pairs: row blocks of n_cols rows
    int kbs;         // pairs: K blocks per shared-memory stage
    int team_pairs;  // pairs with carried ranges: pairs per team (one team per row block)
    int box3d;       // pairs: one TMA box per operand and stage (3-D tensor maps)
    int k_splits;    // work items per (m, n) tile along K (decision head with one row tile)
    int kb_per_split;
    int units_base, units_rem, tiles_per_cta;   // carry: contiguous ranges of 16-row units per CTA
    size_t smem;
};

// Device and pinned-host staging of the host-buffer entry point. The two hidden-state arrays are copied straight from
// the caller's memory; every small input travels in one packed block (one copy), and every output plus the device
// error word comes back in one packed block (one copy), because at small batches a round is a few hundred
// microseconds and each separate copy costs several of them in submission and DMA latency.
struct HostStaging {
    float* target_hidden = nullptr; float* draft_hidden = nullptr;   // sized for fp32 rows; 16-bit rows use half of it
    cudaStream_t copy_stream = nullptr;            // large batches: hidden states travel group by group on this stream
    cudaEvent_t copy_ev[8] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
    uint8_t* dev_in = nullptr;        // packed small inputs, layout chosen per call
    uint8_t* pin = nullptr;           // pinned, device-mapped host: [in_cap | out_cap]
    uint8_t* pin_dev = nullptr;       // the same block as the device sees it
    size_t in_cap = 0, out_cap = 0;
    bool ready = false;
};

}  // namespace

struct wisv_ctx {
    wisv_config cfg;
    wisv_weights w;
    int device = 0;
    int sm_count = 0;
    int max_smem = 0;
    int max_pos = 0;          // capacity of evaluated head positions
    int rows_alloc = 0;       // max_rows rounded up to the tile height
    int pos_alloc = 0;
    // workspace
    __nv_bfloat16* X = nullptr;       // [rows_alloc, H]
    __nv_bfloat16* Z = nullptr;       // [pos_alloc, H_d + H]
    __nv_bfloat16* W1p = nullptr;     // [d_J, H_d + H]
    float* W1c = nullptr;             // [d_J, d_c]
    float4* lm_part = nullptr;
    size_t lm_part_elems = 0;
    float* head_part = nullptr;
    size_t head_part_elems = 0;
    float* splitk_buf = nullptr;      // [sm_count][128][kSplitTileN] raw partial head tiles
    int32_t* splitk_count = nullptr;  // per (m, n) tile arrival counters, zero between calls
    int splitk_tiles = 0;
    int max_pairs = 0;                // CTA pairs that can be resident at once
    int32_t* row_tok = nullptr; int32_t* row_flag = nullptr; float* tok_logit = nullptr;
    int32_t* pos_req = nullptr; int32_t* pos_i = nullptr;
    int32_t* err = nullptr;
    int32_t* err_copy_next = nullptr;           // where the next round's tail kernel mirrors the error word
    volatile int32_t* done_flag_next = nullptr; // where it announces that the results are written (host-buffer calls)
    int32_t done_seq = 0;                       // value it announces with
    int32_t* done_count = nullptr;              // blocks of that kernel that have finished
    int32_t* saved_arg = nullptr;               // [rows_alloc] argmax per row, localize -> decide
    unsigned long long* saved_mask = nullptr;   // [max_requests] candidate sets, localize -> decide
    bool loc_valid = false;                     // a localize call is waiting for its decide
    int loc_B = 0, loc_T = 0, loc_K = 0;
    const int32_t* loc_k_off = nullptr;
    // TMA descriptors
    CUtensorMap tmX[kNumRowVariants], tmZ[kNumRowVariants];   // box heights 8, 16, ..., 128 rows
    CUtensorMap tmW[kNumTileVariants];
    CUtensorMap tmW1[kNumTileVariants];
    // CTA-pair LM head, boxes of 2 ([0]) or 4 ([1]) K blocks: window rows (8..128 per box) and weight rows (16..128)
    CUtensorMap tmX3[2][kNumRowVariants];
    CUtensorMap tmW3[2][kNumTileVariants / 2];
    bool have_box3d = false;
    // profiling
    int prof_n = 0;
    long long prof_calls = 0;
    cudaEvent_t* prof_ev = nullptr;   // [prof_n][kStages + 1]
    long long launches = 0;
    wisv_tuning tune = {0, 0, 0, 0, 0, 0, 0, 0, 0};
    HostStaging hs;
};

namespace {

#define WISV_CUDA(call)                                   \
    do {                                                  \
        cudaError_t e_ = (call);                          \
        if (e_ != cudaSuccess) { (void)cudaGetLastError(); return WISV_ECUDA; } \
    } while (0)

int encode_2d(EncodeTiledFn fn, CUtensorMap* out, const void* base, uint64_t inner, uint64_t outer,
              uint32_t box_inner, uint32_t box_outer)
{
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {inner * 2};            // bytes between rows (bf16)
    cuuint32_t box[2] = {box_inner, box_outer};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? WISV_OK : WISV_ECUDA;
}

// The same matrix seen as (column inside a K block of 64, row, K block): a box of `box_kb` K blocks of `box_rows` rows
// lands in shared memory block after block, each block in the layout the 2-D box gives.  Only for inner % 64 == 0.
int encode_3d(EncodeTiledFn fn, CUtensorMap* out, const void* base, uint64_t inner, uint64_t outer, uint32_t box_rows,
              uint32_t box_kb)
{
    cuuint64_t dims[3] = {(cuuint64_t)kBlockK, outer, inner / kBlockK};
    cuuint64_t strides[2] = {inner * 2, (cuuint64_t)kBlockK * 2};
    cuuint32_t box[3] = {(cuuint32_t)kBlockK, box_rows, box_kb};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? WISV_OK : WISV_ECUDA;
}

int round_up(int x, int m) { return (x + m - 1) / m * m; }

size_t gemm_fixed_bytes(int tile_n, int a_rows, int d_c)
{
    return 1024 + gemm_tail_bytes(tile_n, d_c) + gemm_overread_bytes(a_rows);
}

// stage count, tile geometry -> shared memory; fills stages / smem of the plan
// On entry tile_n is the largest tile height allowed; n_total = rows of the weight matrix.
void finish_plan(const wisv_ctx* c, Plan* p, int d_c, int k_blocks, int forced_stages, int sms, int n_total)
{
    if (p->k_splits < 1) { p->k_splits = 1; p->kb_per_split = k_blocks; }
    p->carry = (p->m_tiles == 1 && p->k_splits == 1) ? 1 : 0;
    if (p->carry) {
        // One row tile and no split of K: every CTA gets one contiguous range of the weight rows, in units
        // of 16 rows, base or base + 1 units each, and cuts it into tiles of (nearly) equal height.  The CTAs
        // then finish together whatever the number of rows and CTAs - there is no last, partly filled wave.
        const int units = (n_total + 15) / 16;
        const int ctas = units < sms ? units : sms;
        p->units_base = units / ctas;
        p->units_rem = units % ctas;
        const int umax = p->units_base + (p->units_rem ? 1 : 0);
        const int cap = p->tile_n / 16 > 0 ? p->tile_n / 16 : 1;
        p->tiles_per_cta = (umax + cap - 1) / cap;
        p->tile_n = (umax + p->tiles_per_cta - 1) / p->tiles_per_cta * 16;
        p->ctas = ctas;
        p->n_tiles = ctas * p->tiles_per_cta;
        p->parts = ctas;
    } else {
        const long long items = (long long)p->m_tiles * p->n_tiles * p->k_splits;
        p->ctas = (int)(items < sms ? items : sms);
        p->parts = p->n_tiles;
    }
    const size_t fixed = gemm_fixed_bytes(p->tile_n, p->a_rows, d_c);
    const size_t stage = gemm_stage_bytes(p->tile_n, p->a_rows);
    int s = (int)(((size_t)c->max_smem - fixed) / stage);
    if (s > kMaxStages) s = kMaxStages;
    if (s > k_blocks * 4 && k_blocks > 0) s = k_blocks * 4 > 2 ? k_blocks * 4 : 2;
    if (forced_stages >= 2 && forced_stages < s) s = forced_stages;
    p->stages = s;
    p->smem = fixed + (size_t)s * stage;
}

// CTA-pair LM head: K blocks per stage and ring depth for row blocks of n_cols rows.
void pair_ring(const wisv_ctx* c, Plan* p)
{
    int kbs = c->tune.lm_kb_per_stage > 0 ? c->tune.lm_kb_per_stage : kPairKbPerStage;
    const int k_blocks = (c->cfg.H + kBlockK - 1) / kBlockK;
    while (kbs > 1 && (kbs > k_blocks || ((size_t)c->max_smem - pair_fixed_bytes()) / pair_stage_bytes(p->n_cols, kbs) < 2)) kbs /= 2;
    const size_t stage = pair_stage_bytes(p->n_cols, kbs);
    int ss = (int)(((size_t)c->max_smem - pair_fixed_bytes()) / stage);
    if (ss > kMaxStages) ss = kMaxStages;
    if (c->tune.lm_stages >= 2 && c->tune.lm_stages < ss) ss = c->tune.lm_stages;
    p->kbs = kbs;
    p->box3d = (c->have_box3d && (kbs == 2 || kbs == 4)) ? 1 : 0;
    p->stages = ss;
    p->smem = pair_fixed_bytes() + (size_t)ss * stage;
}

// LM head.  Up to 128 window rows: single CTAs with the rows on the M side, each with one contiguous range of the
// vocabulary (HBM-bound).  More rows: CTA pairs with the vocabulary on the M side and the rows on the N side
// (wisv_gemm2.cuh) - one row block with carried vocabulary ranges up to 256 rows, one team of pairs per row block
// with carried ranges while that costs no extra tile (2-4 blocks), (vocabulary tile, row block) items dealt out
// round-robin above.  The tuning switches lm_single_cta / lm_tile_n keep every size on the single-CTA kernel.
Plan plan_lm(const wisv_ctx* c, int R, bool single_only = false, int sms = 0, int reserved_pairs = 0)
{
    Plan p{};
    if (sms <= 0) sms = c->sm_count;
    const int V = c->cfg.V;
    p.m_tiles = (R + kTileM - 1) / kTileM;
    if (p.m_tiles >= 2 && c->max_pairs > 0 && !single_only && !c->tune.lm_single_cta && !c->tune.lm_tile_n) {
        p.pair = 1;
        p.a_rows = kTileM;
        p.k_splits = 1;
        p.kb_per_split = (c->cfg.H + kBlockK - 1) / kBlockK;
        int pairs_free = c->max_pairs - reserved_pairs;
        if (pairs_free < 1) pairs_free = 1;
        // the rows are cut into ceil(R / 256) blocks of equal width (a multiple of 16): no block is padded by more
        // than 15 rows, and an MMA of N columns costs N / 2 clocks
        p.n_blocks = (R + kPairMaxCols - 1) / kPairMaxCols;
        p.n_cols = round_up((R + p.n_blocks - 1) / p.n_blocks, 16);
        p.m_tiles = p.n_blocks;
        pair_ring(c, &p);
        const int units = (V + 31) / 32;
        const int n_tiles_256 = (V + kPairTileN - 1) / kPairTileN;
        // teams (one per row block, each dealing out the whole vocabulary): when they need no more tiles per pair than
        // round-robin items need rounds, and all window rows (every team reads its own) stay in L2
        int team_pairs = pairs_free / p.n_blocks;
        if (team_pairs > units) team_pairs = units;
        bool teams = false;
        if (p.n_blocks > 1 && team_pairs >= 1 && c->tune.lm_teams >= 0) {
            const int umax = (units + team_pairs - 1) / team_pairs;
            const long long team_tiles = (umax + kPairTileN / 32 - 1) / (kPairTileN / 32);
            const long long item_rounds = ((long long)p.n_blocks * n_tiles_256 + pairs_free - 1) / pairs_free;
            const bool fits = (long long)p.n_blocks * p.n_cols * c->cfg.H * 2 <= kTeamRowBytes;
            teams = fits && (team_tiles <= item_rounds || c->tune.lm_teams > 0);
        }
        if (p.n_blocks == 1 || teams) {
            // One row block (HBM-bound): like the single-CTA kernel with one row tile, every pair gets one contiguous
            // range of the vocabulary, here in units of 32 rows (each CTA of a pair loads half a tile, a multiple of
            // 16 rows), cut into tiles of nearly equal height; one partial per (row, CTA).  Teams: the same inside
            // each team.
            const int pairs = p.n_blocks == 1 ? (units < pairs_free ? units : pairs_free) : team_pairs;
            p.team_pairs = pairs;
            p.units_base = units / pairs;
            p.units_rem = units % pairs;
            const int umax = p.units_base + (p.units_rem ? 1 : 0);
            const int cap = kPairTileN / 32;
            p.tiles_per_cta = (umax + cap - 1) / cap;
            p.tile_n = (umax + p.tiles_per_cta - 1) / p.tiles_per_cta * 32;
            p.n_tiles = pairs * p.tiles_per_cta;
            p.ctas = 2 * pairs * p.n_blocks;
            p.carry = 1;
            p.parts = 2 * pairs;
            return p;
        }
        // Several row blocks (tensor-bound): work items (vocabulary tile of 256, row block) dealt out round-robin; one
        // partial per (row, vocabulary tile, CTA).
        p.carry = 0;
        p.tile_n = kPairTileN;
        p.n_tiles = n_tiles_256;
        const long long items = (long long)p.n_blocks * p.n_tiles;
        p.ctas = 2 * (int)(items < pairs_free ? items : pairs_free);
        p.parts = 2 * p.n_tiles;
        return p;
    }
    int best = 0;
    if (c->tune.lm_tile_n >= 16 && c->tune.lm_tile_n <= kMaxTileN && c->tune.lm_tile_n % 16 == 0) {
        best = c->tune.lm_tile_n;
    } else {
        // one row tile (HBM-bound): finish_plan balances the vocabulary over the CTAs, tiles as high as allowed
        // (fewest MMA instructions per byte streamed); several row tiles (tensor-bound): the largest tile
        best = kMaxTileN;
    }
    if (best > round_up(V, 16)) best = round_up(V, 16);
    p.tile_n = best;
    p.n_tiles = (V + best - 1) / best;
    p.a_rows = p.m_tiles == 1 ? round_up(R, 8) : kTileM;
    finish_plan(c, &p, 0, (c->cfg.H + kBlockK - 1) / kBlockK, c->tune.lm_stages, sms, V);
    return p;
}

Plan plan_head(const wisv_ctx* c, int P)
{
    Plan p{};
    const int N = c->cfg.d_J;
    p.m_tiles = (P + kTileM - 1) / kTileM;
    int best = 16;
    const int k_blocks = (c->cfg.H_d + c->cfg.H + kBlockK - 1) / kBlockK;
    if (c->tune.head_tile_n >= 16 && c->tune.head_tile_n <= kMaxTileN && c->tune.head_tile_n % 16 == 0) {
        best = c->tune.head_tile_n;
    } else if (p.m_tiles == 1) {
        // one row tile: too few column tiles to fill the GPU and every CTA would walk all of K, so K is
        // split as well: about one work item per SM, partial tiles combined by the last item to finish
        best = kSplitTileN;
        const int nt = (N + best - 1) / best;
        int splits = c->sm_count / nt;
        if (splits > k_blocks) splits = k_blocks;
        if (splits > kMaxKSplits) splits = kMaxKSplits;
        if (splits > 1) {
            p.kb_per_split = (k_blocks + splits - 1) / splits;
            p.k_splits = (k_blocks + p.kb_per_split - 1) / p.kb_per_split;     // no empty split
        }
    } else if (p.m_tiles <= kSplitMaxRowTiles &&
               c->sm_count / (p.m_tiles * ((N + kSplitTileN - 1) / kSplitTileN)) >= 2) {
        // a few row tiles (B=64, K=8: four): still far fewer column tiles than SMs, and every CTA would walk all of
        // K at the pace of narrow tiles (set by barrier round trips, not by the MMAs), so K is split here too while the work items fit the GPU once
        best = kSplitTileN;
        const int nt = (N + best - 1) / best;
        int splits = c->sm_count / (p.m_tiles * nt);
        if (splits > k_blocks) splits = k_blocks;
        if (splits > kMaxKSplits) splits = kMaxKSplits;
        p.kb_per_split = (k_blocks + splits - 1) / splits;
        p.k_splits = (k_blocks + p.kb_per_split - 1) / p.kb_per_split;
    } else {
        // Every work item walks all of K.  Measured with 5 to 64 row tiles of positions (d_J = 1024, 96 K blocks): the
        // kernel takes about 20 us plus, per round of items, 38 / 45 / 63 us with tiles 64 / 128 / 256 columns wide
        // (narrow tiles need more bytes per flop, so their rounds are not shorter in proportion).  So: the width whose
        // rounds cost least, at equal cost the wider tile - 64 columns while that is one round (up to 9 row tiles on
        // 148 SMs), 128 up to 18 row tiles, 256 beyond.
        static const int widths[3] = {64, 128, 256};
        static const double per_round[3] = {38.0, 45.0, 63.0};
        double best_cost = 1e30;
        for (int k = 0; k < 3; ++k) {
            const int tn = widths[k];
            const long long tiles = (long long)p.m_tiles * ((N + tn - 1) / tn);
            const long long rounds = (tiles + c->sm_count - 1) / c->sm_count;
            const double cost = (double)rounds * per_round[k];
            if (cost <= best_cost + 1e-9) { best_cost = cost; best = tn; }
        }
    }
    if (best > round_up(N, 16)) best = round_up(N, 16);
    p.tile_n = best;
    p.n_tiles = (N + best - 1) / best;
    p.a_rows = p.m_tiles == 1 ? round_up(P, 8) : kTileM;
    finish_plan(c, &p, c->cfg.d_c, k_blocks, c->tune.head_stages, c->sm_count, N);
    return p;
}

// Small batches (one row tile of window rows, one of head positions): the two GEMMs share one launch.
// The decision head gets a few CTAs of its own - enough to finish well inside the time the LM head needs
// to stream its weights - and the LM head is planned for the SMs that remain.
constexpr int kFusedHeadCtas = 6;
constexpr int kFusedHeadCtasTwoTiles = 8;     // head positions in two row tiles (129..255)

// decision-head plan for `want` CTAs that share a launch with the LM head (K never split)
Plan plan_head_beside(const wisv_ctx* c, int P, int want)
{
    Plan h{};
    const int N = c->cfg.d_J;
    const int head_m_tiles = (P + kTileM - 1) / kTileM;
    int tn = head_m_tiles > 1 ? 128 : kSplitTileN;
    if (c->tune.head_tile_n >= 16 && c->tune.head_tile_n <= kMaxTileN && c->tune.head_tile_n % 16 == 0) tn = c->tune.head_tile_n;
    if (tn > round_up(N, 16)) tn = round_up(N, 16);
    h.m_tiles = head_m_tiles; h.tile_n = tn; h.n_tiles = (N + tn - 1) / tn;
    h.a_rows = head_m_tiles > 1 ? kTileM : round_up(P, 8);
    h.k_splits = 1;
    h.kb_per_split = (c->cfg.H_d + c->cfg.H + kBlockK - 1) / kBlockK;
    finish_plan(c, &h, c->cfg.d_c, h.kb_per_split, c->tune.head_stages, want, N);
    return h;
}

// rounds of tiles the slowest CTA (or pair) of a plan works through
long long plan_waves(const Plan& p)
{
    if (p.pair && p.carry) return p.tiles_per_cta;        // teams: every pair walks its own range
    const long long units = p.pair ? p.ctas / 2 : p.ctas;
    const long long items = (long long)p.m_tiles * p.n_tiles * (p.k_splits > 0 ? p.k_splits : 1);
    return units > 0 ? (items + units - 1) / units : 0;
}

bool plan_fused(const wisv_ctx* c, int R, int P, Plan* lm, Plan* hd)
{
    if (c->tune.head_ctas < 0 || R < 1 || P < 1) return false;
    const bool small = R <= kTileM && P <= kTileM;
    // up to 256 window rows: the LM head runs on CTA pairs (one row tile of 256, still bound by HBM) and the
    // decision head on a few clusters of the same launch
    const bool with_pairs = !small && R <= kPairTileM && P <= kPairTileM && c->max_pairs > 2 &&
                            !c->tune.lm_single_cta && !c->tune.lm_tile_n;
    if (small || with_pairs) {
        const int head_m_tiles = (P + kTileM - 1) / kTileM;
        int want = c->tune.head_ctas > 0 ? c->tune.head_ctas : (head_m_tiles > 1 ? kFusedHeadCtasTwoTiles : kFusedHeadCtas);
        if (want > c->sm_count / 2) want = c->sm_count / 2;
        if (want < 1) return false;
        const Plan h = plan_head_beside(c, P, want);
        *hd = h;
        if (small) *lm = plan_lm(c, R, true, c->sm_count - h.ctas);
        else *lm = plan_lm(c, R, false, 0, (h.ctas + 1) / 2);
        return true;
    }
    // More rows (tensor-bound, tiles dealt out round-robin): giving SMs to the decision head pays only if the LM
    // head does not need another round of tiles for it and the head finishes well inside the LM head's time.
    // Times are counted in tiles: an LM-head tile and a decision-head item both walk a K range of similar cost
    // (64 K blocks of 128 x 256 against 96 of 128 x 128), so an item is taken as 1.2 tiles.
    if (c->tune.lm_tile_n) return false;
    const Plan base = plan_lm(c, R);
    const long long base_waves = plan_waves(base);
    for (int want = 2; want <= 16; want += 2) {
        if (c->tune.head_ctas > 0 && want != round_up(c->tune.head_ctas, 2)) continue;
        if (want > c->sm_count / 4) break;
        const Plan h = plan_head_beside(c, P, want);
        const Plan l = plan_lm(c, R, false, c->sm_count - round_up(h.ctas, 2), (h.ctas + 1) / 2);
        if (l.pair != base.pair || plan_waves(l) != base_waves) continue;
        const long long head_rounds = plan_waves(h);
        if (c->tune.head_ctas == 0 && head_rounds * 12 > base_waves * 8) continue;     // 1.2 tiles each, 80 % of the time
        *hd = h; *lm = l;
        return true;
    }
    return false;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

void free_ctx(wisv_ctx* c)
{
    if (!c) return;
    cudaFree(c->X); cudaFree(c->Z); cudaFree(c->W1p); cudaFree(c->W1c); cudaFree(c->lm_part);
    cudaFree(c->head_part); cudaFree(c->row_tok); cudaFree(c->row_flag); cudaFree(c->tok_logit);
    cudaFree(c->pos_req); cudaFree(c->pos_i); cudaFree(c->err); cudaFree(c->splitk_buf); cudaFree(c->splitk_count);
    cudaFree(c->saved_arg); cudaFree(c->saved_mask); cudaFree(c->done_count);
    if (c->prof_ev) {
        for (int i = 0; i < c->prof_n * (kStages + 1); ++i) cudaEventDestroy(c->prof_ev[i]);
        free(c->prof_ev);
    }
    HostStaging& h = c->hs;
    cudaFree(h.target_hidden); cudaFree(h.draft_hidden); cudaFree(h.dev_in);
    for (int i = 0; i < 8; ++i) if (h.copy_ev[i]) cudaEventDestroy(h.copy_ev[i]);
    if (h.copy_stream) cudaStreamDestroy(h.copy_stream);
    if (h.pin) cudaFreeHost(h.pin);
    (void)cudaGetLastError();
    delete c;
}

template <typename T>
int dev_alloc(T** p, size_t n)
{
    void* q = nullptr;
    if (cudaMalloc(&q, (n ? n : 1) * sizeof(T)) != cudaSuccess) { (void)cudaGetLastError(); return WISV_ENOMEM; }
    *p = static_cast<T*>(q);
    return WISV_OK;
}

// Device address of a pinned host array if the kernels can read it in place (registered with CUDA, 16-byte aligned,
// at most kZeroCopyBytes), else `staged`.
constexpr size_t kZeroCopyBytes = 1u << 20;
constexpr size_t kSmallInputsInPlace = 8u << 10;   // packed small inputs up to this size are not copied either
constexpr size_t kPipelineBytes = 32u << 20;       // host-buffer calls with at least this much hidden state travel in groups
constexpr long long kPipelineFirstRows = 256;      // window rows of the first group; each later group is twice the one before
const void* mapped_or(const void* host, size_t bytes, const void* staged)
{
    if (!host || bytes == 0 || bytes > kZeroCopyBytes) return staged;
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, host) != cudaSuccess) { (void)cudaGetLastError(); return staged; }
    if (at.type != cudaMemoryTypeHost || !at.devicePointer) return staged;
    if (reinterpret_cast<uintptr_t>(at.devicePointer) & 15u) return staged;
    return at.devicePointer;
}

inline size_t pad16(size_t n) { return (n + 15) & ~size_t(15); }

// Offsets (past the 16 bytes that hold the mirrored error word) of the packed outputs for B requests, R rows, T drafted tokens and
// P evaluated positions; returns the bytes used. Order: accept_len, correction, argmax, lse, p_draft, head_prob,
// mismatch_mask, n_mismatch, status.
enum { OUT_ACCEPT = 0, OUT_CORR, OUT_ARGMAX, OUT_LSE, OUT_PDRAFT, OUT_HEADP, OUT_MASK, OUT_NMIS, OUT_STATUS, OUT_FIELDS };
size_t out_arena_layout(int B, int R, int T, int P, size_t* off)
{
    const size_t sz[OUT_FIELDS] = {4u * (size_t)B, 4u * (size_t)B, 4u * (size_t)R, 4u * (size_t)R, 4u * (size_t)T,
                                   4u * (size_t)P, 8u * (size_t)B, 4u * (size_t)B, 4u * (size_t)B};
    size_t at = 0;
    for (int i = 0; i < OUT_FIELDS; ++i) { if (off) off[i] = at; at += pad16(sz[i]); }
    return at;
}

// The same for the small inputs: k_off, draft_tokens, sel_off, sel_pos, csi, draft_q, uniforms.
// IN_KOFF_G / IN_SELOFF_G: the offsets again, rebased to zero for each group of requests of a pipelined call.
constexpr int kMaxCopyGroups = 8;
enum { IN_KOFF = 0, IN_TOK, IN_SELOFF, IN_SELPOS, IN_CSI, IN_Q, IN_U, IN_KOFF_G, IN_SELOFF_G, IN_FIELDS };
size_t in_arena_layout(int B, int T, int P, int d_c, size_t* off, size_t* bytes)
{
    const size_t sz[IN_FIELDS] = {4u * ((size_t)B + 1), 4u * (size_t)T, 4u * ((size_t)B + 1), 4u * (size_t)P,
                                  4u * (size_t)B * (size_t)d_c, 4u * (size_t)T, 4u * (size_t)T,
                                  4u * ((size_t)B + kMaxCopyGroups), 4u * ((size_t)B + kMaxCopyGroups)};
    size_t at = 0;
    for (int i = 0; i < IN_FIELDS; ++i) { if (off) off[i] = at; if (bytes) bytes[i] = sz[i]; at += pad16(sz[i]); }
    return at;
}

enum { PHASE_FULL = 0, PHASE_LOCALIZE = 1, PHASE_DECIDE = 2, PHASE_GATHERED = 3, PHASE_SHARD = 4 };

int validate_batch(const wisv_ctx* c, const wisv_batch* b, const wisv_result* r, int* T_out, int* R_out, int* P_out,
                   int phase = PHASE_FULL)
{
    if (!c || !b || (!r && phase != PHASE_SHARD)) return WISV_EINVAL;
    if (b->B < 0 || b->K < 0) return WISV_ESHAPE;
    if (b->mode & ~3u) return WISV_EINVAL;
    if (b->target_hidden_dtype < 0 || b->target_hidden_dtype > WISV_DT_F16 || b->draft_hidden_dtype < 0 ||
        b->draft_hidden_dtype > WISV_DT_F16) return WISV_EINVAL;
    const bool sh = (b->mode & WISV_MODE_SH) != 0;
    const bool stoch = (b->mode & WISV_ACCEPT_STOCHASTIC) != 0;
    if (b->K == 0 && !b->k_off && b->B > 0 && b->T_total != 0) return WISV_EINVAL;
    if (b->K > WISV_MAX_K) return WISV_ESHAPE;
    long long T = b->k_off ? (long long)b->T_total : (long long)b->B * b->K;
    if (b->k_off && b->K != 0) return WISV_EINVAL;
    if (!b->k_off && b->T_total != 0 && b->T_total != T) return WISV_ESHAPE;
    if (T < 0 || T > (long long)WISV_MAX_K * b->B) return WISV_ESHAPE;
    const long long R = T + b->B;
    if (b->B > c->cfg.max_requests || R > c->cfg.max_rows) return WISV_ECAPACITY;
    long long P = T;
    if (phase == PHASE_LOCALIZE || phase == PHASE_SHARD) {
        P = 0;
    } else if (sh) {
        if (b->M_sel < 0) return WISV_ESHAPE;
        if (b->M_sel > c->max_pos || b->M_sel > T) return b->M_sel > T ? WISV_ESHAPE : WISV_ECAPACITY;
        P = b->M_sel;
        if (b->B > 0 && !b->sel_off) return WISV_EINVAL;
        if (P > 0 && !b->sel_pos) return WISV_EINVAL;
    }
    if (P > c->max_pos) return WISV_ECAPACITY;
    if (b->B > 0) {
        if (!b->target_hidden) return WISV_EINVAL;
        if (phase != PHASE_LOCALIZE && phase != PHASE_SHARD && (!r || !r->accept_len || !r->correction_token))
            return WISV_EINVAL;
        if (phase != PHASE_DECIDE && T > 0 && !b->draft_tokens) return WISV_EINVAL;
        if (P > 0 && (!b->draft_hidden || (c->cfg.d_c > 0 && !b->csi))) return WISV_EINVAL;
        if (phase != PHASE_DECIDE && phase != PHASE_SHARD && stoch && T > 0 && (!b->draft_q || !b->uniforms))
            return WISV_EINVAL;
        if (!aligned16(b->target_hidden) || (P > 0 && !aligned16(b->draft_hidden))) return WISV_EALIGN;
    }
    if (!(b->tau != b->tau) && b->tau < 0.0f) return WISV_EINVAL;
    *T_out = (int)T; *R_out = (int)R; *P_out = (int)P;
    return WISV_OK;
}

// Launch with programmatic stream serialisation: the kernel may be scheduled while its predecessor in
// the stream is still running; it synchronises with it through griddepcontrol.wait in device code.
template <typename... KArgs, typename... Args>
int launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args)
{
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    WISV_CUDA(cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...));
    return WISV_OK;
}

// index of the tensor map whose box is `tile_n` weight rows high, and of the one 16 rows lower (the second
// tile height of a balanced plan; never used when tile_n is 16)
inline int map_hi(const Plan& pl) { return pl.tile_n / 16 - 1; }
inline int map_lo(const Plan& pl) { return pl.tile_n / 16 - 2 > 0 ? pl.tile_n / 16 - 2 : 0; }

// tensor maps of the pair kernel's weight tiles: each CTA of a pair loads half of a tile's rows
inline int pair_map_hi(const Plan& pl) { return pl.tile_n / 32 - 1; }
inline int pair_map_lo(const Plan& pl) { return pl.tile_n / 32 - 2 > 0 ? pl.tile_n / 32 - 2 : 0; }
// tensor maps of the CTA-pair LM head: half a row block of window rows; half a tile of tile_n (or tile_n - 32) weight rows
inline const CUtensorMap& pair_tm_x(const wisv_ctx* c, const Plan& pl)
{
    return pl.box3d ? c->tmX3[pl.kbs / 4][pl.n_cols / 16 - 1] : c->tmX[pl.n_cols / 16 - 1];
}
inline const CUtensorMap& pair_tm_w(const wisv_ctx* c, const Plan& pl, bool lower)
{
    const int i = lower ? pair_map_lo(pl) : pair_map_hi(pl);
    return pl.box3d ? c->tmW3[pl.kbs / 4][i] : c->tmW[i];
}

PairParams pair_params(const wisv_ctx* c, const Plan& pl, int R)
{
    const wisv_config& cf = c->cfg;
    PairParams sp;
    memset(&sp, 0, sizeof sp);
    sp.rows = R; sp.n_cols = pl.n_cols; sp.row_blocks = pl.n_blocks; sp.n_total = cf.V;
    sp.k_blocks = (cf.H + kBlockK - 1) / kBlockK; sp.carry = pl.carry; sp.n_tiles = pl.n_tiles;
    {
        // raster groups: keep a group's bf16 rows within 48 MB of L2 while the weights stream past them (measured at
        // 8704 rows: 3 groups of 25 MB and 2 of 36 MB read 4-6.5 GB and 2.6-5.4 GB from HBM per launch, the second
        // 1 % faster; one group of 71 MB reads 11 GB and is 10 % slower)
        const long long block_bytes = (long long)pl.n_cols * cf.H * 2;
        int bg_max = (int)((48ll << 20) / block_bytes);
        if (bg_max < 1) bg_max = 1;
        const int groups = (pl.n_blocks + bg_max - 1) / bg_max;
        sp.b_group = (pl.n_blocks + groups - 1) / groups;
    }
    sp.stages = pl.stages; sp.kbs = pl.kbs > 0 ? pl.kbs : 1; sp.units_base = pl.units_base; sp.units_rem = pl.units_rem;
    sp.tiles_per_pair = pl.tiles_per_cta > 0 ? pl.tiles_per_cta : 1; sp.tile_m = pl.tile_n;
    sp.team_pairs = pl.team_pairs > 0 ? pl.team_pairs : 1;
    sp.box3d = pl.box3d;
    sp.part_stride = pl.parts; sp.err = c->err;
    sp.lm_part = c->lm_part; sp.row_tok = c->row_tok; sp.tok_logit = c->tok_logit;
    return sp;
}

template <int EPI, bool HEAD_WAITS_LAST = true>
int launch_gemm(wisv_ctx* c, const CUtensorMap& tA, const CUtensorMap* tB, const GemmParams& gp, const Plan& pl,
                cudaStream_t st)
{
    const int rc = launch_pdl(gemm_rowreduce_kernel<EPI, HEAD_WAITS_LAST>, dim3(pl.ctas), dim3(kGemmThreads), pl.smem,
                              st, tA, tB[map_hi(pl)], tB[map_lo(pl)], gp);
    if (rc != WISV_OK) return rc;
    c->launches++;
    return WISV_OK;
}

// After a reported time-out: clear the error word and the split-K arrival counters (an aborted launch may have left
// them part-way, and a later round would then take an early item for the last arriver of its tile).
int reset_after_device_error(wisv_ctx* c)
{
    WISV_CUDA(cudaMemset(c->err, 0, sizeof(int32_t)));
    WISV_CUDA(cudaMemset(c->splitk_count, 0, sizeof(int32_t) * c->splitk_tiles));
    return WISV_OK;
}

GemmParams base_params(const wisv_ctx* c, const Plan& pl, int rows, int n_total, int kdim)
{
    GemmParams gp;
    memset(&gp, 0, sizeof gp);
    gp.rows = rows; gp.n_total = n_total; gp.k_blocks = (kdim + kBlockK - 1) / kBlockK;
    gp.tile_n = pl.tile_n; gp.m_tiles = pl.m_tiles; gp.n_tiles = pl.n_tiles; gp.stages = pl.stages;
    gp.a_rows = pl.a_rows; gp.carry = pl.carry; gp.part_stride = pl.parts;
    gp.k_splits = pl.k_splits; gp.kb_per_split = pl.kb_per_split;
    // row tiles with at most 64 valid rows (a small batch, or the ragged last tile of a large one): MMAs of 64
    // rows do the same job with half the tensor work
    gp.mma_m = c->tune.lm_mma_m != kTileM ? 64 : kTileM;
    gp.units_base = pl.units_base; gp.units_rem = pl.units_rem; gp.tiles_per_cta = pl.tiles_per_cta;
    gp.splitk_buf = c->splitk_buf; gp.splitk_count = c->splitk_count;
    gp.err = c->err;
    return gp;
}

}  // namespace

extern "C" {

int wisv_version(void) { return WISV_VERSION; }

const char* wisv_strerror(int code)
{
    switch (code) {
        case WISV_OK: return "ok";
        case WISV_EINVAL: return "invalid argument";
        case WISV_ESHAPE: return "dimension out of range";
        case WISV_EALIGN: return "pointer or pitch misaligned";
        case WISV_ECAPACITY: return "batch exceeds the context capacity";
        case WISV_ECUDA: return "CUDA call failed";
        case WISV_EARCH: return "device is not sm_100";
        case WISV_ENOMEM: return "out of memory";
        case WISV_EDEVICE: return "a kernel reported a pipeline time-out";
        default: return "unknown error";
    }
}

int wisv_create(const wisv_config* cfg, const wisv_weights* w, wisv_ctx** out)
{
    if (out) *out = nullptr;
    if (!cfg || !w || !out) return WISV_EINVAL;
    if (!w->lm_head || !w->W1 || !w->b1 || !w->w2) return WISV_EINVAL;
    if (cfg->act != WISV_ACT_RELU && cfg->act != WISV_ACT_GELU) return WISV_EINVAL;
    if (cfg->head_row_shift != 0 && cfg->head_row_shift != 1) return WISV_EINVAL;
    if (!(cfg->tau >= 0.0f)) return WISV_EINVAL;
    if (cfg->H < 64 || cfg->H % 8 || cfg->H_d < 8 || cfg->H_d % 8 || cfg->V < 1 || cfg->d_J < 1) return WISV_ESHAPE;
    if (cfg->d_c < 0 || cfg->d_c > WISV_MAX_DC) return WISV_ESHAPE;
    if (cfg->vocab_base < 0 || cfg->vocab_total < 0) return WISV_ESHAPE;
    if (cfg->vocab_total > 0 && (long long)cfg->vocab_base + cfg->V > cfg->vocab_total) return WISV_ESHAPE;
    if (cfg->vocab_total == 0 && cfg->vocab_base != 0) return WISV_ESHAPE;
    if (cfg->max_requests < 1 || cfg->max_rows < cfg->max_requests || cfg->max_sel < 0) return WISV_ESHAPE;
    if ((long long)cfg->max_rows > (long long)(WISV_MAX_K + 1) * cfg->max_requests) return WISV_ESHAPE;
    if (!aligned16(w->lm_head)) return WISV_EALIGN;

    int dev = 0;
    WISV_CUDA(cudaGetDevice(&dev));
    cudaDeviceProp prop;
    WISV_CUDA(cudaGetDeviceProperties(&prop, dev));
    if (prop.major != 10) return WISV_EARCH;

    // every GEMM instantiation may use the full opt-in shared memory
    WISV_CUDA(cudaFuncSetAttribute(gemm_rowreduce_kernel<EPI_LMHEAD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)prop.sharedMemPerBlockOptin));
    WISV_CUDA(cudaFuncSetAttribute(gemm_rowreduce_kernel<EPI_HEAD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)prop.sharedMemPerBlockOptin));
    WISV_CUDA(cudaFuncSetAttribute(gemm_rowreduce_kernel<EPI_HEAD, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)prop.sharedMemPerBlockOptin));
    WISV_CUDA(cudaFuncSetAttribute(gemm_rowreduce_kernel<EPI_RAW>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)prop.sharedMemPerBlockOptin));
    WISV_CUDA(cudaFuncSetAttribute(lmhead_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)prop.sharedMemPerBlockOptin));
    WISV_CUDA(cudaFuncSetAttribute(round_small_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)prop.sharedMemPerBlockOptin));

    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    WISV_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
    if (!fn || qres != cudaDriverEntryPointSuccess) return WISV_ECUDA;
    EncodeTiledFn encode = reinterpret_cast<EncodeTiledFn>(fn);

    wisv_ctx* c = new (std::nothrow) wisv_ctx();
    if (!c) return WISV_ENOMEM;
    c->cfg = *cfg;
    c->w = *w;
    c->device = dev;
    c->sm_count = prop.multiProcessorCount;
    c->max_smem = (int)prop.sharedMemPerBlockOptin;
    {
        // how many CTA pairs of the pair kernel fit on the device at once (sizes its persistent grid)
        cudaLaunchConfig_t qc;
        memset(&qc, 0, sizeof qc);
        qc.gridDim = dim3(2 * prop.multiProcessorCount); qc.blockDim = dim3(kGemmThreads);
        qc.dynamicSmemBytes = (size_t)prop.sharedMemPerBlockOptin;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, lmhead_pair_kernel, &qc) == cudaSuccess && n > 0) {
            c->max_pairs = n < prop.multiProcessorCount / 2 ? n : prop.multiProcessorCount / 2;
        } else {
            (void)cudaGetLastError();
            c->max_pairs = 0;          // pairs unavailable: the single-CTA kernel serves every size
        }
    }
    const int max_T = cfg->max_rows - 1;
    c->max_pos = cfg->max_sel > 0 ? (cfg->max_sel > max_T ? cfg->max_sel : max_T) : max_T;
    if (c->max_pos < 1) c->max_pos = 1;
    c->rows_alloc = round_up(cfg->max_rows, kPairTileM);
    c->pos_alloc = round_up(c->max_pos, kTileM);
    const int hd_h = cfg->H_d + cfg->H;

    // partial buffers sized for the worst plan at any row count up to the capacity
    size_t lm_elems = 0, head_elems = 0;
    {
        const int r1 = cfg->max_rows < kTileM ? cfg->max_rows : kTileM;
        // one row tile: at most one partial per (row, CTA), or per 16-row vocabulary tile when tuned
        lm_elems = (size_t)r1 * ((cfg->V + 15) / 16 < c->sm_count ? (cfg->V + 15) / 16 : c->sm_count);
        if (cfg->max_rows > kTileM) {
            // 129..256 rows on CTA pairs with carried ranges: up to one partial per (row, CTA of a pair)
            const int r2 = cfg->max_rows < kPairTileM ? cfg->max_rows : kPairTileM;
            const int pairs = (cfg->V + 31) / 32 < c->sm_count / 2 ? (cfg->V + 31) / 32 : c->sm_count / 2;
            const size_t e2 = (size_t)r2 * 2 * (pairs > 0 ? pairs : 1);
            if (e2 > lm_elems) lm_elems = e2;
        }
        if (cfg->max_rows > kTileM) {
            // several row tiles (single CTAs, when tuned so): one partial per (row, vocabulary tile of 256); several row
            // blocks on pairs: two, one per CTA; automatic plans only, a finer tuned tile is refused
            const size_t nt = (size_t)(cfg->V + kPairTileN - 1) / kPairTileN;
            const size_t e = (size_t)cfg->max_rows * 2 * nt;
            if (e > lm_elems) lm_elems = e;
        }
        if (cfg->max_rows > kPairTileM) {
            // teams of pairs: R rows x 2 partials x at most (pairs / ceil(R / 256)) pairs per team <= 512 per pair
            const size_t e = (size_t)2 * kPairMaxCols * (c->sm_count / 2 > 0 ? c->sm_count / 2 : 1);
            if (e > lm_elems) lm_elems = e;
        }
        head_elems = (size_t)c->max_pos * ((cfg->d_J + 15) / 16);
    }
    c->lm_part_elems = lm_elems;
    c->head_part_elems = head_elems;

    int rc = WISV_OK;
    do {
        if ((rc = dev_alloc(&c->X, (size_t)c->rows_alloc * cfg->H))) break;
        if ((rc = dev_alloc(&c->Z, (size_t)c->pos_alloc * hd_h))) break;
        if ((rc = dev_alloc(&c->W1p, (size_t)cfg->d_J * hd_h))) break;
        if ((rc = dev_alloc(&c->W1c, (size_t)cfg->d_J * (cfg->d_c > 0 ? cfg->d_c : 1)))) break;
        if ((rc = dev_alloc(&c->lm_part, lm_elems))) break;
        if ((rc = dev_alloc(&c->head_part, head_elems))) break;
        if ((rc = dev_alloc(&c->row_tok, (size_t)c->rows_alloc))) break;
        if ((rc = dev_alloc(&c->row_flag, (size_t)c->rows_alloc))) break;
        if ((rc = dev_alloc(&c->tok_logit, (size_t)c->rows_alloc))) break;
        if ((rc = dev_alloc(&c->pos_req, (size_t)c->pos_alloc))) break;
        if ((rc = dev_alloc(&c->pos_i, (size_t)c->pos_alloc))) break;
        if ((rc = dev_alloc(&c->err, 1))) break;
        if ((rc = dev_alloc(&c->done_count, 1))) break;
        if (cudaMemset(c->done_count, 0, sizeof(int32_t)) != cudaSuccess) { rc = WISV_ECUDA; break; }
        if ((rc = dev_alloc(&c->saved_arg, (size_t)c->rows_alloc))) break;
        if ((rc = dev_alloc(&c->saved_mask, (size_t)cfg->max_requests))) break;
        c->splitk_tiles = kSplitMaxRowTiles * ((cfg->d_J + 15) / 16);
        if ((rc = dev_alloc(&c->splitk_buf, (size_t)c->sm_count * kTileM * kSplitTileN))) break;
        if ((rc = dev_alloc(&c->splitk_count, (size_t)c->splitk_tiles))) break;
        if (cudaMemset(c->splitk_count, 0, sizeof(int32_t) * c->splitk_tiles) != cudaSuccess) { rc = WISV_ECUDA; break; }
        if (cudaMemset(c->X, 0, (size_t)c->rows_alloc * cfg->H * 2) != cudaSuccess ||
            cudaMemset(c->Z, 0, (size_t)c->pos_alloc * hd_h * 2) != cudaSuccess ||
            cudaMemset(c->err, 0, sizeof(int32_t)) != cudaSuccess) { rc = WISV_ECUDA; break; }

        split_w1_kernel<<<cfg->d_J, 256>>>(static_cast<const __nv_bfloat16*>(w->W1), c->W1p, c->W1c, cfg->d_J, hd_h,
                                           cfg->d_c);
        if (cudaGetLastError() != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) { rc = WISV_ECUDA; break; }
        c->launches++;

        for (int i = 0; i < kNumRowVariants && rc == WISV_OK; ++i) {
            const uint32_t rows = 8u * (i + 1);
            rc = encode_2d(encode, &c->tmX[i], c->X, (uint64_t)cfg->H, (uint64_t)c->rows_alloc, kBlockK, rows);
            if (rc == WISV_OK)
                rc = encode_2d(encode, &c->tmZ[i], c->Z, (uint64_t)hd_h, (uint64_t)c->pos_alloc, kBlockK, rows);
        }
        if (rc != WISV_OK) break;
        for (int i = 0; i < kNumTileVariants && rc == WISV_OK; ++i) {
            const uint32_t tn = 16u * (i + 1);
            rc = encode_2d(encode, &c->tmW[i], w->lm_head, (uint64_t)cfg->H, (uint64_t)cfg->V, kBlockK, tn);
            if (rc == WISV_OK)
                rc = encode_2d(encode, &c->tmW1[i], c->W1p, (uint64_t)hd_h, (uint64_t)cfg->d_J, kBlockK, tn);
        }
        if (rc == WISV_OK && cfg->H % kBlockK == 0 && cfg->H >= 2 * kBlockK) {
            // (a driver that refuses these maps only costs the wider boxes, not the context)
            int rc3 = WISV_OK;
            for (int q = 0; q < 2 && rc3 == WISV_OK; ++q) {
                const uint32_t kb = q ? 4u : 2u;
                for (int i = 0; i < kNumRowVariants && rc3 == WISV_OK; ++i)
                    rc3 = encode_3d(encode, &c->tmX3[q][i], c->X, (uint64_t)cfg->H, (uint64_t)c->rows_alloc, 8u * (i + 1), kb);
                for (int i = 0; i < kNumTileVariants / 2 && rc3 == WISV_OK; ++i)
                    rc3 = encode_3d(encode, &c->tmW3[q][i], w->lm_head, (uint64_t)cfg->H, (uint64_t)cfg->V, 16u * (i + 1), kb);
            }
            c->have_box3d = rc3 == WISV_OK;
        }
    } while (0);
    if (rc != WISV_OK) { free_ctx(c); return rc; }
    *out = c;
    return WISV_OK;
}

int wisv_destroy(wisv_ctx* ctx)
{
    if (!ctx) return WISV_EINVAL;
    free_ctx(ctx);
    return WISV_OK;
}

int wisv_plan(const wisv_ctx* c, int32_t R, int32_t P, int32_t* lm_tile_n, int32_t* lm_tiles, int32_t* lm_ctas,
              int32_t* head_tile_n, int32_t* head_tiles, int32_t* head_ctas)
{
    if (!c || R < 1 || P < 0) return WISV_EINVAL;
    Plan a, h;
    if (!plan_fused(c, R, P, &a, &h)) {
        a = plan_lm(c, R);
        h = plan_head(c, P > 0 ? P : 1);
    }
    if (lm_tile_n) *lm_tile_n = a.tile_n;
    if (lm_tiles) *lm_tiles = a.m_tiles * a.n_tiles;
    if (lm_ctas) *lm_ctas = a.ctas;
    if (head_tile_n) *head_tile_n = h.tile_n;
    if (head_tiles) *head_tiles = P > 0 ? h.m_tiles * h.n_tiles : 0;
    if (head_ctas) *head_ctas = P > 0 ? h.ctas : 0;
    return WISV_OK;
}

int wisv_plan_kernels(const wisv_ctx* c, int32_t R, int32_t P)
{
    if (!c || R < 1 || P < 0) return WISV_EINVAL;
    Plan a, h;
    if (plan_fused(c, R, P, &a, &h)) return 3;        // pack, LM head + decision head, merge/scan
    return P > 0 ? 4 : 3;
}

int wisv_plan_host(const wisv_config* cfg, int32_t sm_count, int32_t max_smem_bytes, int32_t R, int32_t P,
                   wisv_plan_info* out)
{
    if (!cfg || !out || R < 1 || P < 0 || sm_count < 2 || max_smem_bytes < 64 * 1024) return WISV_EINVAL;
    if (cfg->H < 8 || cfg->V < 1 || cfg->H_d < 0 || cfg->d_c < 0 || cfg->d_c > kMaxDc || cfg->d_J < 1) return WISV_ESHAPE;
    wisv_ctx* c = new (std::nothrow) wisv_ctx();       // a plain record here: nothing is allocated on any device
    if (!c) return WISV_ENOMEM;
    c->cfg = *cfg;
    c->sm_count = sm_count;
    c->max_smem = max_smem_bytes;
    c->max_pairs = sm_count / 2;
    memset(out, 0, sizeof *out);
    Plan a{}, h{};
    const bool fused = plan_fused(c, R, P, &a, &h);
    const Plan alone = plan_lm(c, R);
    if (!fused) {
        a = alone;
        if (P > 0) h = plan_head(c, P);
    }
    out->kernels = fused ? 3 : (P > 0 ? 4 : 3);
    out->head_in_lm_launch = fused ? 1 : 0;
    out->lm_n_cols = a.n_cols; out->lm_row_blocks = a.n_blocks; out->lm_parts = a.parts;
    out->lm_pair = a.pair; out->lm_carry = a.carry; out->lm_tile_n = a.tile_n; out->lm_ctas = a.ctas;
    out->lm_m_tiles = a.m_tiles; out->lm_n_tiles = a.n_tiles; out->lm_stages = a.stages; out->lm_smem_bytes = (int32_t)a.smem;
    out->lm_units_base = a.units_base; out->lm_units_rem = a.units_rem; out->lm_tiles_per_cta = a.tiles_per_cta;
    // rounds of tiles: round-robin items, or the tiles of a pair's range when teams of pairs deal out the vocabulary
    out->lm_rounds = (a.carry && a.n_blocks <= 1) ? 0 : (int32_t)plan_waves(a);
    out->lm_rounds_alone = (alone.carry && alone.n_blocks <= 1) ? 0 : (int32_t)plan_waves(alone);
    if (P > 0) {
        out->head_carry = h.carry; out->head_tile_n = h.tile_n; out->head_ctas = h.ctas; out->head_m_tiles = h.m_tiles;
        out->head_n_tiles = h.n_tiles; out->head_k_splits = h.k_splits; out->head_kb_per_split = h.kb_per_split;
        out->head_stages = h.stages; out->head_smem_bytes = (int32_t)h.smem;
        out->head_units_base = h.units_base; out->head_units_rem = h.units_rem; out->head_tiles_per_cta = h.tiles_per_cta;
    }
    delete c;
    return WISV_OK;
}

int64_t wisv_launch_count(const wisv_ctx* c) { return c ? c->launches : 0; }

int wisv_set_tuning(wisv_ctx* c, const wisv_tuning* t)
{
    if (!c) return WISV_EINVAL;
    if (!t) { c->tune = wisv_tuning{0, 0, 0, 0, 0, 0, 0, 0, 0}; return WISV_OK; }
    const int32_t tn[2] = {t->lm_tile_n, t->head_tile_n};
    for (int i = 0; i < 2; ++i)
        if (tn[i] != 0 && (tn[i] < 16 || tn[i] > kMaxTileN || tn[i] % 16)) return WISV_ESHAPE;
    if (t->lm_stages < 0 || t->head_stages < 0 || t->lm_stages == 1 || t->head_stages == 1) return WISV_ESHAPE;
    if (t->lm_mma_m != 0 && t->lm_mma_m != 64 && t->lm_mma_m != 128) return WISV_ESHAPE;
    if (t->lm_teams < -1 || t->lm_teams > 1) return WISV_ESHAPE;
    if (t->lm_kb_per_stage != 0 && t->lm_kb_per_stage != 1 && t->lm_kb_per_stage != 2 && t->lm_kb_per_stage != 4) return WISV_ESHAPE;
    c->tune = *t;
    return WISV_OK;
}

}  // extern "C"

namespace {

// A barrier that nothing ever arrives on, waited for with the same bounded wait the GEMM kernels use:
// the wait must give up after limit_cycles and report through the error word, leaving the context usable.
__global__ void wait_probe_kernel(int32_t* err, unsigned long long limit_cycles)
{
    __shared__ uint64_t bar;
    __shared__ int flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        flag = 0;
        fence_barrier_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const bool ok = mbar_wait_bounded(smem_u32(&bar), 0, &flag, limit_cycles);
        if (!ok) atomicOr(err, 2);
    }
}

// One verification round, or one of its two phases (localize: pack rows + LM head + merge;
// decide: pack positions + decision head + scan on the candidate sets the localize call saved).
int run_round(wisv_ctx* c, const wisv_batch* b, const wisv_result* r, void* cuda_stream, int phase,
              float4* shard_out = nullptr, const float4* gathered = nullptr, int n_shards = 0)
{
    int T = 0, R = 0, P = 0;
    const int vrc = validate_batch(c, b, r, &T, &R, &P, phase);
    if (vrc != WISV_OK) return vrc;
    if (phase == PHASE_DECIDE || phase == PHASE_GATHERED) {
        if (!c->loc_valid) return WISV_EINVAL;
        if (b->B != c->loc_B || T != c->loc_T || (b->k_off ? 0 : b->K) != c->loc_K || b->k_off != c->loc_k_off)
            return WISV_ESHAPE;
    }
    if (b->B == 0) return WISV_OK;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const bool sh = (b->mode & WISV_MODE_SH) != 0;
    const bool stoch = (b->mode & WISV_ACCEPT_STOCHASTIC) != 0;
    const wisv_config& cf = c->cfg;

    cudaEvent_t* ev = nullptr;
    if (c->prof_n > 0) ev = c->prof_ev + (size_t)(c->prof_calls % c->prof_n) * (kStages + 1);

    BatchIndex ix{b->B, b->k_off ? 0 : b->K, b->k_off};

    // ---- 1. pack: bf16 window rows, head input rows, row -> token map
    if (ev) WISV_CUDA(cudaEventRecord(ev[0], st));
    PackParams pp;
    memset(&pp, 0, sizeof pp);
    const bool rows_done = phase == PHASE_DECIDE || phase == PHASE_GATHERED;   // reduced by an earlier call
    const int pack_rows = rows_done ? 0 : R;
    pp.vocab_base = cf.vocab_base; pp.vocab_total = cf.vocab_total > 0 ? cf.vocab_total : cf.V;
    pp.ix = ix; pp.R = pack_rows; pp.P = P; pp.H = cf.H; pp.H_d = cf.H_d; pp.V = cf.V; pp.shift = cf.head_row_shift;
    pp.mode_sh = sh ? 1 : 0; pp.R_total = R; pp.T_total = T;
    pp.target_hidden = b->target_hidden; pp.draft_hidden = b->draft_hidden; pp.draft_tokens = b->draft_tokens;
    pp.th_dtype = b->target_hidden_dtype; pp.dh_dtype = b->draft_hidden_dtype;
    pp.sel_off = b->sel_off; pp.sel_pos = b->sel_pos;
    pp.X = c->X; pp.Z = c->Z; pp.row_tok = c->row_tok; pp.row_flag = c->row_flag; pp.tok_logit = c->tok_logit;
    pp.pos_req = c->pos_req; pp.pos_i = c->pos_i;
    if (pack_rows + P > 0) {
        const int rc = launch_pdl(pack_kernel, dim3(pack_rows + P), dim3(256), 0, st, pp);
        if (rc != WISV_OK) return rc;
        c->launches++;
    }

    // ---- 2. LM head: logits reduced on the fly
    if (ev) WISV_CUDA(cudaEventRecord(ev[1], st));
    Plan pl{}, ph{};
    const bool fused = phase == PHASE_FULL && plan_fused(c, R, P, &pl, &ph);
    if (!fused) pl = plan_lm(c, R);
    if ((size_t)R * pl.parts > c->lm_part_elems) return WISV_ECAPACITY;
    if (fused) {
        // both GEMMs in one launch: LM-head CTAs and decision-head CTAs side by side
        if ((size_t)P * ph.parts > c->head_part_elems) return WISV_ECAPACITY;
        GemmParams gh = base_params(c, ph, P, cf.d_J, cf.H_d + cf.H);
        gh.head_part = c->head_part; gh.b1 = c->w.b1; gh.w2 = c->w.w2; gh.w1c = c->W1c; gh.csi = b->csi;
        gh.pos_req = c->pos_req; gh.d_c = cf.d_c; gh.act = cf.act;
        const size_t smem = pl.smem > ph.smem ? pl.smem : ph.smem;
        if (pl.pair) {
            const PairParams sp = pair_params(c, pl, R);
            const int rc = launch_pdl(lmhead_pair_kernel, dim3(pl.ctas + round_up(ph.ctas, 2)), dim3(kGemmThreads), smem,
                                      st, pair_tm_x(c, pl), pair_tm_w(c, pl, false), pair_tm_w(c, pl, true),
                                      sp, c->tmZ[ph.a_rows / 8 - 1], c->tmW1[map_hi(ph)], c->tmW1[map_lo(ph)], gh,
                                      pl.ctas, ph.ctas);
            if (rc != WISV_OK) return rc;
        } else {
            GemmParams gl = base_params(c, pl, R, cf.V, cf.H);
            gl.lm_part = c->lm_part; gl.row_tok = c->row_tok; gl.tok_logit = c->tok_logit;
            const int rc = launch_pdl(round_small_kernel, dim3(pl.ctas + ph.ctas), dim3(kGemmThreads), smem, st,
                                      c->tmX[pl.a_rows / 8 - 1], c->tmW[map_hi(pl)], c->tmW[map_lo(pl)],
                                      c->tmZ[ph.a_rows / 8 - 1], c->tmW1[map_hi(ph)], c->tmW1[map_lo(ph)], gl, gh,
                                      pl.ctas);
            if (rc != WISV_OK) return rc;
        }
        c->launches++;
    } else if (!rows_done && pl.pair) {
        const PairParams sp = pair_params(c, pl, R);
        GemmParams none;
        memset(&none, 0, sizeof none);
        const int rc = launch_pdl(lmhead_pair_kernel, dim3(pl.ctas), dim3(kGemmThreads), pl.smem, st,
                                  pair_tm_x(c, pl), pair_tm_w(c, pl, false), pair_tm_w(c, pl, true), sp,
                                  c->tmZ[0], c->tmW1[0], c->tmW1[0], none, pl.ctas, 0);
        if (rc != WISV_OK) return rc;
        c->launches++;
    } else if (!rows_done) {
        GemmParams gp = base_params(c, pl, R, cf.V, cf.H);
        gp.lm_part = c->lm_part; gp.row_tok = c->row_tok; gp.tok_logit = c->tok_logit;
        const int rc = launch_gemm<EPI_LMHEAD>(c, c->tmX[pl.a_rows / 8 - 1], c->tmW, gp, pl, st);
        if (rc != WISV_OK) return rc;
    }

    if (phase == PHASE_SHARD) {
        // this shard's rows reduced to one partial each; the caller gathers them across shards
        const int rc = launch_pdl(shard_rows_kernel, dim3((R + 3) / 4), dim3(128), 0, st,
                                  (const float4*)c->lm_part, pl.parts, R, (int)cf.vocab_base,
                                  (const int32_t*)c->row_tok, (const float*)c->tok_logit, shard_out);
        if (rc != WISV_OK) return rc;
        c->launches++;
        c->loc_valid = true; c->loc_B = b->B; c->loc_T = T; c->loc_K = b->k_off ? 0 : b->K; c->loc_k_off = b->k_off;
        return WISV_OK;
    }

    // ---- 3. decision head on the evaluated positions
    if (ev) WISV_CUDA(cudaEventRecord(ev[2], st));
    if (P > 0 && !fused) {
        ph = plan_head(c, P);
        if ((size_t)P * ph.parts > c->head_part_elems) return WISV_ECAPACITY;
        GemmParams gp = base_params(c, ph, P, cf.d_J, cf.H_d + cf.H);
        gp.head_part = c->head_part; gp.b1 = c->w.b1; gp.w2 = c->w.w2; gp.w1c = c->W1c; gp.csi = b->csi;
        gp.pos_req = c->pos_req; gp.d_c = cf.d_c; gp.act = cf.act;
        // Where an LM-head launch precedes it in this round the head may start early and wait at its end; in the
        // decide and gathered phases it follows the pack kernel directly and must wait before its first read.
        const int rc = rows_done ? launch_gemm<EPI_HEAD, false>(c, c->tmZ[ph.a_rows / 8 - 1], c->tmW1, gp, ph, st)
                                 : launch_gemm<EPI_HEAD, true>(c, c->tmZ[ph.a_rows / 8 - 1], c->tmW1, gp, ph, st);
        if (rc != WISV_OK) return rc;
    }

    // ---- 4. merge, localize, scan, emit
    if (ev) WISV_CUDA(cudaEventRecord(ev[3], st));
    TailParams tp;
    memset(&tp, 0, sizeof tp);
    tp.ix = ix; tp.P = P; tp.V = cf.V; tp.n_tiles_lm = pl.parts; tp.n_tiles_head = ph.parts; tp.mode_sh = sh ? 1 : 0;
    tp.T_total = T; tp.phase = phase; tp.saved_arg = c->saved_arg; tp.saved_mask = c->saved_mask;
    tp.vocab_base = cf.vocab_base; tp.part_rstride = pl.parts; tp.part_nstride = 1;
    tp.stochastic = stoch ? 1 : 0; tp.b2 = c->w.b2; tp.tau = (b->tau != b->tau) ? cf.tau : b->tau;
    tp.lm_part = c->lm_part;
    if (phase == PHASE_GATHERED) {
        tp.lm_part = gathered; tp.n_tiles_lm = n_shards; tp.part_rstride = 1; tp.part_nstride = R;
    }
    tp.tok_logit = c->tok_logit; tp.row_flag = c->row_flag; tp.draft_tokens = b->draft_tokens;
    tp.head_part = c->head_part; tp.pos_i = c->pos_i; tp.sel_off = b->sel_off; tp.draft_q = b->draft_q;
    tp.uniforms = b->uniforms;
    tp.accept_len = r->accept_len; tp.correction = r->correction_token; tp.argmax = r->argmax; tp.lse = r->lse;
    tp.p_draft = r->p_draft; tp.head_prob = r->head_prob;
    tp.mismatch_mask = reinterpret_cast<unsigned long long*>(r->mismatch_mask); tp.n_mismatch = r->n_mismatch;
    tp.status = r->status;
    tp.err_src = c->err; tp.err_copy = c->err_copy_next;
    c->err_copy_next = nullptr;
    tp.done_flag = c->done_flag_next; tp.done_count = c->done_count; tp.done_seq = c->done_seq;
    c->done_flag_next = nullptr;
    {
        // few requests: one warp per window row and head position, so nothing in a block runs one after the other
        // one block per request; its warps share out the request's rows and positions, each task a chain of loads.
        // 32 warps while all blocks are resident at once (two per SM), 8 otherwise (measured: 64-256 requests
        // 28-40 -> 19-35 us with 32 warps, 512 requests 55 us with 8 warps against 64 with 16)
        const int tail_threads = b->B <= 2 * c->sm_count ? 1024 : 256;
        const int rc = launch_pdl(tail_kernel, dim3(b->B), dim3(tail_threads), 0, st, tp);
        if (rc != WISV_OK) return rc;
    }
    c->launches++;
    if (ev) { WISV_CUDA(cudaEventRecord(ev[4], st)); c->prof_calls++; }
    if (phase == PHASE_LOCALIZE) {
        c->loc_valid = true; c->loc_B = b->B; c->loc_T = T; c->loc_K = b->k_off ? 0 : b->K; c->loc_k_off = b->k_off;
    } else {
        c->loc_valid = false;
    }
    return WISV_OK;
}

}  // namespace

extern "C" {

int wisv_verify(wisv_ctx* c, const wisv_batch* b, const wisv_result* r, void* cuda_stream)
{
    return run_round(c, b, r, cuda_stream, PHASE_FULL);
}

int wisv_localize(wisv_ctx* c, const wisv_batch* b, const wisv_result* r, void* cuda_stream)
{
    return run_round(c, b, r, cuda_stream, PHASE_LOCALIZE);
}

int wisv_decide(wisv_ctx* c, const wisv_batch* b, const wisv_result* r, void* cuda_stream)
{
    return run_round(c, b, r, cuda_stream, PHASE_DECIDE);
}

int wisv_shard_rows(wisv_ctx* c, const wisv_batch* b, wisv_row_partial* out, void* cuda_stream)
{
    if (!out) return WISV_EINVAL;
    return run_round(c, b, nullptr, cuda_stream, PHASE_SHARD, reinterpret_cast<float4*>(out));
}

int wisv_verify_gathered(wisv_ctx* c, const wisv_batch* b, const wisv_row_partial* gathered, int32_t n_shards,
                         const wisv_result* r, void* cuda_stream)
{
    if (!gathered || n_shards < 1 || n_shards > 1024) return WISV_EINVAL;
    if ((reinterpret_cast<uintptr_t>(gathered) & 15u) != 0) return WISV_EALIGN;
    return run_round(c, b, r, cuda_stream, PHASE_GATHERED, nullptr, reinterpret_cast<const float4*>(gathered), n_shards);
}

int wisv_debug_logits(wisv_ctx* c, const float* target_hidden, int32_t R, float* logits_out, void* cuda_stream)
{
    if (!c || !target_hidden || !logits_out) return WISV_EINVAL;
    if (R < 1 || R > c->cfg.max_rows) return WISV_ECAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // rows are cast with the pack kernel, as a batch of R one-row windows without tokens
    PackParams pp;
    memset(&pp, 0, sizeof pp);
    pp.ix = BatchIndex{R, 0, nullptr}; pp.R = R; pp.R_total = R; pp.T_total = 0; pp.P = 0; pp.H = c->cfg.H; pp.H_d = c->cfg.H_d; pp.V = c->cfg.V;
    pp.target_hidden = target_hidden; pp.X = c->X; pp.row_tok = c->row_tok; pp.row_flag = c->row_flag;
    pp.tok_logit = c->tok_logit;
    pack_kernel<<<R, 256, 0, st>>>(pp);
    WISV_CUDA(cudaGetLastError());
    c->launches++;
    const Plan pl = plan_lm(c, R, true);            // the raw-logits epilogue exists for the single-CTA kernel only
    GemmParams gp = base_params(c, pl, R, c->cfg.V, c->cfg.H);
    gp.raw_out = logits_out;
    return launch_gemm<EPI_RAW>(c, c->tmX[pl.a_rows / 8 - 1], c->tmW, gp, pl, st);
}

int wisv_debug_wait_probe(wisv_ctx* c, uint64_t limit_cycles, void* cuda_stream)
{
    if (!c || limit_cycles == 0 || limit_cycles > 2000000000ull) return WISV_EINVAL;
    wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(c->err, limit_cycles);
    WISV_CUDA(cudaGetLastError());
    c->launches++;
    return WISV_OK;
}

int wisv_debug_poison(wisv_ctx* c, void* cuda_stream)
{
    if (!c) return WISV_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const wisv_config& cf = c->cfg;
    const size_t hd_h = (size_t)cf.H_d + cf.H;
    // 0xFF bytes: NaN as bf16 and as fp32; 0x7F bytes: 0x7F7F7F7F as int32 (no valid token, row or request)
    WISV_CUDA(cudaMemsetAsync(c->X, 0xFF, (size_t)c->rows_alloc * cf.H * 2, st));
    WISV_CUDA(cudaMemsetAsync(c->Z, 0xFF, (size_t)c->pos_alloc * hd_h * 2, st));
    WISV_CUDA(cudaMemsetAsync(c->lm_part, 0xFF, c->lm_part_elems * sizeof(float4), st));
    WISV_CUDA(cudaMemsetAsync(c->head_part, 0xFF, c->head_part_elems * sizeof(float), st));
    WISV_CUDA(cudaMemsetAsync(c->splitk_buf, 0xFF, (size_t)c->sm_count * kTileM * kSplitTileN * sizeof(float), st));
    WISV_CUDA(cudaMemsetAsync(c->tok_logit, 0xFF, (size_t)c->rows_alloc * sizeof(float), st));
    WISV_CUDA(cudaMemsetAsync(c->row_tok, 0x7F, (size_t)c->rows_alloc * sizeof(int32_t), st));
    WISV_CUDA(cudaMemsetAsync(c->row_flag, 0x7F, (size_t)c->rows_alloc * sizeof(int32_t), st));
    WISV_CUDA(cudaMemsetAsync(c->pos_req, 0x7F, (size_t)c->pos_alloc * sizeof(int32_t), st));
    WISV_CUDA(cudaMemsetAsync(c->pos_i, 0x7F, (size_t)c->pos_alloc * sizeof(int32_t), st));
    WISV_CUDA(cudaMemsetAsync(c->saved_arg, 0x7F, (size_t)c->rows_alloc * sizeof(int32_t), st));
    WISV_CUDA(cudaMemsetAsync(c->saved_mask, 0xFF, (size_t)cf.max_requests * sizeof(unsigned long long), st));
    c->loc_valid = false;
    return WISV_OK;
}

int wisv_device_error(wisv_ctx* c, void* cuda_stream, int32_t* flags)
{
    if (!c || !flags) return WISV_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    WISV_CUDA(cudaStreamSynchronize(st));
    int32_t v = 0;
    WISV_CUDA(cudaMemcpy(&v, c->err, sizeof v, cudaMemcpyDeviceToHost));
    if (v != 0) {
        const int rc = reset_after_device_error(c);
        if (rc != WISV_OK) return rc;
    }
    *flags = v;
    return WISV_OK;
}

int wisv_profile_enable(wisv_ctx* c, int32_t n_calls)
{
    if (!c || n_calls < 0 || n_calls > 4096) return WISV_EINVAL;
    if (c->prof_ev) {
        for (int i = 0; i < c->prof_n * (kStages + 1); ++i) cudaEventDestroy(c->prof_ev[i]);
        free(c->prof_ev);
        c->prof_ev = nullptr;
    }
    c->prof_n = 0;
    c->prof_calls = 0;
    if (n_calls == 0) return WISV_OK;
    c->prof_ev = static_cast<cudaEvent_t*>(calloc((size_t)n_calls * (kStages + 1), sizeof(cudaEvent_t)));
    if (!c->prof_ev) return WISV_ENOMEM;
    for (int i = 0; i < n_calls * (kStages + 1); ++i) WISV_CUDA(cudaEventCreate(&c->prof_ev[i]));
    c->prof_n = n_calls;
    return WISV_OK;
}

int wisv_profile_read(wisv_ctx* c, int32_t stage, float* ms, int32_t cap, int32_t* n_out)
{
    if (!c || !ms || !n_out || stage < 0 || stage >= kStages || cap < 0) return WISV_EINVAL;
    *n_out = 0;
    if (c->prof_n == 0) return WISV_OK;
    const long long have = c->prof_calls < c->prof_n ? c->prof_calls : c->prof_n;
    const long long first = c->prof_calls - have;
    int n = 0;
    for (long long k = first; k < c->prof_calls && n < cap; ++k) {
        cudaEvent_t* ev = c->prof_ev + (size_t)(k % c->prof_n) * (kStages + 1);
        WISV_CUDA(cudaEventSynchronize(ev[kStages]));
        float t = 0.0f;
        WISV_CUDA(cudaEventElapsedTime(&t, ev[stage], ev[stage + 1]));
        ms[n++] = t;
    }
    *n_out = n;
    return WISV_OK;
}

int wisv_verify_host(wisv_ctx* c, const wisv_batch* hb, const wisv_result* hr, void* cuda_stream)
{
    if (!c || !hb || !hr) return WISV_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    HostStaging& h = c->hs;
    const wisv_config& cf = c->cfg;
    const int maxB = cf.max_requests, maxR = cf.max_rows;
    if (!h.ready) {
        int rc = WISV_OK;
        do {
            if ((rc = dev_alloc(&h.target_hidden, (size_t)maxR * cf.H))) break;
            if ((rc = dev_alloc(&h.draft_hidden, (size_t)c->max_pos * cf.H_d))) break;
            h.in_cap = in_arena_layout(maxB, maxR, c->max_pos, cf.d_c, nullptr, nullptr);
            h.out_cap = 16 + out_arena_layout(maxB, maxR, maxR, c->max_pos, nullptr);
            if ((rc = dev_alloc(&h.dev_in, h.in_cap))) break;
            if (cudaHostAlloc(reinterpret_cast<void**>(&h.pin), h.in_cap + h.out_cap, cudaHostAllocMapped) != cudaSuccess ||
                cudaHostGetDevicePointer(reinterpret_cast<void**>(&h.pin_dev), h.pin, 0) != cudaSuccess) {
                (void)cudaGetLastError();
                if (h.pin) cudaFreeHost(h.pin);
                h.pin = nullptr;
                rc = WISV_ENOMEM;
                break;
            }
        } while (0);
        if (rc != WISV_OK) return rc;
        h.ready = true;
    }
    // sizes of this call as the batch states them; out-of-range ones are left for validate_batch to name
    const int B = hb->B;
    const bool sh = (hb->mode & WISV_MODE_SH) != 0;
    const bool stoch = (hb->mode & WISV_ACCEPT_STOCHASTIC) != 0;
    const long long T_ll = hb->k_off ? (long long)hb->T_total : (long long)hb->B * hb->K;
    const long long P_ll = sh ? (long long)hb->M_sel : T_ll;
    const bool fits = B >= 0 && B <= maxB && T_ll >= 0 && T_ll + B <= maxR && P_ll >= 0 && P_ll <= c->max_pos;
    const int T = fits ? (int)T_ll : 0, P = fits ? (int)P_ll : 0, R = fits ? T + B : 0;
    size_t ioff[IN_FIELDS], ibytes[IN_FIELDS], ooff[OUT_FIELDS];
    const size_t in_used = in_arena_layout(fits ? B : 0, T, P, cf.d_c, ioff, ibytes);
    const size_t out_used = 16 + out_arena_layout(fits ? B : 0, R, T, P, ooff);
    if (in_used > h.in_cap || out_used > h.out_cap) return WISV_ECAPACITY;
    uint8_t* pin_in = h.pin;
    uint8_t* pin_out = h.pin + h.in_cap;
    uint8_t* dev_out = h.pin_dev + h.in_cap + 16;   // the tail kernel writes the results straight to host memory
    // the device-side view of the batch, validated before any copy
    wisv_batch db = *hb;
    wisv_result dr;
    memset(&dr, 0, sizeof dr);
    const void* src[IN_FIELDS] = {hb->k_off, hb->draft_tokens, sh ? hb->sel_off : nullptr, sh ? hb->sel_pos : nullptr,
                                  hb->csi, stoch ? hb->draft_q : nullptr, stoch ? hb->uniforms : nullptr};
    // A few KB of small inputs are read by the kernels in place from the pinned block (each is touched once or
    // twice per round, and a separate copy costs more in submission and DMA latency than those reads over PCIe);
    // larger ones are copied to the device in one piece.
    const bool small_in_place = in_used <= kSmallInputsInPlace;
    uint8_t* in_base = small_in_place ? h.pin_dev : h.dev_in;
    db.k_off = hb->k_off ? reinterpret_cast<int32_t*>(in_base + ioff[IN_KOFF]) : nullptr;
    // a small hidden-state array in pinned memory is read in place by the pack kernel (one pass over PCIe, no
    // separate copy to wait for); a large or pageable one goes through the copy engine
    auto elem = [](int dt) -> size_t { return dt == WISV_DT_F32 ? 4u : 2u; };
    const size_t th_es = elem(hb->target_hidden_dtype), dh_es = elem(hb->draft_hidden_dtype);
    const size_t th_bytes = th_es * (size_t)R * cf.H, dh_bytes = dh_es * (size_t)P * cf.H_d;
    const void* th_dev = mapped_or(hb->target_hidden, th_bytes, h.target_hidden);
    const void* dh_dev = mapped_or(hb->draft_hidden, dh_bytes, h.draft_hidden);
    db.target_hidden = hb->target_hidden ? th_dev : nullptr;
    db.draft_tokens = hb->draft_tokens ? reinterpret_cast<int32_t*>(in_base + ioff[IN_TOK]) : nullptr;
    db.draft_hidden = hb->draft_hidden ? dh_dev : nullptr;
    db.sel_off = hb->sel_off ? reinterpret_cast<int32_t*>(in_base + ioff[IN_SELOFF]) : nullptr;
    db.sel_pos = hb->sel_pos ? reinterpret_cast<int32_t*>(in_base + ioff[IN_SELPOS]) : nullptr;
    db.csi = hb->csi ? reinterpret_cast<float*>(in_base + ioff[IN_CSI]) : nullptr;
    db.draft_q = hb->draft_q ? reinterpret_cast<float*>(in_base + ioff[IN_Q]) : nullptr;
    db.uniforms = hb->uniforms ? reinterpret_cast<float*>(in_base + ioff[IN_U]) : nullptr;
    dr.accept_len = hr->accept_len ? reinterpret_cast<int32_t*>(dev_out + ooff[OUT_ACCEPT]) : nullptr;
    dr.correction_token = hr->correction_token ? reinterpret_cast<int32_t*>(dev_out + ooff[OUT_CORR]) : nullptr;
    dr.argmax = hr->argmax ? reinterpret_cast<int32_t*>(dev_out + ooff[OUT_ARGMAX]) : nullptr;
    dr.lse = hr->lse ? reinterpret_cast<float*>(dev_out + ooff[OUT_LSE]) : nullptr;
    dr.p_draft = hr->p_draft ? reinterpret_cast<float*>(dev_out + ooff[OUT_PDRAFT]) : nullptr;
    dr.head_prob = hr->head_prob ? reinterpret_cast<float*>(dev_out + ooff[OUT_HEADP]) : nullptr;
    dr.mismatch_mask = hr->mismatch_mask ? reinterpret_cast<uint64_t*>(dev_out + ooff[OUT_MASK]) : nullptr;
    dr.n_mismatch = hr->n_mismatch ? reinterpret_cast<int32_t*>(dev_out + ooff[OUT_NMIS]) : nullptr;
    dr.status = hr->status ? reinterpret_cast<int32_t*>(dev_out + ooff[OUT_STATUS]) : nullptr;
    int Tv = 0, Rv = 0, Pv = 0;
    const int vrc = validate_batch(c, &db, &dr, &Tv, &Rv, &Pv);
    if (vrc != WISV_OK) return vrc;
    if (!fits) return WISV_ESHAPE;
    if (B == 0) return WISV_OK;
    if (hb->k_off) {
        // here the row offsets are host memory: check what wisv_verify has to leave to the device's status bits
        if (hb->k_off[0] != 0 || hb->k_off[B] != T) return WISV_ESHAPE;
        for (int i = 0; i < B; ++i) {
            const long long kb = (long long)hb->k_off[i + 1] - hb->k_off[i];
            if (kb < 0 || kb > WISV_MAX_K) return WISV_ESHAPE;
        }
    }
    if (sh) {
        if (hb->sel_off[0] != 0 || hb->sel_off[B] != P) return WISV_ESHAPE;
        for (int i = 0; i < B; ++i)
            if (hb->sel_off[i + 1] < hb->sel_off[i]) return WISV_ESHAPE;
    }
    // Large batches: the hidden states cross PCIe for milliseconds, and windows are verified independently (Section
    // II-A), so the batch is cut into groups of whole requests, small ones first: group g is verified while group
    // g + 1 is still on its way (copies on a stream of the context's own, one event per group).
    int gb[kMaxCopyGroups + 1];
    int n_groups = 1;
    gb[0] = 0; gb[1] = B;
    auto tok_of = [&](int b) { return hb->k_off ? (long long)hb->k_off[b] : (long long)b * hb->K; };
    const bool staged = th_dev == h.target_hidden && (P == 0 || dh_dev == h.draft_hidden);
    if (staged && th_bytes + dh_bytes >= kPipelineBytes && B >= 2) {
        n_groups = 0;
        long long target = kPipelineFirstRows, step = kPipelineFirstRows;
        int prev = 0;
        while (prev < B && n_groups < kMaxCopyGroups - 1) {
            int b = prev + 1;
            while (b < B && tok_of(b + 1) + b + 1 <= target) ++b;       // whole requests up to `target` window rows
            if ((long long)R - (tok_of(b) + b) < 3 * kPipelineFirstRows) b = B;    // no small group at the end
            gb[++n_groups] = b;
            prev = b;
            step *= 2; target += step;
        }
        if (prev < B) gb[++n_groups] = B;
    }
    if (n_groups > 1) {
        // per-group offsets, rebased to zero, behind the plain ones in the packed block
        int32_t* kg = reinterpret_cast<int32_t*>(pin_in + ioff[IN_KOFF_G]);
        int32_t* sg = reinterpret_cast<int32_t*>(pin_in + ioff[IN_SELOFF_G]);
        size_t at = 0;
        for (int g = 0; g < n_groups; ++g)
            for (int b = gb[g]; b <= gb[g + 1]; ++b, ++at) {
                kg[at] = hb->k_off ? hb->k_off[b] - hb->k_off[gb[g]] : 0;
                sg[at] = sh ? hb->sel_off[b] - hb->sel_off[gb[g]] : 0;
            }
    }
    for (int i = 0; i < IN_KOFF_G; ++i)
        if (src[i] && ibytes[i] > 0) memcpy(pin_in + ioff[i], src[i], ibytes[i]);
    if (!small_in_place) WISV_CUDA(cudaMemcpyAsync(h.dev_in, pin_in, in_used, cudaMemcpyHostToDevice, st));
    memset(pin_out, 0, 4);
    // The merge/scan kernel stores a fresh sequence number next to the results when all of them are written;
    // watching that word costs less than a stream synchronisation at the end of a round of a few hundred
    // microseconds.  The stream is polled now and then as well, so a failed launch or kernel ends the wait.
    volatile int32_t* host_flag = reinterpret_cast<volatile int32_t*>(pin_out + 4);
    c->done_seq = c->done_seq == 0x7fffffff ? 1 : c->done_seq + 1;
    *host_flag = 0;
    int rc = WISV_OK;
    if (n_groups == 1) {
        if (th_dev != h.target_hidden)
            ;   // the pack kernel reads the caller's pinned array in place
        else if (hb->target_hidden)
            WISV_CUDA(cudaMemcpyAsync(h.target_hidden, hb->target_hidden, th_bytes, cudaMemcpyHostToDevice, st));
        if (dh_dev != h.draft_hidden)
            ;
        else if (hb->draft_hidden && P > 0)
            WISV_CUDA(cudaMemcpyAsync(h.draft_hidden, hb->draft_hidden, dh_bytes, cudaMemcpyHostToDevice, st));
        c->err_copy_next = reinterpret_cast<int32_t*>(h.pin_dev + h.in_cap);
        c->done_flag_next = reinterpret_cast<volatile int32_t*>(h.pin_dev + h.in_cap + 4);
        rc = wisv_verify(c, &db, &dr, cuda_stream);
    } else {
        if (!h.copy_stream) {
            WISV_CUDA(cudaStreamCreateWithFlags(&h.copy_stream, cudaStreamNonBlocking));
            for (int i = 0; i < kMaxCopyGroups; ++i) WISV_CUDA(cudaEventCreateWithFlags(&h.copy_ev[i], cudaEventDisableTiming));
        }
        // the staging buffers were last read by the previous call, which had completed before it returned; the
        // copies must still not overtake work the caller queued on `st` that this call's inputs may depend on
        WISV_CUDA(cudaEventRecord(h.copy_ev[0], st));
        WISV_CUDA(cudaStreamWaitEvent(h.copy_stream, h.copy_ev[0], 0));
        const uint8_t* th_src = static_cast<const uint8_t*>(hb->target_hidden);
        const uint8_t* dh_src = static_cast<const uint8_t*>(hb->draft_hidden);
        uint8_t* th_dst = reinterpret_cast<uint8_t*>(h.target_hidden);
        uint8_t* dh_dst = reinterpret_cast<uint8_t*>(h.draft_hidden);
        size_t off_at = 0;
        for (int g = 0; g < n_groups && rc == WISV_OK; ++g) {
            const int b0 = gb[g], b1 = gb[g + 1];
            const long long t0 = tok_of(b0), t1 = tok_of(b1);
            const long long r0 = t0 + b0, r1 = t1 + b1;
            const long long e0 = sh ? hb->sel_off[b0] : t0, e1 = sh ? hb->sel_off[b1] : t1;    // evaluated positions
            const size_t row_b = th_es * cf.H, pos_b = dh_es * cf.H_d;
            WISV_CUDA(cudaMemcpyAsync(th_dst + r0 * row_b, th_src + r0 * row_b, (size_t)(r1 - r0) * row_b,
                                      cudaMemcpyHostToDevice, h.copy_stream));
            if (e1 > e0)
                WISV_CUDA(cudaMemcpyAsync(dh_dst + e0 * pos_b, dh_src + e0 * pos_b, (size_t)(e1 - e0) * pos_b,
                                          cudaMemcpyHostToDevice, h.copy_stream));
            WISV_CUDA(cudaEventRecord(h.copy_ev[g], h.copy_stream));
            WISV_CUDA(cudaStreamWaitEvent(st, h.copy_ev[g], 0));
            wisv_batch gbt = db;
            wisv_result grs = dr;
            gbt.B = b1 - b0;
            gbt.T_total = (int32_t)(t1 - t0);
            gbt.k_off = hb->k_off ? reinterpret_cast<int32_t*>(in_base + ioff[IN_KOFF_G]) + off_at : nullptr;
            gbt.sel_off = sh ? reinterpret_cast<int32_t*>(in_base + ioff[IN_SELOFF_G]) + off_at : nullptr;
            off_at += (size_t)(b1 - b0) + 1;
            gbt.target_hidden = th_dst + r0 * row_b;
            gbt.draft_hidden = hb->draft_hidden ? dh_dst + e0 * pos_b : nullptr;
            gbt.draft_tokens = db.draft_tokens ? db.draft_tokens + t0 : nullptr;
            gbt.sel_pos = db.sel_pos ? db.sel_pos + e0 : nullptr;
            gbt.M_sel = sh ? (int32_t)(e1 - e0) : 0;
            gbt.csi = db.csi ? db.csi + (size_t)b0 * cf.d_c : nullptr;
            gbt.draft_q = db.draft_q ? db.draft_q + t0 : nullptr;
            gbt.uniforms = db.uniforms ? db.uniforms + t0 : nullptr;
            grs.accept_len = dr.accept_len + b0; grs.correction_token = dr.correction_token + b0;
            if (dr.argmax) grs.argmax = dr.argmax + r0;
            if (dr.lse) grs.lse = dr.lse + r0;
            if (dr.p_draft) grs.p_draft = dr.p_draft + t0;
            if (dr.head_prob) grs.head_prob = dr.head_prob + e0;
            if (dr.mismatch_mask) grs.mismatch_mask = dr.mismatch_mask + b0;
            if (dr.n_mismatch) grs.n_mismatch = dr.n_mismatch + b0;
            if (dr.status) grs.status = dr.status + b0;
            if (g == n_groups - 1) {
                // the last group's merge/scan kernel mirrors the error word and announces completion
                c->err_copy_next = reinterpret_cast<int32_t*>(h.pin_dev + h.in_cap);
                c->done_flag_next = reinterpret_cast<volatile int32_t*>(h.pin_dev + h.in_cap + 4);
            }
            rc = wisv_verify(c, &gbt, &grs, cuda_stream);
        }
    }
    c->err_copy_next = nullptr;
    c->done_flag_next = nullptr;
    if (rc != WISV_OK) return rc;
    for (unsigned spins = 1; *host_flag != c->done_seq; ++spins) {
        if ((spins & 0x3FFu) == 0) {
            const cudaError_t q = cudaStreamQuery(st);
            if (q == cudaErrorNotReady) continue;
            if (q != cudaSuccess) { (void)cudaGetLastError(); return WISV_ECUDA; }
            break;                               // stream idle: everything has been written
        }
    }
    __atomic_thread_fence(__ATOMIC_ACQUIRE);
    int32_t dev_err = 0;
    memcpy(&dev_err, pin_out, sizeof dev_err);
    if (dev_err != 0) {
        // the stream has to be idle before the counters are cleared: the round's kernels may still be retiring
        if (cudaStreamSynchronize(st) != cudaSuccess) { (void)cudaGetLastError(); return WISV_ECUDA; }
        (void)reset_after_device_error(c);
        return WISV_EDEVICE;
    }
    const uint8_t* po = pin_out + 16;
    void* dst[OUT_FIELDS] = {hr->accept_len, hr->correction_token, hr->argmax, hr->lse, hr->p_draft,
                             hr->head_prob, hr->mismatch_mask, hr->n_mismatch, hr->status};
    const size_t obytes[OUT_FIELDS] = {4u * (size_t)B, 4u * (size_t)B, 4u * (size_t)R, 4u * (size_t)R, 4u * (size_t)T,
                                       4u * (size_t)P, 8u * (size_t)B, 4u * (size_t)B, 4u * (size_t)B};
    for (int i = 0; i < OUT_FIELDS; ++i)
        if (dst[i] && obytes[i] > 0) memcpy(dst[i], po + ooff[i], obytes[i]);
    return WISV_OK;
}

}  // extern "C"
