// The small kernels around the two GEMMs:
//   pack_kernel  - rounds the fp32 hidden states to bf16 (nearest even) and builds
//                  the decision head's input rows z = [h^D ; h^T] for every evaluated
//                  position (all T in full-hidden mode, the packed list in
//                  selective-hidden mode), plus the row -> draft-token map.
//   tail_kernel  - per request: merges the LM-head partials into argmax / log-sum-exp,
//                  forms the candidate set S, finishes the head probabilities, finds
//                  the first rejected position and emits the feedback pair.
//   split_w1_kernel - one-time repack of W1 into a TMA-legal bf16 block and an fp32 CSI block.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <math_constants.h>
#include <stdint.h>

namespace wisv {

struct BatchIndex {
    int32_t B, K;               // K > 0: uniform windows; K == 0: ragged, k_off given
    const int32_t* k_off;       // [B+1] or nullptr
    __device__ __forceinline__ int koff(int b) const { return k_off ? k_off[b] : b * K; }
    __device__ __forceinline__ int roff(int b) const { return koff(b) + b; }
    // request owning token t (largest b with koff(b) <= t)
    __device__ int req_of_token(int t) const {
        if (!k_off) return K > 0 ? min(t / K, B - 1) : 0;
        int lo = 0, hi = B - 1;
        while (lo < hi) { int mid = (lo + hi + 1) >> 1; if (k_off[mid] <= t) lo = mid; else hi = mid - 1; }
        return lo;
    }
    // request owning window row r (largest b with roff(b) <= r)
    __device__ int req_of_row(int r) const {
        if (!k_off) return min(r / (K + 1), B - 1);
        int lo = 0, hi = B - 1;
        while (lo < hi) { int mid = (lo + hi + 1) >> 1; if (k_off[mid] + mid <= r) lo = mid; else hi = mid - 1; }
        return lo;
    }
};

struct PackParams {
    BatchIndex ix;
    int32_t R, P, H, H_d, V, shift, mode_sh;
    int32_t R_total, T_total;     // window rows and draft tokens of the batch (bounds for indices derived from k_off)
    int32_t vocab_base, vocab_total;   // this context's LM-head rows are tokens [vocab_base, vocab_base + V) of vocab_total
    const void* target_hidden;    // [R, H], element type th_dtype (0 fp32, 1 bf16, 2 fp16)
    const void* draft_hidden;     // [P, H_d], element type dh_dtype
    int32_t th_dtype, dh_dtype;
    const int32_t* draft_tokens;  // [T]
    const int32_t* sel_off;       // [B+1] (SH)
    const int32_t* sel_pos;       // [P]   (SH)
    __nv_bfloat16* X;             // [R, H]
    __nv_bfloat16* Z;             // [P, H_d + H]
    int32_t* row_tok;             // [R] clamped draft token or -1
    int32_t* row_flag;            // [R] WISV_ST_BAD_TOKEN or 0
    float* tok_logit;             // [R]
    int32_t* pos_req;             // [P]
    int32_t* pos_i;               // [P] window position or -1 when the list entry is invalid
};

__device__ __forceinline__ void cast_row(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, int n) {
    // n % 8 == 0; 8 floats in, one 16-byte store out; the loads of four steps are issued before the first store
    const int step = blockDim.x * 8;
    for (int i0 = threadIdx.x * 8; i0 < n; i0 += 4 * step) {
        float4 a[4], b[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = i0 + u * step;
            if (i < n) {
                a[u] = *reinterpret_cast<const float4*>(src + i);
                b[u] = *reinterpret_cast<const float4*>(src + i + 4);
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = i0 + u * step;
            if (i < n) {
                __nv_bfloat162 o[4];
                o[0] = __floats2bfloat162_rn(a[u].x, a[u].y);
                o[1] = __floats2bfloat162_rn(a[u].z, a[u].w);
                o[2] = __floats2bfloat162_rn(b[u].x, b[u].y);
                o[3] = __floats2bfloat162_rn(b[u].z, b[u].w);
                *reinterpret_cast<uint4*>(dst + i) = *reinterpret_cast<const uint4*>(o);
            }
        }
    }
}

// 16-bit sources: bf16 rows are copied, fp16 rows converted (exactly) to fp32 and rounded to bf16; 8 elements per step
__device__ __forceinline__ void copy_row_bf16(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ dst, int n) {
    for (int i = threadIdx.x * 8; i < n; i += blockDim.x * 8)
        *reinterpret_cast<uint4*>(dst + i) = *reinterpret_cast<const uint4*>(src + i);
}
__device__ __forceinline__ void cast_row_f16(const __half* __restrict__ src, __nv_bfloat16* __restrict__ dst, int n) {
    for (int i = threadIdx.x * 8; i < n; i += blockDim.x * 8) {
        const uint4 raw = *reinterpret_cast<const uint4*>(src + i);
        const __half2* h = reinterpret_cast<const __half2*>(&raw);
        __nv_bfloat162 o[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float2 f = __half22float2(h[u]);
            o[u] = __floats2bfloat162_rn(f.x, f.y);
        }
        *reinterpret_cast<uint4*>(dst + i) = *reinterpret_cast<const uint4*>(o);
    }
}
// row `row` (n elements) of a hidden-state array of the given element type -> bf16
__device__ __forceinline__ void pack_row(const void* base, int dtype, size_t row, __nv_bfloat16* dst, int n) {
    if (dtype == 0) cast_row(static_cast<const float*>(base) + row * n, dst, n);
    else if (dtype == 1) copy_row_bf16(static_cast<const __nv_bfloat16*>(base) + row * n, dst, n);
    else cast_row_f16(static_cast<const __half*>(base) + row * n, dst, n);
}

__global__ void __launch_bounds__(256) pack_kernel(const PackParams p)
{
    __shared__ int s_src_row;
    // Let the GEMM kernel that follows be scheduled at once: until its own wait it only sets up barriers and
    // tensor memory and requests weight tiles, which depend on nothing this kernel or its predecessors write.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // the previous round's kernels still read the buffers this kernel rewrites
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int blk = blockIdx.x;
    if (blk < p.R) {
        const int r = blk;
        if (threadIdx.x == 0) {
            const int b = p.ix.req_of_row(r);
            const int i = r - p.ix.roff(b);
            const int Kb = p.ix.koff(b + 1) - p.ix.koff(b);
            int tok = -1, flag = 0;
            const int t = p.ix.koff(b) + i;
            if (i >= 0 && i < Kb && t >= 0 && t < p.T_total) {       // (the last two only fail on a corrupt k_off)
                tok = p.draft_tokens[t];
                if (tok < 0 || tok >= p.vocab_total) { flag = 2; tok = tok < 0 ? 0 : p.vocab_total - 1; }
                tok -= p.vocab_base;                       // row index in this context's LM head
                if (tok < 0 || tok >= p.V) tok = -1;       // another shard owns the token
            }
            p.row_tok[r] = tok;
            p.row_flag[r] = flag;
            p.tok_logit[r] = 0.0f;
        }
        pack_row(p.target_hidden, p.th_dtype, (size_t)r, p.X + (size_t)r * p.H, p.H);
    } else {
        const int j = blk - p.R;          // evaluated position
        if (threadIdx.x == 0) {
            int b, i;
            if (p.mode_sh) {
                int lo = 0, hi = p.ix.B - 1;
                while (lo < hi) { int mid = (lo + hi + 1) >> 1; if (p.sel_off[mid] <= j) lo = mid; else hi = mid - 1; }
                b = lo;
                i = p.sel_pos[j];
            } else {
                b = p.ix.req_of_token(j);
                i = j - p.ix.koff(b);
            }
            const int Kb = p.ix.koff(b + 1) - p.ix.koff(b);
            const bool good = (i >= 0 && i < Kb);
            p.pos_req[j] = b;
            p.pos_i[j] = good ? i : -1;
            s_src_row = max(0, min(p.ix.roff(b) + (good ? i + p.shift : 0), p.R_total - 1));
        }
        __syncthreads();
        const size_t zw = (size_t)(p.H_d + p.H);
        pack_row(p.draft_hidden, p.dh_dtype, (size_t)j, p.Z + (size_t)j * zw, p.H_d);
        pack_row(p.target_hidden, p.th_dtype, (size_t)s_src_row, p.Z + (size_t)j * zw + p.H_d, p.H);
    }
}

// W1 [d_J, H_d + H + d_c] bf16 -> W1p [d_J, H_d + H] bf16 (16-byte pitch) and W1c [d_J, d_c] fp32
__global__ void split_w1_kernel(const __nv_bfloat16* __restrict__ W1, __nv_bfloat16* __restrict__ W1p,
                                float* __restrict__ W1c, int d_J, int hd_h, int d_c)
{
    const int j = blockIdx.x;
    const size_t src = (size_t)j * (hd_h + d_c);
    for (int k = threadIdx.x; k < hd_h; k += blockDim.x) W1p[(size_t)j * hd_h + k] = W1[src + k];
    for (int c = threadIdx.x; c < d_c; c += blockDim.x) W1c[(size_t)j * d_c + c] = __bfloat162float(W1[src + hd_h + c]);
}

struct TailParams {
    BatchIndex ix;
    int32_t P, V, n_tiles_lm, n_tiles_head, mode_sh, stochastic;
    int32_t T_total;              // draft tokens of the batch
    int32_t phase;                // 0: whole round; 1: localize only (no head); 2: decide from a saved localize;
                                  // 3: whole round on per-shard row partials gathered from G vocabulary shards
    int32_t vocab_base;           // added to the argidx of per-tile partials (phases 0 and 1)
    int32_t part_rstride, part_nstride;   // partial of (row r, part n) is lm_part[r * part_rstride + n * part_nstride]
    int32_t* saved_arg;           // [R] argmax per window row kept between the two phases
    unsigned long long* saved_mask;  // [B] candidate set S per request kept between the two phases
    float b2, tau;
    const float4* lm_part;        // [R][n_tiles_lm]
    const float* tok_logit;       // [R]
    const int32_t* row_flag;      // [R]
    const int32_t* draft_tokens;  // [T]
    const float* head_part;       // [P][n_tiles_head]
    const int32_t* pos_i;         // [P]
    const int32_t* sel_off;       // [B+1] (SH)
    const float* draft_q;         // [T] (stochastic)
    const float* uniforms;        // [T] (stochastic)
    int32_t* accept_len; int32_t* correction; int32_t* argmax; float* lse; float* p_draft; float* head_prob;
    unsigned long long* mismatch_mask; int32_t* n_mismatch; int32_t* status;
    const int32_t* err_src;       // device error word of the earlier kernels of this round
    int32_t* err_copy;            // if set, receives *err_src (lets a host caller read it with the results)
    // Host-buffer calls only: once every block has written its results (to device-mapped host memory) the last
    // block to finish stores done_seq to *done_flag, so the host can watch for it instead of synchronising
    // the stream.  done_count is a device counter that the last block leaves at zero.
    volatile int32_t* done_flag;
    int32_t* done_count;
    int32_t done_seq;
};

struct RowStat { float mx; int idx; float sum; };

__device__ __forceinline__ void merge_stat(RowStat& a, float mx, int idx, float sum) {
    if (mx == -CUDART_INF_F && sum == 0.0f) return;               // empty
    if (mx > a.mx) {
        a.sum = a.sum * expf(a.mx - mx) + sum;                  // exp(-inf) = 0 covers the first merge
        a.mx = mx; a.idx = idx;
    } else {
        a.sum += sum * expf(mx - a.mx);
        if (mx == a.mx && idx < a.idx) a.idx = idx;               // lowest token id wins ties
    }
}

// Latency matters here more than throughput (at batch 1 the whole kernel is a handful of dependent global
// loads): every warp takes one task at a time - a window row to merge or a head position to finish - and
// issues all the loads of the task before it uses any of them; the scan warp fetches its tokens first.
__global__ void __launch_bounds__(1024) tail_kernel(const TailParams p)
{
    constexpr int kMaxK = 64;
    __shared__ int s_arg[kMaxK + 1];
    __shared__ float s_lse[kMaxK + 1];
    __shared__ float s_tl[kMaxK + 1];            // logit of the draft token (gathered flow: from the owning shard)
    __shared__ float s_prob[kMaxK];
    __shared__ int s_has[kMaxK];
    __shared__ int s_flag;

    const int b = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;

    if (threadIdx.x < kMaxK) { s_has[threadIdx.x] = 0; s_prob[threadIdx.x] = 0.0f; }
    if (threadIdx.x == 0) s_flag = 0;
    __syncthreads();
    // The next round's pack kernel may be scheduled already; it waits for this kernel to complete before it
    // writes anything, and in turn lets the next GEMM kernel set up and prefetch weights meanwhile.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // partials of the LM-head and decision-head kernels must be complete and visible
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // A window outside 0..64 tokens, or offsets outside 0..T, can only come from a device-side k_off the host never
    // saw: the window is cut to what is in range (the scan covers at most 64 positions) and the request's status
    // word says so.
    const int k0_raw = p.ix.koff(b);
    const int k0 = max(0, min(k0_raw, p.T_total));
    const int Kb_raw = p.ix.koff(b + 1) - k0_raw;
    const int Kb = max(0, min(min(Kb_raw, kMaxK), p.T_total - k0));
    const int r0 = k0 + b;

    if (p.err_copy && b == 0 && threadIdx.x == 0) *p.err_copy = *p.err_src;

    // what the scan needs of the inputs, requested before anything else (warp 0, positions lane and lane + 32)
    int tokv[2] = {0, 0};
    float qv[2] = {1.0f, 1.0f}, uv[2] = {0.0f, 0.0f};
    if (warp == 0 && p.phase != 2) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int i = lane + 32 * h;
            if (i < Kb) {
                if (p.stochastic) { qv[h] = p.draft_q[k0 + i]; uv[h] = p.uniforms[k0 + i]; }
                else tokv[h] = p.draft_tokens[k0 + i];
            }
        }
    }

    int flag = 0;
    if (p.phase == 2) {
        // second phase: the rows were reduced by the localize call
        for (int i = threadIdx.x; i <= Kb; i += blockDim.x) { s_arg[i] = p.saved_arg[r0 + i]; flag |= p.row_flag[r0 + i]; }
    }
    const int row_tasks = p.phase == 2 ? 0 : Kb + 1;
    int e0, e1;
    if (p.phase == 1) { e0 = 0; e1 = 0; }
    else if (p.mode_sh) { e0 = max(p.sel_off[b], 0); e1 = min(p.sel_off[b + 1], p.P); } else { e0 = k0; e1 = k0 + Kb; }
    const int pos_tasks = e1 > e0 ? e1 - e0 : 0;

    for (int task = warp; task < row_tasks + pos_tasks; task += nwarps) {
        if (task < row_tasks) {
            // ---- merge the (max, argidx, sumexp) partials of one window row: one per vocabulary tile or CTA,
            //      or per shard {max, global argidx, sumexp, draft-token logit or -inf} in the gathered flow
            const int i = task;
            const int r = r0 + i;
            float tlg = 0.0f;
            int rf = 0;
            if (lane == 0) {
                rf = p.row_flag[r];
                if (p.phase != 3) tlg = p.tok_logit[r];
            }
            RowStat st{-CUDART_INF_F, 0x7fffffff, 0.0f};
            float tl = -CUDART_INF_F;
            const float4* part = p.lm_part + (size_t)r * p.part_rstride;
            for (int base = 0; base < p.n_tiles_lm; base += 256) {
                float4 v[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int n = base + j * 32 + lane;
                    v[j] = n < p.n_tiles_lm ? part[(size_t)n * p.part_nstride]
                                            : make_float4(-CUDART_INF_F, 0.0f, 0.0f, -CUDART_INF_F);
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    merge_stat(st, v[j].x, __float_as_int(v[j].y), v[j].z);
                    tl = fmaxf(tl, v[j].w);
                }
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                const float omx = __shfl_xor_sync(0xffffffffu, st.mx, off);
                const int oidx = __shfl_xor_sync(0xffffffffu, st.idx, off);
                const float osum = __shfl_xor_sync(0xffffffffu, st.sum, off);
                merge_stat(st, omx, oidx, osum);
                tl = fmaxf(tl, __shfl_xor_sync(0xffffffffu, tl, off));
            }
            const float l = st.mx + logf(st.sum);
            if (p.phase != 3) st.idx += p.vocab_base;
            if (lane == 0) {
                s_arg[i] = st.idx;
                s_lse[i] = l;
                s_tl[i] = p.phase == 3 ? tl : tlg;
                if (p.phase == 1) p.saved_arg[r] = st.idx;
                if (p.argmax) p.argmax[r] = st.idx;
                if (p.lse) p.lse[r] = l;
                if (!isfinite(l)) flag |= 4;
                flag |= rf;
            }
        } else {
            // ---- finish the decision head of one position: s = b2 + sum of the partial dot products
            const int e = e0 + (task - row_tasks);
            int pi = 0;
            if (lane == 0) pi = p.pos_i[e];
            float s = 0.0f;
            const float* hp = p.head_part + (size_t)e * p.n_tiles_head;
            for (int base = 0; base < p.n_tiles_head; base += 128) {
                float x[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int n = base + j * 32 + lane;
                    x[j] = n < p.n_tiles_head ? hp[n] : 0.0f;
                }
                s += (x[0] + x[1]) + (x[2] + x[3]);
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
            s += p.b2;
            const float prob = 1.0f / (1.0f + expf(-s));
            if (lane == 0) {
                if (p.head_prob) p.head_prob[e] = prob;
                if (pi >= 0 && pi < Kb) { s_prob[pi] = prob; s_has[pi] = 1; } else { flag |= 8; }
                if (!isfinite(s)) flag |= 4;
            }
        }
    }
    if (flag) atomicOr(&s_flag, flag);
    __syncthreads();

    // ---- Localize, first-reject scan, emission (one warp; windows hold at most 64 tokens)
    if (warp == 0) {
        unsigned cand_bits[2], rej_bits[2];
        int missing = 0;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int i = lane + 32 * h;
            bool cand = false, rej = false;
            if (i < Kb) {
                const int t = k0 + i;
                if (p.phase == 2) {
                    cand = (p.saved_mask[b] >> i) & 1ull;
                } else {
                    const float pd = expf(s_tl[i] - s_lse[i]);
                    if (p.p_draft) p.p_draft[t] = pd;
                    if (p.stochastic) {
                        const float alpha = fminf(1.0f, pd / qv[h]);
                        cand = !(uv[h] < alpha);
                    } else {
                        cand = tokv[h] != s_arg[i];
                    }
                }
                const bool has = s_has[i] != 0;
                rej = cand && (!has || s_prob[i] >= p.tau);      // localize phase: no uploads yet, greedy
                if (cand && !has && p.phase != 1) missing = 1;
            }
            cand_bits[h] = __ballot_sync(0xffffffffu, cand);
            rej_bits[h] = __ballot_sync(0xffffffffu, rej);
        }
        missing = __any_sync(0xffffffffu, missing);
        if (lane == 0) {
            const unsigned long long rej = (unsigned long long)rej_bits[0] | ((unsigned long long)rej_bits[1] << 32);
            const unsigned long long cnd = (unsigned long long)cand_bits[0] | ((unsigned long long)cand_bits[1] << 32);
            const int A = rej ? (__ffsll((long long)rej) - 1) : Kb;
            if (p.accept_len) p.accept_len[b] = A;
            if (p.correction) p.correction[b] = s_arg[A];
            if (p.phase == 1) p.saved_mask[b] = cnd;
            if (p.mismatch_mask) p.mismatch_mask[b] = cnd;
            if (p.n_mismatch) p.n_mismatch[b] = __popcll(cnd);
            if (p.status) p.status[b] = s_flag | (missing ? 1 : 0) | ((Kb != Kb_raw || k0 != k0_raw) ? 16 : 0);
        }
    }
    if (p.done_flag) {
        __threadfence_system();                  // this thread's results before the flag, as the host sees them
        __syncthreads();
        if (threadIdx.x == 0) {
            const int old = atomicAdd(p.done_count, 1);
            if (old == static_cast<int>(gridDim.x) - 1) {
                *p.done_count = 0;
                __threadfence_system();
                *p.done_flag = p.done_seq;
            }
        }
    }
}

}  // namespace wisv

namespace wisv {

// Vocabulary-sharded LM head: reduce the per-tile partials of this shard to one partial per window row,
// {max, global argidx, sumexp, logit of the draft token if this shard owns it else -inf}.
__global__ void __launch_bounds__(128) shard_rows_kernel(const float4* __restrict__ lm_part, int n_parts, int R,
                                                         int vocab_base, const int32_t* __restrict__ row_tok,
                                                         const float* __restrict__ tok_logit, float4* __restrict__ out)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (r >= R) return;
    RowStat st{-CUDART_INF_F, 0x7fffffff, 0.0f};
    for (int n = lane; n < n_parts; n += 32) {
        const float4 v = lm_part[(size_t)r * n_parts + n];
        merge_stat(st, v.x, __float_as_int(v.y), v.z);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float omx = __shfl_xor_sync(0xffffffffu, st.mx, off);
        const int oidx = __shfl_xor_sync(0xffffffffu, st.idx, off);
        const float osum = __shfl_xor_sync(0xffffffffu, st.sum, off);
        merge_stat(st, omx, oidx, osum);
    }
    if (lane == 0)
        out[r] = make_float4(st.mx, __int_as_float(st.idx + vocab_base), st.sum,
                             row_tok[r] >= 0 ? tok_logit[r] : -CUDART_INF_F);
}

}  // namespace wisv
