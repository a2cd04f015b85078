// Kernels and entry points of libpcg: PCG group-level verification on sm_100a.
//
//   position_kernel  one thread block per drafted position (b,i).  Streams the target row, then the draft row
//                    (softmax statistics with a lazy reference, 128-bit loads), draws the group label of the draft
//                    token, forms the label group's target and draft mass from a handful of gathered logits and
//                    takes the accept decision.  This kernel moves ~all of the bytes.
// The per-sequence stage of pcg_verify (first rejection, residual (P-Q)_+ of ALL groups at that position, group
// draw, token draw, outputs) exists in two forms:
//   terminal_kernel  one thread-block cluster per sequence: a token-sliced segmented reduction in shared memory,
//                    slices combined over distributed shared memory (a handful of sequences: lowest latency).
//   batched          residual_transpose_kernel (which also finds the first rejections), group_spmm_kernel,
//                    terminal_pick_kernel: the residual of all sequences as one sparse product over a transposed,
//                    L2-resident operand.
// pcg_group_probs writes P of every row with the same two aggregations; dense mode of pcg_verify stores P and Q of
// every position that way and draws with terminal_prepare_kernel / terminal_draw_kernel; pcg_verify_thinning
// replaces the per-sequence stage by thinning_kernel (pcg_thinning.cuh), which enumerates nothing.  Every kernel
// after the first of a call is launched with programmatic stream serialisation (pdl_enter, launch_after).
#include <cooperative_groups.h>

#include <algorithm>
#include <atomic>
#include <cmath>
#include <mutex>

#include "pcg_common.cuh"

namespace cg = cooperative_groups;


namespace pcg {

constexpr float kLog2e = 1.4426950408889634f;
constexpr size_t kMaxDynSmem = 227 * 1024;  // dynamic shared memory a block may opt in to

// ================================================================ position kernel ==========================
//
// Per row the kernel needs Z = sum_t 2^(l_t*s - RS) for SOME reference RS: any value works as long as the same
// RS is used for the group masses, because it cancels in P = S/Z.  So no running maximum is kept.  Each thread
// holds a reference rs; it adds the terms of a 16-byte vector relative to rs and only then looks at their
// sum: a sum above 2^32 (or an overflow to +inf) means some logit sits far above the reference, and the thread
// redoes that one vector after raising rs to the vector's maximum (rescaling what it has summed so far).
// That happens on a thread's first vector and practically never again, so the fast path costs exactly one
// ex2 per logit and no max instructions.  Terms therefore stay below 2^32 and Z below V * 2^32.
//
// A block handles one drafted position: all its threads stream the target row, then the draft row (one long
// contiguous run per block: measured 5 % faster than two half-blocks on a row each), with 128-bit loads issued
// one batch (kBatch vectors per thread) ahead of the arithmetic and the draft row's first batch issued before the
// target row is reduced.  The chain of dependent loads that leads from the draft token to the label group's
// logits (token -> its groups -> label -> group's token list -> logits) is spread over the streaming loop, one hop
// per batch, so its latency is hidden.

constexpr int kPosThreads = 256;       // threads of a position block for long rows ...
constexpr int kPosThreadsSmall = 128;  // ... and for rows of at most kPosSmallRowBytes (more batches per row, more blocks per SM)
constexpr size_t kPosSmallRowBytes = 64 * 1024;
constexpr int kBatch = 4;
constexpr float kRefInit = -1.0e30f;     // "no logit seen yet": finite, so that -inf logits give 2^-inf = 0, not NaN
constexpr float kVecSumLimit = 4294967296.f;  // 2^32
constexpr float kRunSumLimit = 1.8446744e19f;  // 2^64: a thread's unchecked running sum beyond it is formed again, checked

struct RefSum {
    float rs;   // scaled reference: the exponent subtracted from l*s
    float acc;  // sum of 2^(l*s - rs)
};

template <int NV>
__device__ __forceinline__ void absorb_slow(RefSum &st, const float (&v)[NV], float s) {
    float vm = v[0];
#pragma unroll
    for (int i = 1; i < NV; ++i) vm = fmaxf(vm, v[i]);
    if (vm > kNegInf) {  // (a vector of -inf only adds zeros and cannot get here)
        const float nrs = vm * s;
        st.acc *= ex2(st.rs - nrs);
        st.rs = nrs;
    }
    float vs = 0.f;
#pragma unroll
    for (int i = 0; i < NV; ++i) vs += ex2(__fmaf_rn(v[i], s, -st.rs));
    st.acc += vs;
}

template <int NV>
__device__ __forceinline__ void absorb(RefSum &st, const float (&v)[NV], float s) {
    float vs = 0.f;
#pragma unroll
    for (int i = 0; i < NV; ++i) vs += ex2(__fmaf_rn(v[i], s, -st.rs));
    if (vs <= kVecSumLimit)
        st.acc += vs;
    else  // reference too low for this vector (always so for a thread's first vector): raise it and redo
        absorb_slow<NV>(st, v, s);
}

// The same without the check: the sum is added as it is.  A vector far above the reference makes the running sum
// huge, infinite or NaN, and it stays so: the caller tests the sum once per row (kRunSumLimit) and, if it left the
// safe range, forms the thread's sum again with absorb.  A sum that is large but inside the range is as exact as any
// other (floating point); the limit keeps the 256 threads' sums of a row from overflowing when they are merged.
template <int NV>
__device__ __forceinline__ void absorb_unchecked(RefSum &st, const float (&v)[NV], float s) {
    float vs = 0.f;
#pragma unroll
    for (int i = 0; i < NV; ++i) vs += ex2(__fmaf_rn(v[i], s, -st.rs));
    st.acc += vs;
}

__device__ __forceinline__ void absorb1(RefSum &st, float l, float s) {
    const float v[1] = {l};
    absorb<1>(st, v, s);
}

__device__ __forceinline__ void merge(float &rs, float &acc, float rs2, float acc2) {
    const float m = fmaxf(rs, rs2);
    acc = acc * ex2(rs - m) + acc2 * ex2(rs2 - m);
    rs = m;
}

struct PositionArgs {
    const void *target;      // [B, K+1, V]
    const void *draft;       // [B, K, V]
    const int32_t *draft_tokens;  // [B, K]
    const float *uniforms;   // [B, K+1, 2]
    int K;
    float s;                 // log2(e) / temperature
    float bias;              // constant added to the acceptance ratio (0 for PCG)
    int32_t *accept;         // [B*K] 1 = accepted
    int32_t *labels;         // [B*K] group label of the draft token
    int32_t *posflags;       // [B*K]
    float4 *stats;           // [B*K] (RS_p, 1/Z_p, RS_q, 1/Z_q): scaled reference and reciprocal normaliser
    float2 *strata;          // [B*K, NT] or null: every thread's own (reference, sum) of the target row; thread h of the
                             // block's NT has summed its 16-byte words h, h + NT, h + 2 NT, ... (see pcg_thinning.cuh)
    float4 *bonus_stats;     // [B] or null: (RS, 1/Z, 0, 0) of the bonus row (target row K), written by the block of a
                             // sequence's LAST drafted position if that position was accepted (no sequence that
                             // needs its bonus row can have its last position rejected)
    int32_t *bonus_flags;    // [B] flags of that row (with bonus_stats)
    int32_t *zero_words;     // counters of a later kernel of the call that must start at zero (block 0 clears them), or null
    int zero_count;          // how many
};

// Group-label coupling: the label of draft token x is drawn from the groups containing x (reverse membership
// entries [r0, r0+n), ascending group id) -- uniformly for the equal split, by inverse CDF over w_{.,x} otherwise.
__device__ __forceinline__ int draw_label(const GroupsDev &G, int r0, int n, float u0) {
    int j;
    if (!G.rev_w) {
        j = (int)floor((double)u0 * (double)n);  // exact: float times small integer in double
        j = min(max(j, 0), n - 1);
    } else {
        double tot = 0.0, run = 0.0;
        for (int e = 0; e < n; ++e) tot += (double)G.rev_w[r0 + e];
        const double target = (double)u0 * tot;
        j = -1;
        int last_pos = 0;
        for (int e = 0; e < n; ++e) {
            const double w = (double)G.rev_w[r0 + e];
            if (w > 0.0) last_pos = e;
            run += w;
            if (run > target) {
                j = e;
                break;
            }
        }
        if (j < 0) j = last_pos;
    }
    return G.rev_grp[r0 + j];
}

// Softmax statistics of one row by the whole block (the bonus row of a sequence whose last drafted position was
// accepted).  Kept out of line so that the streaming loop of the position kernel keeps its registers.
template <typename T, int NT>
__device__ __noinline__ void bonus_row_stats(const T *row, int V, float s, float *red, float4 *stats_out, int32_t *flags_out) {
    constexpr int NW = NT / 32, NV = Elem<T>::kPerVec;
    const int tid = threadIdx.x;
    RefSum st{kRefInit * s, 0.f};
    int head = (int)(((16u - (unsigned)((uintptr_t)row & 15u)) & 15u) / sizeof(T));
    if (head > V) head = V;
    const int nvec = (V - head) / NV;
    const uint4 *vp = reinterpret_cast<const uint4 *>(row + head);
    int idx = tid;
    for (; idx + 3 * NT < nvec; idx += 4 * NT) {
        uint4 r[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) r[j] = ld_stream(vp + idx + j * NT);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float v[NV];
            Elem<T>::unpack(r[j], v);
            absorb<NV>(st, v, s);
        }
    }
    for (; idx < nvec; idx += NT) {
        float v[NV];
        Elem<T>::unpack(ld_stream(vp + idx), v);
        absorb<NV>(st, v, s);
    }
    for (int t = tid; t < head; t += NT) absorb1(st, Elem<T>::widen(row[t]), s);
    for (int t = head + nvec * NV + tid; t < V; t += NT) absorb1(st, Elem<T>::widen(row[t]), s);
    float rs = st.rs, Z = st.acc;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) merge(rs, Z, __shfl_xor_sync(0xffffffffu, rs, o), __shfl_xor_sync(0xffffffffu, Z, o));
    if ((tid & 31) == 0) {
        red[2 * (tid >> 5)] = rs;
        red[2 * (tid >> 5) + 1] = Z;
    }
    __syncthreads();
    if (tid == 0) {
        rs = red[0];
        Z = red[1];
        for (int w = 1; w < NW; ++w) merge(rs, Z, red[2 * w], red[2 * w + 1]);
        *stats_out = make_float4(rs, 1.0f / Z, 0.f, 0.f);
        *flags_out = (!(Z > 0.f) || isinf(Z) || isinf(rs)) ? PCG_FLAG_NONFINITE : 0;
    }
}

template <typename T, int NT>
__global__ void __launch_bounds__(NT, 1024 / NT) position_kernel(PositionArgs a, GroupsDev G) {
    constexpr int NW = NT / 32;
    constexpr int NV = Elem<T>::kPerVec;
    constexpr int U = kBatch;
    constexpr int kChainSteps = 6;
    __shared__ float red_z[4 * NW];
    __shared__ float red_s[1];
    const int tid = threadIdx.x;
    const int V = G.V, K = a.K;
    const float s = a.s;
    // Block order: the LAST drafted position of every sequence first (blocks 0 .. B-1), then the others.  Those
    // blocks may have a third row to stream (the bonus row, see PositionArgs::bonus_stats); up front that extra
    // work is spread over the first wave instead of lengthening the tail of the kernel.
    // (Without bonus rows -- the cluster terminal and the thinning entry point fetch them themselves -- the blocks
    // simply follow the positions: measured 3 us faster at B = 256, K = 16, V = 65536.)
    const int nseq = (int)gridDim.x / K;
    int b, i;
    if (a.bonus_stats) {
        b = (int)blockIdx.x < nseq ? (int)blockIdx.x : ((int)blockIdx.x - nseq) / (K - 1);
        i = (int)blockIdx.x < nseq ? K - 1 : ((int)blockIdx.x - nseq) - b * (K - 1);
    } else {
        b = (int)blockIdx.x / K;
        i = (int)blockIdx.x - b * K;
    }
    const int pos = b * K + i;
    pdl_enter();  // (the first kernel of a call: lets the kernel behind it be scheduled while this one drains)
    if (a.zero_words && blockIdx.x == 0)  // (this grid completes before their user starts)
        for (int k = tid; k < a.zero_count; k += NT) a.zero_words[k] = 0;
    const T *trow = reinterpret_cast<const T *>(a.target) + ((int64_t)b * (K + 1) + i) * V;
    const T *qrow = reinterpret_cast<const T *>(a.draft) + (int64_t)pos * V;
    const float *u = a.uniforms + ((int64_t)b * (K + 1) + i) * 2;
    const uint64_t pol = l2_evict_first_policy();

    // ---- dependent-load chain towards the label group's logits: WARP 0 only (lane k takes the group's k-th token;
    // the other warps' streaming loops stay free of it) ----
    const bool chain_warp = tid < 32;
    int c_x = 0, c_r0 = 0, c_n = 1, c_g = 0, c_lo = 0, c_hi = 0, c_t = 0, c_flag = 0;
    float c_u0 = 0.f, c_u1 = 0.f, c_lp = kNegInf, c_lq = kNegInf, c_w = 0.f;
    auto chain = [&](int step) {
        switch (step) {
            case 0:
                c_x = a.draft_tokens[pos];
                c_u0 = u[0];
                c_u1 = u[1];
                break;
            case 1:
                if (c_x < 0 || c_x >= V) {
                    c_x = 0;
                    c_flag = PCG_FLAG_BAD_DRAFT_TOKEN;
                }
                c_r0 = G.rev_ptr[c_x];
                c_n = G.rev_ptr[c_x + 1] - c_r0;
                break;
            case 2:
                c_g = draw_label(G, c_r0, c_n, c_u0);
                break;
            case 3:
                c_lo = G.group_ptr[c_g];
                c_hi = G.group_ptr[c_g + 1];
                break;
            case 4:
                if (c_lo + tid < c_hi) c_t = G.group_tok[c_lo + tid];
                break;
            case 5:
                if (c_lo + tid < c_hi) {
                    c_lp = Elem<T>::widen(trow[c_t]);
                    c_lq = Elem<T>::widen(qrow[c_t]);
                    c_w = G.pair_w ? G.pair_w[c_lo + tid] : G.inv_deg[c_t];
                }
                break;
        }
    };
    int chained = 0;

    // The whole block streams the target row, then the draft row: thread h takes the 16-byte words h, h + 256, ...
    // of a row, U of them in flight.  A row = elements before the first 16-byte boundary, whole vectors, the rest.
    uint4 cur[U];
    auto plan_head = [&](const T *row) {
        const int head = (int)(((16u - (unsigned)((uintptr_t)row & 15u)) & 15u) / sizeof(T));
        return head > V ? V : head;
    };
    auto first_batch = [&](const T *row) {  // the first U vectors of this thread, if the row has a full batch
        const int head = plan_head(row);
        if ((V - head) / NV / (NT * U) > 0) {
            const uint4 *p = reinterpret_cast<const uint4 *>(row + head) + tid;
#pragma unroll
            for (int j = 0; j < U; ++j) cur[j] = ld_stream(p + j * NT, pol);
        }
    };
    auto stream_row = [&](const T *row, RefSum &st) {  // `cur` holds the first batch on entry
        const int head = plan_head(row);
        const int nvec = (V - head) / NV;
        const int nfull = nvec / (NT * U);  // batches in which every thread has all U vectors
        const uint4 *p = reinterpret_cast<const uint4 *>(row + head) + tid;
        uint4 nxt[U];
        // The reference of a thread is set by its first vector (as the checked form does when that vector's sum
        // overflows against the initial reference); the batches are then summed without a branch per vector: the
        // branch kept the exponentials of one vector from overlapping the next one's (4 us of the kernel at
        // B = 256, K = 16, V = 65536).
        if (nfull > 0) {
            float v[NV];
            Elem<T>::unpack(cur[0], v);
            float vm = v[0];
#pragma unroll
            for (int i = 1; i < NV; ++i) vm = fmaxf(vm, v[i]);
            if (vm > kNegInf) st.rs = vm * s;
        }
        // the batches during which the chain advances, then the rest in a loop of their own, free of the chain's test
        // and dispatch (1.6 us of the kernel at B = 256, K = 16, V = 65536)
        const int nchain = min(nfull, kChainSteps - min(chained, kChainSteps));
        int bi = 0;
        for (; bi < nchain; ++bi) {
            p += NT * U;
            if (bi + 1 < nfull) {  // (making these loads unconditional as in the second loop costs registers: spills)
#pragma unroll
                for (int j = 0; j < U; ++j) nxt[j] = ld_stream(p + j * NT, pol);
            }
            if (chain_warp) chain(chained);
            ++chained;
#pragma unroll
            for (int j = 0; j < U; ++j) {
                float v[NV];
                Elem<T>::unpack(cur[j], v);
                absorb_unchecked<NV>(st, v, s);
            }
#pragma unroll
            for (int j = 0; j < U; ++j) cur[j] = nxt[j];
        }
        for (; bi + 1 < nfull; ++bi) {  // every batch but the last: the next one's loads go out unconditionally
            p += NT * U;
#pragma unroll
            for (int j = 0; j < U; ++j) nxt[j] = ld_stream(p + j * NT, pol);
#pragma unroll
            for (int j = 0; j < U; ++j) {
                float v[NV];
                Elem<T>::unpack(cur[j], v);
                absorb_unchecked<NV>(st, v, s);
            }
#pragma unroll
            for (int j = 0; j < U; ++j) cur[j] = nxt[j];
        }
        if (bi < nfull) {  // the last batch
#pragma unroll
            for (int j = 0; j < U; ++j) {
                float v[NV];
                Elem<T>::unpack(cur[j], v);
                absorb_unchecked<NV>(st, v, s);
            }
        }
        if (!(st.acc <= kRunSumLimit)) {  // (rare: a later vector far above the thread's reference, or NaN) this thread's vectors again, checked
            st = RefSum{kRefInit * s, 0.f};
            const uint4 *vp = reinterpret_cast<const uint4 *>(row + head) + tid;
#pragma unroll 1
            for (int k = 0; k < nfull * U; ++k) {  // (not unrolled, and not a call: either cost the loop above registers)
                float v[NV];
                Elem<T>::unpack(ld_stream(vp + (size_t)k * NT), v);
                absorb<NV>(st, v, s);
            }
        }
        // remaining whole vectors (fewer than NT*U), then the scalar head and tail
        for (int idx = nfull * NT * U + tid; idx < nvec; idx += NT) {
            float v[NV];
            Elem<T>::unpack(ld_stream(reinterpret_cast<const uint4 *>(row + head) + idx), v);
            absorb<NV>(st, v, s);
        }
        for (int t = tid; t < head; t += NT) absorb1(st, Elem<T>::widen(row[t]), s);
        for (int t = head + nvec * NV + tid; t < V; t += NT) absorb1(st, Elem<T>::widen(row[t]), s);
    };
    // (rs, Z) of a row from the threads' pairs: xor butterfly inside a warp, then a fixed-order pass over the warps
    auto reduce_row = [&](const RefSum &st, float *red, float &rs_out, float &Z_out) {
        float rs = st.rs, Z = st.acc;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) merge(rs, Z, __shfl_xor_sync(0xffffffffu, rs, o), __shfl_xor_sync(0xffffffffu, Z, o));
        if ((tid & 31) == 0) {
            red[2 * (tid >> 5)] = rs;
            red[2 * (tid >> 5) + 1] = Z;
        }
        __syncthreads();
        rs = red[0], Z = red[1];
#pragma unroll
        for (int w = 1; w < NW; ++w) merge(rs, Z, red[2 * w], red[2 * w + 1]);
        rs_out = rs, Z_out = Z;
    };

    first_batch(trow);
    RefSum st{kRefInit * s, 0.f};
    stream_row(trow, st);
    if (a.strata) a.strata[(size_t)pos * NT + tid] = make_float2(st.rs, st.acc);  // a free by-product
    first_batch(qrow);  // the draft row's first loads go out before the target row's reduction
    float rs_p, Zp, rs_q, Zq;
    reduce_row(st, red_z, rs_p, Zp);
    st = RefSum{kRefInit * s, 0.f};
    stream_row(qrow, st);
    if (chain_warp)
        while (chained < kChainSteps) chain(chained++);
    reduce_row(st, red_z + 2 * NW, rs_q, Zq);

    // ---- masses of the label group under the two rows, by warp 0 (the first 32 tokens were prefetched by the
    // chain), then the accept test ----
    if (chain_warp) {
        float part_p = __fmul_rn(ex2(__fmaf_rn(c_lp, s, -rs_p)), c_w);
        float part_q = __fmul_rn(ex2(__fmaf_rn(c_lq, s, -rs_q)), c_w);
        for (int k = c_lo + tid + 32; k < c_hi; k += 32) {  // groups of more than 32 tokens
            const int t = G.group_tok[k];
            const float w = G.pair_w ? G.pair_w[k] : G.inv_deg[t];
            part_p += __fmul_rn(ex2(__fmaf_rn(Elem<T>::widen(trow[t]), s, -rs_p)), w);
            part_q += __fmul_rn(ex2(__fmaf_rn(Elem<T>::widen(qrow[t]), s, -rs_q)), w);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            part_p += __shfl_xor_sync(0xffffffffu, part_p, o);
            part_q += __shfl_xor_sync(0xffffffffu, part_q, o);
        }
        if (tid == 0) {
            const float Sp = part_p, Sq = part_q;
            // acceptance u < min(1, P/Q) without a division: P = Sp/Zp, Q = Sq/Zq
            const float lhs = Sp * Zq, rhs = Sq * Zp;
            const int acc = (lhs >= rhs) || (c_u1 * rhs < __fmaf_rn(a.bias, rhs, lhs));
            int flag = c_flag;
            if (!(Zp > 0.f) || !(Zq > 0.f) || isinf(Zp) || isinf(Zq) || isinf(rs_p) || isinf(rs_q))
                flag |= PCG_FLAG_NONFINITE;
            a.accept[pos] = acc;
            a.labels[pos] = c_g;
            a.posflags[pos] = flag;
            a.stats[pos] = make_float4(rs_p, 1.0f / Zp, rs_q, 1.0f / Zq);
            red_s[0] = acc ? 1.f : 0.f;
        }
    }
    if (a.bonus_stats && i == K - 1) {  // block-uniform: the last drafted position of its sequence
        __syncthreads();
        if (red_s[0] != 0.f)  // accepted: the sequence may need its bonus row
            bonus_row_stats<T, NT>(reinterpret_cast<const T *>(a.target) + ((int64_t)b * (K + 1) + K) * V, V, s, red_z,
                               a.bonus_stats + b, a.bonus_flags + b);
    }
}

// ================================================================ token-sliced aggregation ==================
//
// A cluster of C thread blocks handles one row (or one sequence).  Block c owns the token slice
// [c*SL, (c+1)*SL): it holds one float per token of the slice in shared memory, sweeps the slice's part of
// every group (16-bit in-slice offsets, ordered by group) into partial[g], and after a cluster barrier the
// blocks add the C partial sums of "their" M/C groups in a fixed order through distributed shared memory.

struct AggSmem {
    float *d;          // [SL]  per-token value of this slice
    float *partial;    // [M]   this slice's share of every group
    float *own;        // [Mc]  totals of the groups this block owns
    float *scratch;    // reductions
    double *dscratch;  // scans
    double *xchg;      // values other blocks of the cluster read: [0] block total, [1] slice max
    int *ibox;         // block-wide integers
};

__device__ __forceinline__ AggSmem carve_smem(unsigned char *raw, const GroupsDev &G) {
    AggSmem sm;
    sm.d = reinterpret_cast<float *>(raw);
    sm.partial = sm.d + G.slice_len + 32;  // d[slice_len] is the always-zero slot of padding entries
    sm.own = sm.partial + G.M;
    unsigned char *tail = reinterpret_cast<unsigned char *>(sm.own + G.groups_per_slice);
    tail = reinterpret_cast<unsigned char *>(((uintptr_t)tail + 15) & ~(uintptr_t)15);
    sm.dscratch = reinterpret_cast<double *>(tail);                    // 32 doubles
    sm.xchg = sm.dscratch + 32;                                        // 4 doubles
    sm.scratch = reinterpret_cast<float *>(sm.xchg + 4);               // 64 floats
    sm.ibox = reinterpret_cast<int *>(sm.scratch + 64);                // 8 ints
    return sm;
}

// Copy this block's slice of a row into shared memory as floats; returns the block-wide maximum.
template <typename T, int NT>
__device__ __forceinline__ float load_slice_max(const T *__restrict__ row, int n, float *d, float *scratch) {
    constexpr int NV = Elem<T>::kPerVec;
    float vm = kNegInf;
    if (n > 0 && ((uintptr_t)row & 15u) == 0) {
        const int nvec = n / NV;
        const uint4 *vp = reinterpret_cast<const uint4 *>(row);
        for (int idx = threadIdx.x; idx < nvec; idx += NT) {
            float v[NV];
            Elem<T>::unpack(ld_stream(vp + idx), v);
#pragma unroll
            for (int e = 0; e < NV; ++e) {
                d[idx * NV + e] = v[e];
                vm = fmaxf(vm, v[e]);
            }
        }
        for (int t = nvec * NV + threadIdx.x; t < n; t += NT) {
            const float l = Elem<T>::widen(row[t]);
            d[t] = l;
            vm = fmaxf(vm, l);
        }
    } else {
        for (int t = threadIdx.x; t < n; t += NT) {
            const float l = Elem<T>::widen(row[t]);
            d[t] = l;
            vm = fmaxf(vm, l);
        }
    }
    return block_max<NT>(vm, scratch);
}

// Segmented reduction of the slice: partial[g] = sum over the slice's tokens of group g of d[t] (* w).
// Thread t walks column t of the slice's entry rows (coalesced 32-bit loads, kept several rows ahead in
// registers), adds d[token] into a register while the group id stays the same and stores the sum when it
// changes; a group's entries never span two threads, so every partial[g] has exactly one writer and a fixed
// summation order.  partial[] must be zero-filled and d[slice_len] must be 0 before the call.
template <int NT>
__device__ __forceinline__ void sweep_slice(const GroupsDev &G, int c, const float *d, float *partial) {
    constexpr int R = 8;  // rows in flight per thread
    const int begin = G.ent_off[c], rows = (G.ent_off[c + 1] - begin) / NT;
    const uint32_t *ep = G.ent + begin + threadIdx.x;
    const float *wp = G.ent_w ? G.ent_w + begin + threadIdx.x : nullptr;
    uint32_t cur = kNoGroup;
    float acc = 0.f;
    for (int r0 = 0; r0 < rows; r0 += R) {
        uint32_t e[R];
        float w[R];
#pragma unroll
        for (int j = 0; j < R; ++j) {
            const bool in = r0 + j < rows;
            e[j] = in ? ep[(size_t)(r0 + j) * NT] : 0u;
            w[j] = (wp && in) ? wp[(size_t)(r0 + j) * NT] : 1.f;
        }
#pragma unroll
        for (int j = 0; j < R; ++j) {
            if (r0 + j < rows) {
                const uint32_t g = e[j] >> 16;
                if (g != cur) {
                    if (cur != kNoGroup) partial[cur] = acc;
                    cur = g;
                    acc = 0.f;
                }
                const float v = d[e[j] & 0xffffu];
                acc += wp ? __fmul_rn(v, w[j]) : v;
            }
        }
    }
    if (cur != kNoGroup) partial[cur] = acc;
}

// Zero partial[0..M) and the always-zero slot d[slice_len] (block-wide; followed by a barrier at the caller).
template <int NT>
__device__ __forceinline__ void clear_partial(const GroupsDev &G, float *d, float *partial) {
    for (int g = threadIdx.x; g < G.M; g += NT) partial[g] = 0.f;
    if (threadIdx.x == 0) d[G.slice_len] = 0.f;
}

// ---------------------------------------------------------------- pcg_group_probs ----------------------------
struct ProbsArgs {
    const void *logits;  // [rows, V]
    float *out;          // [rows, M]
    float s;
};

template <typename T>
__global__ void __launch_bounds__(kAggThreads, 2) group_probs_kernel(ProbsArgs a, GroupsDev G) {
    pdl_enter();
    constexpr int NT = kAggThreads;
    extern __shared__ __align__(16) unsigned char raw[];
    AggSmem sm = carve_smem(raw, G);
    cg::cluster_group cluster = cg::this_cluster();
    const int C = G.slices;
    const int c = (int)cluster.block_rank();
    const int64_t row = blockIdx.x / C;
    const int t0 = c * G.slice_len;
    const int n = max(0, min(G.slice_len, G.V - t0));
    const T *rp = reinterpret_cast<const T *>(a.logits) + row * G.V + t0;

    // softmax terms of the slice relative to the row maximum (exchanged across the cluster)
    clear_partial<NT>(G, sm.d, sm.partial);
    const float mloc = load_slice_max<T, NT>(rp, n, sm.d, sm.scratch);
    if (threadIdx.x == 0) sm.xchg[1] = (double)mloc;
    cluster.sync();
    float m = kNegInf;
    for (int r = 0; r < C; ++r) m = fmaxf(m, (float)*cluster.map_shared_rank(&sm.xchg[1], r));
    float zloc = 0.f;
    const float rs = m * a.s;
    for (int t = threadIdx.x; t < n; t += NT) {
        const float e = ex2(__fmaf_rn(sm.d[t], a.s, -rs));
        zloc += e;
        sm.d[t] = G.ent_w ? e : __fmul_rn(e, G.inv_deg[t0 + t]);
    }
    const float zc = block_sum<NT>(zloc, sm.scratch);  // contains the barrier that publishes d
    if (threadIdx.x == 0) sm.xchg[0] = (double)zc;
    sweep_slice<NT>(G, c, sm.d, sm.partial);
    cluster.sync();
    float Z = 0.f;
    for (int r = 0; r < C; ++r) Z += (float)*cluster.map_shared_rank(&sm.xchg[0], r);
    const int g0 = c * G.groups_per_slice, g1 = min(G.M, g0 + G.groups_per_slice);
    for (int g = g0 + (int)threadIdx.x; g < g1; g += NT) {
        float tot = 0.f;
        for (int r = 0; r < C; ++r) tot += cluster.map_shared_rank(sm.partial, r)[g];
        a.out[row * G.M + g] = tot / Z;
    }
    cluster.sync();  // no block may exit while another still reads its shared memory
}

// ---------------------------------------------------------------- terminal kernel ----------------------------
struct TerminalArgs {
    const void *target;
    const void *draft;
    const int32_t *draft_tokens;
    const float *uniforms;
    int K;
    float s;
    const int32_t *accept;
    const int32_t *labels;
    const int32_t *posflags;
    const float4 *stats;
    int32_t *out_accept_len;
    int32_t *out_tokens;
    int32_t *out_groups;  // may be null
    int32_t *out_flags;   // may be null
};

template <typename T>
__global__ void __launch_bounds__(kAggThreads, 2) terminal_kernel(TerminalArgs a, GroupsDev G) {
    pdl_enter();
    constexpr int NT = kAggThreads;
    extern __shared__ __align__(16) unsigned char raw[];
    AggSmem sm = carve_smem(raw, G);
    cg::cluster_group cluster = cg::this_cluster();
    const int C = G.slices, K = a.K, V = G.V, M = G.M;
    const int c = (int)cluster.block_rank();
    const int b = blockIdx.x / C;
    const int tid = threadIdx.x;

    // ---- first rejected position: warp ballots over the accept bits, 32 positions at a time ----
    if (tid < 32) {
        // 32 accept bits per ballot; the first word with a rejection ends the search
        int n = K, flags = 0;
        for (int base = 0; base < K && n == K; base += 32) {
            const int i = base + tid;
            const int rej = (i < K) && (a.accept[b * K + i] == 0);
            const unsigned mask = __ballot_sync(0xffffffffu, rej);
            if (mask) n = base + __ffs(mask) - 1;
        }
        for (int base = 0; base < K && base <= n; base += 32) {
            const int i = base + tid;
            const int f = (i < K && i <= n) ? a.posflags[b * K + i] : 0;
            flags |= __reduce_or_sync(0xffffffffu, f);
        }
        if (tid == 0) {
            sm.ibox[0] = n;
            sm.ibox[1] = flags;
        }
    }
    __syncthreads();
    const int n = sm.ibox[0];
    int flags = sm.ibox[1];
    const T *trow = reinterpret_cast<const T *>(a.target) + ((int64_t)b * (K + 1) + n) * V;
    const T *qrow = reinterpret_cast<const T *>(a.draft) + ((int64_t)b * K + min(n, K - 1)) * V;
    const int t0 = c * G.slice_len;
    const int ns = max(0, min(G.slice_len, V - t0));
    const int g0 = c * G.groups_per_slice, g1 = min(M, g0 + G.groups_per_slice);
    const int nown = max(0, g1 - g0);
    const float u_group = a.uniforms[((int64_t)b * (K + 1) + K) * 2];
    const float u_token = a.uniforms[((int64_t)b * (K + 1) + K) * 2 + 1];

    bool residual = n < K;  // false: draw from the target's coarse distribution itself (bonus token)
    float rs_tgt = 0.f;  // scaled reference of the target row's softmax terms
    double Ztot = 0.0, my_off = 0.0, my_excl = 0.0, my_incl = 0.0, my_sum = 0.0;
    const int per = (nown + NT - 1) / NT;
    const int i0 = min(nown, tid * per), i1 = min(nown, i0 + per);
    for (int attempt = 0; attempt < 2; ++attempt) {
        // ---- per-token values of this slice ----
        clear_partial<NT>(G, sm.d, sm.partial);
        if (residual) {
            const float4 st = a.stats[b * K + n];
            rs_tgt = st.x;
            constexpr int NV = Elem<T>::kPerVec;
            const T *tp = trow + t0, *qp = qrow + t0;
            int done = 0;
            if (ns > 0 && (((uintptr_t)tp | (uintptr_t)qp) & 15u) == 0) {
                const int nvec = ns / NV;
                for (int idx = tid; idx < nvec; idx += NT) {
                    float vp[NV], vq[NV];
                    Elem<T>::unpack(ld_stream(reinterpret_cast<const uint4 *>(tp) + idx), vp);
                    Elem<T>::unpack(ld_stream(reinterpret_cast<const uint4 *>(qp) + idx), vq);
#pragma unroll
                    for (int e = 0; e < NV; ++e) {
                        const float diff = __fmul_rn(ex2(__fmaf_rn(vp[e], a.s, -st.x)), st.y) -
                                           __fmul_rn(ex2(__fmaf_rn(vq[e], a.s, -st.z)), st.w);
                        const int t = idx * NV + e;
                        sm.d[t] = G.ent_w ? diff : __fmul_rn(diff, G.inv_deg[t0 + t]);
                    }
                }
                done = nvec * NV;
            }
            for (int t = done + tid; t < ns; t += NT) {
                const float diff = __fmul_rn(ex2(__fmaf_rn(Elem<T>::widen(tp[t]), a.s, -st.x)), st.y) -
                                   __fmul_rn(ex2(__fmaf_rn(Elem<T>::widen(qp[t]), a.s, -st.z)), st.w);
                sm.d[t] = G.ent_w ? diff : __fmul_rn(diff, G.inv_deg[t0 + t]);
            }
            __syncthreads();
        } else {
            const float mloc = load_slice_max<T, NT>(trow + t0, ns, sm.d, sm.scratch);
            if (tid == 0) sm.xchg[1] = (double)mloc;
            cluster.sync();
            float m = kNegInf;
            for (int r = 0; r < C; ++r) m = fmaxf(m, (float)*cluster.map_shared_rank(&sm.xchg[1], r));
            rs_tgt = m * a.s;
            for (int t = tid; t < ns; t += NT) {
                const float e = ex2(__fmaf_rn(sm.d[t], a.s, -rs_tgt));
                sm.d[t] = G.ent_w ? e : __fmul_rn(e, G.inv_deg[t0 + t]);
            }
            __syncthreads();
        }
        // ---- all groups: slice share, then totals of the owned groups over the cluster ----
        sweep_slice<NT>(G, c, sm.d, sm.partial);
        cluster.sync();
        for (int j = tid; j < nown; j += NT) {
            float tot = 0.f;
            for (int r = 0; r < C; ++r) tot += cluster.map_shared_rank(sm.partial, r)[g0 + j];
            sm.own[j] = fmaxf(tot, 0.f);  // (P - Q)_+ ; NaN becomes 0
        }
        __syncthreads();
        // ---- prefix sums over the owned groups (double), block total to the cluster ----
        my_sum = 0.0;
        for (int j = i0; j < i1; ++j) my_sum += (double)sm.own[j];
        double blk;
        block_scan<NT>(my_sum, sm.dscratch, &my_excl, &my_incl, &blk);
        if (tid == 0) sm.xchg[0] = blk;
        cluster.sync();
        Ztot = 0.0;
        for (int r = 0; r < C; ++r) {
            if (r == c) my_off = Ztot;
            Ztot += *cluster.map_shared_rank(&sm.xchg[0], r);
        }
        if (Ztot > 0.0 || !residual) break;
        // a rejection whose residual vanished (P == Q to rounding): draw from P instead
        flags |= PCG_FLAG_ZERO_RESIDUAL;
        residual = false;
        cluster.sync();  // everyone has read partial/xchg before they are overwritten
    }

    // ---- which block holds the drawn group: first block whose running total exceeds u * Z ----
    const double target = (double)u_group * Ztot;
    int winner = -1, last_nonzero = -1;
    {
        double run = 0.0;
        for (int r = 0; r < C; ++r) {
            const double z = *cluster.map_shared_rank(&sm.xchg[0], r);
            if (z > 0.0) last_nonzero = r;
            run += z;
            if (winner < 0 && run > target) winner = r;
        }
    }
    const bool pick_last = winner < 0;  // rounding left no block above the target: last group with mass
    if (pick_last) winner = last_nonzero;
    if (winner < 0) {  // no mass anywhere (non-finite inputs): emit group 0 / token 0 and flag it
        winner = 0;
        flags |= PCG_FLAG_NONFINITE;
    }
    if (c == winner) {
        if (tid == 0) {
            sm.ibox[2] = NT;   // selected thread (minimum)
            sm.ibox[3] = -1;   // last owned group with mass (maximum)
            sm.ibox[4] = -1;   // drawn group
        }
        __syncthreads();
        int my_last = -1;
        for (int j = i0; j < i1; ++j)
            if (sm.own[j] > 0.f) my_last = j;
        if (my_last >= 0) atomicMax(&sm.ibox[3], my_last);
        if (!pick_last && my_sum > 0.0 && my_off + my_incl > target) atomicMin(&sm.ibox[2], tid);
        __syncthreads();
        if (!pick_last && sm.ibox[2] == tid) {
            double loc = 0.0;
            int pick = my_last;
            for (int j = i0; j < i1; ++j) {
                loc += (double)sm.own[j];
                if (my_off + (my_excl + loc) > target) {
                    pick = j;
                    break;
                }
            }
            sm.ibox[4] = pick;
        }
        __syncthreads();
        int gsel = sm.ibox[4] >= 0 ? sm.ibox[4] : sm.ibox[3];
        int z = 0;
        if (gsel < 0) {
            gsel = 0;
            flags |= PCG_FLAG_NONFINITE;
        } else {
            gsel += g0;
            // ---- token inside the drawn group: target-conditional p(t) w / P[g] over the group's CSR order ----
            const int lo = G.group_ptr[gsel], hi = G.group_ptr[gsel + 1], len = hi - lo;
            const int per2 = (len + NT - 1) / NT;
            const int k0 = min(len, tid * per2), k1 = min(len, k0 + per2);
            auto omega = [&](int k) -> float {
                const int t = G.group_tok[lo + k];
                const float w = G.pair_w ? G.pair_w[lo + k] : G.inv_deg[t];
                return __fmul_rn(ex2(__fmaf_rn(Elem<T>::widen(trow[t]), a.s, -rs_tgt)), w);
            };
            double wsum = 0.0;
            int wlast = -1;
            for (int k = k0; k < k1; ++k) {
                const float w = omega(k);
                wsum += (double)w;
                if (w > 0.f) wlast = k;
            }
            double excl, incl, wtot;
            block_scan<NT>(wsum, sm.dscratch, &excl, &incl, &wtot);
            if (tid == 0) {
                sm.ibox[2] = NT;
                sm.ibox[3] = -1;
                sm.ibox[4] = -1;
            }
            __syncthreads();
            const double target2 = (double)u_token * wtot;
            if (wlast >= 0) atomicMax(&sm.ibox[3], wlast);
            if (wsum > 0.0 && incl > target2) atomicMin(&sm.ibox[2], tid);
            __syncthreads();
            if (sm.ibox[2] == tid) {
                double loc = 0.0;
                int pick = wlast;
                for (int k = k0; k < k1; ++k) {
                    loc += (double)omega(k);
                    if (excl + loc > target2) {
                        pick = k;
                        break;
                    }
                }
                sm.ibox[4] = pick;
            }
            __syncthreads();
            const int ksel = sm.ibox[4] >= 0 ? sm.ibox[4] : sm.ibox[3];
            if (ksel >= 0) {
                z = G.group_tok[lo + ksel];
            } else {  // the drawn group has no token with target mass (non-finite inputs)
                z = len > 0 ? G.group_tok[lo] : 0;
                flags |= PCG_FLAG_NONFINITE;
            }
        }
        // ---- emit: accepted draft tokens, the drawn token, then filler ----
        for (int i = tid; i <= K; i += NT) {
            int tok = -1, grp = -1;
            if (i < n) {
                tok = a.draft_tokens[b * K + i];
                if (tok < 0 || tok >= V) tok = 0;  // verified as token 0 (and flagged), so emitted as token 0
                grp = a.labels[b * K + i];
            } else if (i == n) {
                tok = z;
                grp = gsel;
            }
            a.out_tokens[(int64_t)b * (K + 1) + i] = tok;
            if (a.out_groups) a.out_groups[(int64_t)b * (K + 1) + i] = grp;
        }
        if (tid == 0) {
            a.out_accept_len[b] = n;
            if (a.out_flags) a.out_flags[b] = flags;
        }
    }
    cluster.sync();  // no block may exit while another still reads its shared memory
}

// ================================================================ batched terminal stage ====================
//
// The terminal draw of a sequence needs the residual (P - Q)_+ of ALL groups at one position (the first
// rejection, or the bonus row).  Over a batch that is one sparse-matrix product: R[g, b] = sum_{t in G_g}
// D[b, t], with D[b, t] = (p(t) - q(t)) / N(t) at sequence b's terminal position.  Three kernels:
//   residual_transpose_kernel  finds every sequence's first rejection (warp ballots over the accept bits), re-reads
//                              the two rows of that position and writes D TRANSPOSED: tiles of 32 sequences side by
//                              side, Dt[batch of 32][token][32], one bulk copy per tile
//   group_spmm_kernel          one warp per (part of the groups, block of 32 to 256 sequences): walks the part's
//                              token lists once and adds one row segment of Dt per token (Dt stays in L2); writes
//                              the group sums and, per part, the sum of their positive parts
//   terminal_pick_kernel       one block per sequence: prefix scan over the parts' sums, the part in which the
//                              cumulative mass passes u * Z is opened, group draw, token draw, outputs
// Sequences are processed in chunks whose Dt fits in L2.  pcg_group_probs uses the first two with row-major
// output; dense mode (all groups at every position) uses terminal_prepare_kernel and terminal_draw_kernel.

constexpr int kPrepThreads = 256;  // terminal_prepare_kernel, row_stats_kernel
constexpr int kProbsBatchedRows = 64;  // pcg_group_probs: from this many rows on, the batched kernels
constexpr int kTrThreads = 256;    // residual_transpose_kernel
constexpr int kSpmmThreads = 128;  // group_spmm_kernel
constexpr int kSpmmWide = 4;       // sequences per lane of the sparse product for batches of 128 to 255 sequences (8 beyond, 1 below)
constexpr int kSpmmDepth = 8;      // tokens per batch of that form; two batches of loads are in flight per lane
constexpr int kDrawThreads = 512;  // terminal_draw_kernel (dense mode)
constexpr int kPickThreads = 256;  // terminal_pick_kernel

struct PrepareArgs {
    const void *target;
    int K;
    float s;
    int want_bonus_stats;  // 0 in dense mode (the stored P of the bonus row is used instead)
    const int32_t *accept;
    const int32_t *posflags;
    const float4 *stats;
    int32_t *term_n;      // [B] first rejected position, K if none
    int32_t *term_flags;  // [B] flags of the positions up to and including n
    float4 *term_stats;   // [B] (RS_p, 1/Z_p, RS_q, 1/Z_q) of the terminal position; (RS_p, 1/Z_p, 0, 0) for a bonus row
};

// First rejected position of sequence b by one warp: ballots over the accept bits, 32 positions at a time (the
// first word with a rejection ends the search), and the OR of the flags of the positions up to and including it.
__device__ __forceinline__ void warp_first_reject(const int32_t *accept, const int32_t *posflags, int b, int K, int lane,
                                                  int &n_out, int &flags_out) {
    int n = K, flags = 0;
    for (int base = 0; base < K && n == K; base += 32) {
        const int i = base + lane;
        const int rej = (i < K) && (accept[b * K + i] == 0);
        const unsigned mask = __ballot_sync(0xffffffffu, rej);
        if (mask) n = base + __ffs(mask) - 1;
    }
    for (int base = 0; base < K && base <= n; base += 32) {
        const int i = base + lane;
        const int f = (i < K && i <= n) ? posflags[b * K + i] : 0;
        flags |= __reduce_or_sync(0xffffffffu, f);
    }
    n_out = n;
    flags_out = flags;
}

// Dense mode only: first rejection per sequence from the accept bits of dense_accept_kernel.
template <typename T>
__global__ void __launch_bounds__(kPrepThreads) terminal_prepare_kernel(PrepareArgs a, GroupsDev G) {
    pdl_enter();
    const int b = blockIdx.x, tid = threadIdx.x, K = a.K;
    if (tid < 32) {
        int n, flags;
        warp_first_reject(a.accept, a.posflags, b, K, tid, n, flags);
        if (tid == 0) {
            a.term_n[b] = n;
            a.term_flags[b] = flags;
            a.term_stats[b] = n < K ? a.stats[b * K + n] : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    }
}

// Softmax statistics (scaled reference, 1/Z) of plain rows: one block per row.  Used by the batched route of
// pcg_group_probs.
template <typename T>
__global__ void __launch_bounds__(kPrepThreads) row_stats_kernel(const void *logits, float s, float4 *stats, GroupsDev G) {
    pdl_enter();
    constexpr int NT = kPrepThreads, NW = NT / 32, NV = Elem<T>::kPerVec;
    __shared__ float red[2 * NW];
    const int tid = threadIdx.x, V = G.V;
    const T *row = reinterpret_cast<const T *>(logits) + (int64_t)blockIdx.x * V;
    RefSum st{kRefInit * s, 0.f};
    int head = (int)(((16u - (unsigned)((uintptr_t)row & 15u)) & 15u) / sizeof(T));
    if (head > V) head = V;
    const int nvec = (V - head) / NV;
    const uint4 *vp = reinterpret_cast<const uint4 *>(row + head);
    int idx = tid;
    for (; idx + 3 * NT < nvec; idx += 4 * NT) {
        uint4 r[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) r[j] = ld_stream(vp + idx + j * NT);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float v[NV];
            Elem<T>::unpack(r[j], v);
            absorb<NV>(st, v, s);
        }
    }
    for (; idx < nvec; idx += NT) {
        float v[NV];
        Elem<T>::unpack(ld_stream(vp + idx), v);
        absorb<NV>(st, v, s);
    }
    for (int t = tid; t < head; t += NT) absorb1(st, Elem<T>::widen(row[t]), s);
    for (int t = head + nvec * NV + tid; t < V; t += NT) absorb1(st, Elem<T>::widen(row[t]), s);
    float rs = st.rs, Z = st.acc;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) merge(rs, Z, __shfl_xor_sync(0xffffffffu, rs, o), __shfl_xor_sync(0xffffffffu, Z, o));
    if ((tid & 31) == 0) {
        red[2 * (tid >> 5)] = rs;
        red[2 * (tid >> 5) + 1] = Z;
    }
    __syncthreads();
    if (tid == 0) {
        rs = red[0];
        Z = red[1];
        for (int w = 1; w < NW; ++w) merge(rs, Z, red[2 * w], red[2 * w + 1]);
        stats[blockIdx.x] = make_float4(rs, 1.0f / Z, 0.f, 0.f);
    }
}

// Loads of Dt: cached in L2 only (.cg).  Every line of Dt is read once per group its token belongs to, at
// unrelated times, so it has to survive in L2 between those reads; the streaming form used for the logits
// (ld.global.nc.L1::no_allocate) is retained in L2 for too short a time for that.
__device__ __forceinline__ float ld_l2_f32(const float *p) {
    float r;
    asm volatile("ld.global.cg.f32 %0, [%1];" : "=f"(r) : "l"(p));
    return r;
}
__device__ __forceinline__ float4 ld_l2_f32x4(const float *p) {
    float4 r;
    asm volatile("ld.global.cg.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w)
                 : "l"(p));
    return r;
}

struct TransposeArgs {
    const void *target;
    const void *draft;
    int B, K;
    int b0;             // first sequence of this chunk
    float s;
    // The terminal position of a sequence comes from the accept bits of the position kernel (from_accept = 1: this
    // kernel finds the first rejection itself and leaves term_n / term_flags / term_stats for the kernels behind
    // it), or is read from term_n / term_stats as filled by an earlier kernel (from_accept = 0), or is row 0 of a
    // plain batch of rows whose statistics are in term_stats (from_accept = 2, with K = 0: pcg_group_probs).
    int from_accept;
    const int32_t *accept, *posflags;  // [B*K]
    const float4 *stats;               // [B*K]
    const float4 *bonus_stats;         // [B]
    const int32_t *bonus_flags;        // [B]
    int32_t *term_n;                   // [B]
    int32_t *term_flags;               // [B]
    float4 *term_stats;                // [B]
    float *Dt;                         // [sequences of the chunk / 32][V][32]
};

// The bits of "-inf" in the logits' storage type, two (or one) to a 32-bit word: what a lane uses in place of
// logits it must not read (past the end of a row, the draft row of a bonus position, sequences past the batch).
template <typename T>
struct NegInfBits;
template <>
struct NegInfBits<float> {
    static constexpr uint32_t word = 0xff800000u;
};
template <>
struct NegInfBits<uint16_t> {
    static constexpr uint32_t word = 0xff80ff80u;
};
template <>
struct NegInfBits<f16_t> {
    static constexpr uint32_t word = 0xfc00fc00u;
};

// The logits held by one 32-bit word of a row.
template <typename T>
struct WordElems;
template <>
struct WordElems<float> {
    static constexpr int kPerWord = 1;
    static __device__ __forceinline__ void unpack(uint32_t w, float (&v)[1]) { v[0] = __uint_as_float(w); }
};
template <>
struct WordElems<uint16_t> {
    static constexpr int kPerWord = 2;
    static __device__ __forceinline__ void unpack(uint32_t w, float (&v)[2]) {
        v[0] = __uint_as_float(w << 16);
        v[1] = __uint_as_float(w & 0xffff0000u);
    }
};
template <>
struct WordElems<f16_t> {
    static constexpr int kPerWord = 2;
    static __device__ __forceinline__ void unpack(uint32_t w, float (&v)[2]) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w));
        v[0] = f.x;
        v[1] = f.y;
    }
};

// 32 bytes of a row, streamed (read once: first to leave the L2, so that Dt stays).
__device__ __forceinline__ void ld_stream_32(const void *p, uint32_t (&w)[8]) {
    asm volatile("ld.global.nc.L1::no_allocate.L2::evict_first.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
                 : "l"(p));
}

// A store whose line should be the last to leave the L2: Dt is read back about six times per line by the sparse
// product, and lines of it that were pushed out in between went to DRAM and came back (about 20 MB per call before).
__device__ __forceinline__ uint64_t l2_evict_last_policy() {
    uint64_t pol;
    asm("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void st_keep(float *p, float v, uint64_t pol) {
    asm volatile("st.global.L2::cache_hint.f32 [%0], %1, %2;" ::"l"(p), "f"(v), "l"(pol) : "memory");
}

// Grid (blocks per batch, batches of 32 sequences); block = 8 warps.  LANE = SEQUENCE throughout: a lane reads
// 64 bytes of its own sequence's two rows per step (two whole sectors, one DRAM access: with 32 bytes per step a
// third more bytes than needed came from DRAM; the eight warps of a block take neighbouring steps, so a row is
// fetched in 512-byte stretches), forms D = (p - q) w for those tokens in registers, and the
// warp writes one 128-byte line of Dt per token -- [token][32 sequences] needs no transposition this way.
//   0. once per block, by warp 0: every lane finds its sequence's first rejection from the accept bits (its
//      loads all in flight) and fetches the softmax statistics of that position;
//   1. the block's run of the row is walked with the next step's 128 bytes in flight while the current step's
//      tokens are computed and stored.
// Lanes that have nothing to read (sequences past the batch, the draft row of a bonus position, tokens past the
// end of a row) use -inf logits, which contribute exact zeros.
template <typename T>
__global__ void __launch_bounds__(kTrThreads, 2) residual_transpose_kernel(TransposeArgs a, GroupsDev G) {
    pdl_enter();
    constexpr int PW = WordElems<T>::kPerWord;  // logits per 32-bit word
    constexpr int WPS = 16;                     // 32-bit words per step: 64 bytes of a row
    constexpr int CH = WPS * PW;                // tokens per step
    constexpr int NWARP = kTrThreads / 32;
    __shared__ int s_n[32];
    __shared__ float4 s_st[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int V = G.V, K = a.K;
    const int bbase = a.b0 + blockIdx.y * 32;

    // ---- 0. terminal position and statistics of the batch's sequences ----
    if (warp == 0) {
        const int b = bbase + lane;
        int n = -1, flags = 0;
        float4 st = make_float4(0.f, 0.f, 0.f, 0.f);
        if (b < a.B) {
            if (a.from_accept != 1) {
                n = a.from_accept == 2 ? 0 : a.term_n[b];
                st = a.term_stats[b];
            } else {
                n = K;
                for (int i0 = 0; i0 < K && n == K; i0 += 16) {  // sixteen positions' loads in flight
                    int acc[16], pf[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const bool in = i0 + j < K;
                        acc[j] = in ? a.accept[b * K + i0 + j] : 1;
                        pf[j] = in ? a.posflags[b * K + i0 + j] : 0;
                    }
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        if (n == K) {
                            flags |= pf[j];  // flags of the positions up to and including the first rejection
                            if (acc[j] == 0) n = i0 + j;
                        }
                    }
                }
                if (n < K) {
                    st = a.stats[b * K + n];
                } else {
                    st = a.bonus_stats[b];
                    flags |= a.bonus_flags[b];
                }
                if (blockIdx.x == 0) {
                    a.term_n[b] = n;
                    a.term_flags[b] = flags;
                    a.term_stats[b] = st;
                }
            }
        }
        s_n[lane] = n;
        s_st[lane] = st;
    }
    __syncthreads();

    // ---- 1. this lane's sequence ----
    const int n = s_n[lane];
    float4 st = s_st[lane];
    const bool live = n >= 0, resid = live && n < K;
    if (!live) st = make_float4(0.f, 0.f, 0.f, 0.f);
    if (!resid) st.z = 0.f, st.w = 0.f;  // no draft term: its logits read as -inf and the factor is zero
    const int b = bbase + lane, nn = max(n, 0);
    const T *tp = reinterpret_cast<const T *>(a.target) + ((int64_t)(live ? b : 0) * (K + 1) + nn) * V;
    const T *qp = K > 0 ? reinterpret_cast<const T *>(a.draft) + ((int64_t)(live ? b : 0) * K + min(nn, K - 1)) * V : tp;
    // whole 64-byte pieces can be loaded as such if every live lane's rows start on 64-byte boundaries
    const bool lane_al = !live || ((((uintptr_t)tp | (resid ? (uintptr_t)qp : 0)) & 63u) == 0);
    const bool aligned = __all_sync(0xffffffffu, lane_al) && ((size_t)V * sizeof(T)) % 64 == 0;
    const int nsteps = (V + CH - 1) / CH;
    const int step_lo = (int)(((int64_t)nsteps * blockIdx.x) / gridDim.x);
    const int step_hi = (int)(((int64_t)nsteps * (blockIdx.x + 1)) / gridDim.x);
    float *dst = a.Dt + ((size_t)blockIdx.y * V) * 32 + lane;
    const uint64_t keep = l2_evict_last_policy();

    auto fetch = [&](int step, uint32_t(&wp)[WPS], uint32_t(&wq)[WPS]) {
        const int t = step * CH;
#pragma unroll
        for (int j = 0; j < WPS; ++j) wp[j] = wq[j] = NegInfBits<T>::word;
        if (step >= step_hi) return;
        if (aligned && t + CH <= V) {
            if (live) {
                ld_stream_32(tp + t, *reinterpret_cast<uint32_t(*)[8]>(&wp[0]));
                ld_stream_32(tp + t + CH / 2, *reinterpret_cast<uint32_t(*)[8]>(&wp[8]));
            }
            if (resid) {
                ld_stream_32(qp + t, *reinterpret_cast<uint32_t(*)[8]>(&wq[0]));
                ld_stream_32(qp + t + CH / 2, *reinterpret_cast<uint32_t(*)[8]>(&wq[8]));
            }
        } else {  // ragged end of the row, or rows that are not 64-byte aligned: element by element
            T ep[CH], eq[CH];
            memcpy(ep, wp, 4 * WPS);
            memcpy(eq, wq, 4 * WPS);
#pragma unroll
            for (int e = 0; e < CH; ++e) {
                if (t + e < V) {
                    if (live) ep[e] = tp[t + e];
                    if (resid) eq[e] = qp[t + e];
                }
            }
            memcpy(wp, ep, 4 * WPS);
            memcpy(wq, eq, 4 * WPS);
        }
    };
    auto emit = [&](int step, const uint32_t(&wp)[WPS], const uint32_t(&wq)[WPS]) {
        const int t = step * CH;
        float inv[CH];
        if (!G.ent_w && t + CH <= V) {
#pragma unroll
            for (int j = 0; j < CH / 4; ++j) {
                const float4 v = *reinterpret_cast<const float4 *>(G.inv_deg + t + 4 * j);  // (the same for all lanes)
                inv[4 * j] = v.x, inv[4 * j + 1] = v.y, inv[4 * j + 2] = v.z, inv[4 * j + 3] = v.w;
            }
        } else {
#pragma unroll
            for (int e = 0; e < CH; ++e) inv[e] = (!G.ent_w && t + e < V) ? G.inv_deg[t + e] : 1.f;
        }
#pragma unroll
        for (int j = 0; j < WPS; ++j) {
            float lp[PW], lq[PW];
            WordElems<T>::unpack(wp[j], lp);
            WordElems<T>::unpack(wq[j], lq);
#pragma unroll
            for (int e = 0; e < PW; ++e) {
                float v = __fmul_rn(ex2(__fmaf_rn(lp[e], a.s, -st.x)), st.y);
                v -= __fmul_rn(ex2(__fmaf_rn(lq[e], a.s, -st.z)), st.w);
                const int r = t + j * PW + e;
                if (r < V) st_keep(dst + (size_t)r * 32, __fmul_rn(v, inv[j * PW + e]), keep);
            }
        }
    };
    uint32_t ap[WPS], aq[WPS], bp[WPS], bq[WPS];
    int step = step_lo + warp;
    fetch(step, ap, aq);
    for (; step < step_hi; step += 2 * NWARP) {
        fetch(step + NWARP, bp, bq);
        emit(step, ap, aq);
        if (step + NWARP < step_hi) {
            fetch(step + 2 * NWARP, ap, aq);
            emit(step + NWARP, bp, bq);
        }
    }
}

struct SpmmArgs {
    const float *Dt;  // [sequences of the chunk / 32][V][32]
    int B;
    int b0;           // first sequence of this chunk
    int bpad;         // sequences per row of Rt and Psum (the chunk size, a multiple of 32 * SPL)
    float *R;         // Rt [M, bpad]: raw sums by group
    float *Psum;      // [nparts, bpad]: per part, the sum of the positive parts of its groups' sums (PSUM only)
};

template <int SPL>
struct SeqVec;
template <>
struct SeqVec<1> {
    float v[1];
    __device__ __forceinline__ void load(const float *p) { v[0] = ld_l2_f32(p); }
    __device__ __forceinline__ void store(float *p) const { *p = v[0]; }
};
template <>
struct SeqVec<4> {
    float v[4];
    __device__ __forceinline__ void load(const float *p) {
        const float4 r = ld_l2_f32x4(p);
        v[0] = r.x, v[1] = r.y, v[2] = r.z, v[3] = r.w;
    }
    __device__ __forceinline__ void store(float *p) const { *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]); }
};
template <>
struct SeqVec<8> {  // one 256-bit load per lane
    float v[8];
    __device__ __forceinline__ void load(const float *p) {
        asm volatile("ld.global.cg.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7])
                     : "l"(p));
    }
    __device__ __forceinline__ void store(float *p) const {
        reinterpret_cast<float4 *>(p)[0] = make_float4(v[0], v[1], v[2], v[3]);
        reinterpret_cast<float4 *>(p)[1] = make_float4(v[4], v[5], v[6], v[7]);
    }
};

// Grid (ceil(nparts / warps per block), bpad / (32 * SPL)).  A warp owns one part of the groups -- at most
// kPartMaxGroups consecutive groups, one contiguous range of the CSR; the parts hold about the same number of
// stored pairs, so all warps of the (single) wave finish together -- and a block of 32 * SPL sequences; a lane
// holds SPL consecutive sequences (one 4-, 16- or 32-byte load per token).  The range is walked in batches of
// DEPTH tokens with two register buffers: the loads of batch i+1 are issued before batch i is added, so a warp
// keeps up to 2 * DEPTH lines of Dt in flight at all times.  Token ids are fetched 32 at a time, one block of 32
// ahead.  Sums run in CSR order; a group ends where the running entry index reaches the next group pointer.
// Output by group (verification): a closed group's SPL sums go straight to Rt[g, sequences], their positive
// parts are added up per part and written to Psum[part, sequences] (PSUM; pcg_group_probs needs no part sums and
// turns Rt into its row-major output with rows_from_groups_kernel).
template <int SPL, int DEPTH, bool HAS_W, bool PSUM>
__global__ void __launch_bounds__(kSpmmThreads, 5) group_spmm_kernel(SpmmArgs a, GroupsDev G) {
    constexpr int NS = 32 * SPL;  // sequences per warp
    static_assert(32 % DEPTH == 0 && DEPTH <= 16, "a batch never straddles two blocks of 32 token ids");
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int part = blockIdx.x * (kSpmmThreads / 32) + warp;
    if (part >= G.nparts) return;  // warp-uniform; the kernel has no block-wide barrier
    // the part's groups and stored pairs (both pairs of bounds in one round trip, so that the group pointers and
    // the first token ids can be fetched side by side)
    const int pp_l = lane < 2 ? G.part_ptr[part + lane] : (lane < 4 ? G.part_ent[part + lane - 2] : 0);
    const int g0 = __shfl_sync(0xffffffffu, pp_l, 0), ng = __shfl_sync(0xffffffffu, pp_l, 1) - g0;
    const int e0 = __shfl_sync(0xffffffffu, pp_l, 2), e1 = __shfl_sync(0xffffffffu, pp_l, 3);
    // this lane's SPL sequences: number sq0 of the chunk, in the 32-sequence batch sq0 / 32 of Dt
    const int sq0 = blockIdx.y * NS + lane * SPL;
    const float *col = a.Dt + ((size_t)(sq0 >> 5) * G.V) * 32 + (sq0 & 31);
    const int ptr_l = lane <= ng ? G.group_ptr[g0 + lane] : 0;  // lane i: group_ptr[g0 + i]
    const int nbatch = (e1 - e0 + DEPTH - 1) / DEPTH;

    // token ids (and weights) of entries e0 + 32*blk + lane; entries past the end repeat the last one
    auto load_ids = [&](int blk, int &tok, float &w) {
        const int k = min(e0 + blk * 32 + lane, e1 - 1);
        tok = (e1 > e0) ? G.group_tok[k] : 0;
        w = (HAS_W && e1 > e0) ? G.pair_w[k] : 1.f;
    };
    int ids_cur, ids_nxt;
    float w_cur, w_nxt;
    load_ids(0, ids_cur, w_cur);
    load_ids(1, ids_nxt, w_nxt);
    // Everything above reads the handle's tables only, so it runs while the kernel before (which wrote Dt) drains.
    // The kernel behind this one is released only AFTER the wait: once its blocks run, the kernel that wrote Dt --
    // and with it the terminal positions and their statistics -- is known to have completed, and those may be read
    // ahead of that kernel's own wait (terminal_pick_kernel does).
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;");
    // issue the loads of batch i (its ids live in ids_cur if it belongs to block `blk_cur`, else in ids_nxt)
    int blk_cur = 0;
    auto issue = [&](int i, SeqVec<SPL>(&x)[DEPTH]) {
        const int off = i * DEPTH;  // entry offset from e0
        const bool in_cur = (off >> 5) == blk_cur;
        const int src = in_cur ? ids_cur : ids_nxt;
#pragma unroll
        for (int j = 0; j < DEPTH; ++j) {
            const int tok = __shfl_sync(0xffffffffu, src, (off + j) & 31);
            x[j].load(col + (size_t)tok * 32);  // past the end: a repeat of the last line, never added
        }
    };
    SeqVec<SPL> acc, pos;  // running sums of the open group; sum of the positive parts of the closed ones
#pragma unroll
    for (int q = 0; q < SPL; ++q) acc.v[q] = pos.v[q] = 0.f;
    int gi = 0;
    int gend = __shfl_sync(0xffffffffu, ptr_l, 1);
    auto close_groups = [&](int k) {  // the entry index reached k: close every group that ends at or before k
        while (gi < ng && gend <= k) {
            acc.store(a.R + (size_t)(g0 + gi) * a.bpad + sq0);
            if (PSUM) {
#pragma unroll
                for (int q = 0; q < SPL; ++q) pos.v[q] += fmaxf(acc.v[q], 0.f);  // (P - Q)_+ ; NaN counts as 0
            }
#pragma unroll
            for (int q = 0; q < SPL; ++q) acc.v[q] = 0.f;
            ++gi;
            gend = __shfl_sync(0xffffffffu, ptr_l, min(gi + 1, 31));
        }
    };
    auto consume = [&](int i, const SeqVec<SPL>(&x)[DEPTH]) {
        const int off = i * DEPTH;
        // advance the id blocks once the first batch of a new block is consumed (its loads were issued from ids_nxt)
        if ((off >> 5) != blk_cur) {
            blk_cur = off >> 5;
            ids_cur = ids_nxt;
            w_cur = w_nxt;
            load_ids(blk_cur + 1, ids_nxt, w_nxt);
        }
        const int n = min(DEPTH, e1 - e0 - off);
        if (n == DEPTH && gend > e0 + off + DEPTH) {
            // a whole batch inside one group (most batches): plain adds, in the same order
#pragma unroll
            for (int j = 0; j < DEPTH; ++j) {
                if (HAS_W) {
                    const float w = __shfl_sync(0xffffffffu, w_cur, (off + j) & 31);
#pragma unroll
                    for (int q = 0; q < SPL; ++q) acc.v[q] += __fmul_rn(x[j].v[q], w);
                } else {
#pragma unroll
                    for (int q = 0; q < SPL; ++q) acc.v[q] += x[j].v[q];
                }
            }
            return;
        }
#pragma unroll
        for (int j = 0; j < DEPTH; ++j) {
            if (j < n) {
                if (HAS_W) {
                    const float w = __shfl_sync(0xffffffffu, w_cur, (off + j) & 31);
#pragma unroll
                    for (int q = 0; q < SPL; ++q) acc.v[q] += __fmul_rn(x[j].v[q], w);
                } else {
#pragma unroll
                    for (int q = 0; q < SPL; ++q) acc.v[q] += x[j].v[q];
                }
                close_groups(e0 + off + j + 1);
            }
        }
    };
    close_groups(e0);  // leading empty groups
    SeqVec<SPL> xa[DEPTH], xb[DEPTH];
    if (nbatch > 0) issue(0, xa);
    for (int i = 0; i < nbatch; i += 2) {
        if (i + 1 < nbatch) issue(i + 1, xb);
        consume(i, xa);
        if (i + 2 < nbatch) issue(i + 2, xa);
        if (i + 1 < nbatch) consume(i + 1, xb);
    }
    close_groups(e1);  // trailing empty groups (gi reaches ng)
    if (PSUM) pos.store(a.Psum + (size_t)part * a.bpad + sq0);
}

// out[row, g] = Rt[g, row]: the group-major sums of the sparse product as the row-major result of pcg_group_probs.
// Grid (ceil(M / 32), ceil(rows / 32)) x (32, 8): a 32 x 32 tile through padded shared memory, both sides coalesced.
__global__ void __launch_bounds__(256) rows_from_groups_kernel(const float *Rt, int bpad, int rows, int M, float *out) {
    pdl_enter();
    __shared__ float tile[32][33];
    const int g0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
    for (int j = threadIdx.y; j < 32; j += 8) {
        const int g = g0 + j, r = r0 + (int)threadIdx.x;
        tile[j][threadIdx.x] = (g < M && r < rows) ? Rt[(size_t)g * bpad + r] : 0.f;
    }
    __syncthreads();
    for (int j = threadIdx.y; j < 32; j += 8) {
        const int r = r0 + j, g = g0 + (int)threadIdx.x;
        if (r < rows && g < M) out[(size_t)r * M + g] = tile[threadIdx.x][j];
    }
}

// Token inside a group (stored pairs [lo, lo + len)) by ONE WARP: inverse CDF with u_token over p(t) w_{g,t} in the group's CSR order (the
// target-conditional; the common factor 1/Z cancels, and only ratios inside the group matter, so the terms are
// taken relative to the group's largest logit).  Sums in double by chunked warp scans.  Returns -1 if no term is
// positive (non-finite inputs).
template <typename T>
__device__ __forceinline__ int warp_token_in_range(const GroupsDev &G, const T *trow, int lo, int len, float s, float u_token,
                                                   int lane) {
    // this lane's entry of the first 32 (most groups have no more) stays in registers: token, logit, weight
    const int t0 = lane < len ? G.group_tok[lo + lane] : 0;
    float l0 = kNegInf, w0 = 0.f;
    if (lane < len) {
        l0 = Elem<T>::widen(trow[t0]);
        w0 = G.pair_w ? G.pair_w[lo + lane] : G.inv_deg[t0];
    }
    float mloc = l0;
    for (int k = lane + 32; k < len; k += 32) mloc = fmaxf(mloc, Elem<T>::widen(trow[G.group_tok[lo + k]]));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mloc = fmaxf(mloc, __shfl_xor_sync(0xffffffffu, mloc, o));
    const float rs = mloc > kNegInf ? mloc * s : 0.f;
    auto omega = [&](int k) -> float {
        if (k >= len) return 0.f;
        if (k == lane) return __fmul_rn(ex2(__fmaf_rn(l0, s, -rs)), w0);
        const int t = G.group_tok[lo + k];
        const float w = G.pair_w ? G.pair_w[lo + k] : G.inv_deg[t];
        return __fmul_rn(ex2(__fmaf_rn(Elem<T>::widen(trow[t]), s, -rs)), w);
    };
    double total = 0.0;
    for (int k = lane; k < len; k += 32) total += (double)omega(k);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
    total = __shfl_sync(0xffffffffu, total, 0);  // one value for the whole warp
    const double target = (double)u_token * total;
    double carry = 0.0;
    int pick = -1, last = -1;
    for (int base = 0; base < len && pick < 0; base += 32) {
        const float w = omega(base + lane);
        double inc = (double)w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const double up = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += up;
        }
        const unsigned hit = __ballot_sync(0xffffffffu, w > 0.f && carry + inc > target);
        const unsigned pos = __ballot_sync(0xffffffffu, w > 0.f);
        if (pos) last = base + 31 - __clz(pos);
        if (hit) pick = base + __ffs(hit) - 1;
        carry += __shfl_sync(0xffffffffu, inc, 31);
    }
    const int ksel = pick >= 0 ? pick : last;  // rounding left no prefix above the target: last token with mass
    if (ksel < 0) return -1;
    return ksel < 32 ? __shfl_sync(0xffffffffu, t0, ksel) : G.group_tok[lo + ksel];
}

template <typename T>
__device__ __forceinline__ int warp_token_in_group(const GroupsDev &G, const T *trow, int g, float s, float u_token,
                                                   int lane) {
    const int lo = G.group_ptr[g];
    return warp_token_in_range<T>(G, trow, lo, G.group_ptr[g + 1] - lo, s, u_token, lane);
}

// The same from inside a block-wide code path: warp 0 draws, everybody gets the token (ibox: shared ints).
template <typename T>
__device__ __forceinline__ int block_token_in_group(const GroupsDev &G, const T *trow, int g, float s, float u_token,
                                                    int *ibox, int &flags) {
    if (threadIdx.x < 32) {
        const int zt = warp_token_in_group<T>(G, trow, g, s, u_token, (int)threadIdx.x);
        if (threadIdx.x == 0) ibox[5] = zt;
    }
    __syncthreads();
    const int z = ibox[5];
    if (z >= 0) return z;
    flags |= PCG_FLAG_NONFINITE;  // the drawn group has no token with target mass (non-finite inputs)
    return G.group_ptr[g + 1] > G.group_ptr[g] ? G.group_tok[G.group_ptr[g]] : 0;
}

// Outputs of sequence b: accepted draft tokens, the drawn token z of group gsel at position n, then filler.
template <int NT>
__device__ __forceinline__ void emit_sequence(const GroupsDev &G, int b, int K, int n, int z, int gsel, int flags,
                                              const int32_t *draft_tokens, const int32_t *labels,
                                              int32_t *out_accept_len, int32_t *out_tokens, int32_t *out_groups,
                                              int32_t *out_flags) {
    const int tid = threadIdx.x;
    for (int i = tid; i <= K; i += NT) {
        int tok = -1, grp = -1;
        if (i < n) {
            tok = draft_tokens[b * K + i];
            if (tok < 0 || tok >= G.V) tok = 0;  // verified as token 0 (and flagged), so emitted as token 0
            grp = labels[b * K + i];
        } else if (i == n) {
            tok = z;
            grp = gsel;
        }
        out_tokens[(int64_t)b * (K + 1) + i] = tok;
        if (out_groups) out_groups[(int64_t)b * (K + 1) + i] = grp;
    }
    if (tid == 0) {
        out_accept_len[b] = n;
        if (out_flags) out_flags[b] = flags;
    }
}

struct PickArgs {
    const void *target;
    const int32_t *draft_tokens;
    const float *uniforms;
    int K;
    float s;
    const int32_t *labels;
    const int32_t *term_n;
    const int32_t *term_flags;
    const float4 *term_stats;
    const float *Rt;    // [chunks][M, chunk] group sums of every chunk of sequences
    const float *Psum;  // [chunks][nparts, chunk] per part, the sum of the positive parts of its groups' sums
    int chunk;          // sequences per chunk
    int32_t *out_accept_len;
    int32_t *out_tokens;
    int32_t *out_groups;  // may be null
    int32_t *out_flags;   // may be null
    float *spent;         // scratch no kernel will read again (the transposed operand), or null
    size_t spent_lines;   // its size in 128-byte lines
};

// Group draw from the target's own coarse masses, formed straight from the row (nothing stored): the rare path
// taken when a rejection's residual summed to zero.  Every thread owns a contiguous run of groups; masses are
// formed twice (for the sums, then by the one thread whose run contains the draw).  Returns the group, or -1 if
// no group has mass (non-finite inputs).
template <typename T, int NT>
__device__ __noinline__ int slow_target_group_draw(const GroupsDev &G, const T *trow, float s, float rs, float u_group,
                                                   double *dscratch, int *ibox) {
    const int M = G.M, tid = threadIdx.x;
    const int per = (M + NT - 1) / NT;
    const int i0 = min(M, tid * per), i1 = min(M, i0 + per);
    auto mass = [&](int g) -> float {
        float acc = 0.f;
        for (int k = G.group_ptr[g]; k < G.group_ptr[g + 1]; ++k) {
            const int t = G.group_tok[k];
            const float w = G.pair_w ? G.pair_w[k] : G.inv_deg[t];
            acc += __fmul_rn(ex2(__fmaf_rn(Elem<T>::widen(trow[t]), s, -rs)), w);
        }
        return fmaxf(acc, 0.f);
    };
    double my_sum = 0.0;
    int my_last = -1;
    for (int g = i0; g < i1; ++g) {
        const float v = mass(g);
        my_sum += (double)v;
        if (v > 0.f) my_last = g;
    }
    __syncthreads();
    if (tid == 0) {
        ibox[2] = NT;
        ibox[3] = -1;
        ibox[4] = -1;
    }
    double excl, incl, Ztot;
    block_scan<NT>(my_sum, dscratch, &excl, &incl, &Ztot);  // (its barriers publish the boxes)
    if (!(Ztot > 0.0)) return -1;
    const double target = (double)u_group * Ztot;
    if (my_last >= 0) atomicMax(&ibox[3], my_last);
    if (my_sum > 0.0 && incl > target) atomicMin(&ibox[2], tid);
    __syncthreads();
    if (ibox[2] == tid) {
        double loc = 0.0;
        int pick = my_last;
        for (int g = i0; g < i1; ++g) {
            loc += (double)mass(g);
            if (excl + loc > target) {
                pick = g;
                break;
            }
        }
        ibox[4] = pick;
    }
    __syncthreads();
    return ibox[4] >= 0 ? ibox[4] : ibox[3];
}

// Group and token of one sequence's terminal draw, by the whole block, from the sums of the parts (Ps[p * pstride])
// and of the groups (Rt[g * rstride]).  The cumulative distribution over the groups is walked in two levels: the
// parts' sums (a contiguous run of parts per thread, held in registers; prefix sums in double, block scan), then
// the groups of the one part in which the cumulative mass passes u * Z, by the warp of the thread that owns that
// part, which goes on to draw the token inside the group.  If the sums are all zero after a rejection the group is
// drawn from the target's own masses (rs_target: the scaled reference of the target row) and the sequence flagged.
template <typename T, int NT>
__device__ __forceinline__ void pick_group_and_token(const GroupsDev &G, const T *trow, float s, float rs_target, bool residual,
                                                     float u_group, float u_token, const float *Rt, size_t rstride,
                                                     const float *Ps, size_t pstride, double *dscratch, int *ibox,
                                                     int &flags, int &gsel, int &z) {
    constexpr int PER = 16;  // part sums a thread keeps in registers
    const int NP = G.nparts;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __syncthreads();  // the boxes may still be read from an earlier use
    const int per = (NP + NT - 1) / NT;
    const int p0 = min(NP, tid * per), p1 = min(NP, p0 + per);
    if (tid == 0) {
        ibox[2] = NT;  // selected thread (minimum)
        ibox[3] = -1;  // last part with mass (maximum)
        ibox[4] = -1;  // drawn group
        ibox[5] = -1;  // drawn token
    }
    float v[PER];  // the first PER part sums of this thread's run (all of it unless there are very many parts)
    int pp[PER + 1];  // ... and those parts' group bounds, fetched in the same round trip (one dependent load less later)
#pragma unroll
    for (int j = 0; j < PER; ++j) v[j] = p0 + j < p1 ? Ps[(size_t)(p0 + j) * pstride] : 0.f;
#pragma unroll
    for (int j = 0; j <= PER; ++j) pp[j] = p0 + j <= p1 ? G.part_ptr[p0 + j] : 0;
    double my_sum = 0.0;
    int my_last = -1;  // last part with mass in this thread's run
#pragma unroll
    for (int j = 0; j < PER; ++j) {
        my_sum += (double)v[j];
        if (v[j] > 0.f) my_last = p0 + j;
    }
    for (int p = p0 + PER; p < p1; ++p) {
        const float x = Ps[(size_t)p * pstride];
        my_sum += (double)x;
        if (x > 0.f) my_last = p;
    }
    double my_excl, my_incl, Ztot;
    block_scan<NT>(my_sum, dscratch, &my_excl, &my_incl, &Ztot);  // (its barriers publish the boxes)

    gsel = -1;
    z = -1;
    if (Ztot > 0.0) {
        // ---- group draw: first group whose inclusive prefix exceeds u * Z ----
        const double target = (double)u_group * Ztot;
        if (my_last >= 0) atomicMax(&ibox[3], my_last);
        if (my_sum > 0.0 && my_incl > target) atomicMin(&ibox[2], tid);
        __syncthreads();
        const bool none = ibox[2] == NT;  // rounding left no thread's prefix above the target
        const int owner = none ? 0 : ibox[2];
        if (warp == (owner >> 5)) {
            // the part: the first of the owner's run whose prefix passes the target; if rounding left none, the
            // last part with mass (of the run, or of all parts)
            int part = ibox[3];
            int found = 0, pg0 = -1, pg1 = -1;  // (group bounds of the part, if they are among the prefetched ones)
            double run = my_excl;
            if (tid == owner && !none) {
                part = my_last;
#pragma unroll
                for (int j = 0; j < PER; ++j) {
                    if (!found) {
                        if (v[j] > 0.f && run + (double)v[j] > target) {
                            part = p0 + j;
                            pg0 = pp[j];
                            pg1 = pp[j + 1];
                            found = 1;
                        } else {
                            run += (double)v[j];
                        }
                    }
                }
                for (int p = p0 + PER; p < p1 && !found; ++p) {
                    const float x = Ps[(size_t)p * pstride];
                    if (x > 0.f && run + (double)x > target) {
                        part = p;
                        found = 1;
                    } else {
                        run += (double)x;
                    }
                }
            }
            part = __shfl_sync(0xffffffffu, part, owner & 31);
            found = __shfl_sync(0xffffffffu, found, owner & 31);
            run = __shfl_sync(0xffffffffu, run, owner & 31);
            pg0 = __shfl_sync(0xffffffffu, pg0, owner & 31);
            pg1 = __shfl_sync(0xffffffffu, pg1, owner & 31);
            if (part >= 0) {
                // the group inside it (lane j holds group j of the part): the running sum continues from the parts
                // before; if no prefix passes the target (rounding), the last group with mass
                const int g0 = pg0 >= 0 ? pg0 : G.part_ptr[part];
                const int ng = (pg0 >= 0 ? pg1 : G.part_ptr[part + 1]) - g0;  // at most kPartMaxGroups
                const float r = lane < ng ? fmaxf(Rt[(size_t)(g0 + lane) * rstride], 0.f) : 0.f;
                const int gp = lane <= ng ? G.group_ptr[g0 + lane] : 0;
                int pick = -1, last = -1;
                for (int j = 0; j < ng; ++j) {
                    const float rj = __shfl_sync(0xffffffffu, r, j);
                    if (rj > 0.f) last = j;
                    if (found && pick < 0) {
                        run += (double)rj;
                        if (rj > 0.f && run > target) pick = j;
                    }
                }
                const int j = pick >= 0 ? pick : last;
                if (j >= 0) {
                    const int lo = __shfl_sync(0xffffffffu, gp, j), hi = __shfl_sync(0xffffffffu, gp, j + 1);
                    const int zt = warp_token_in_range<T>(G, trow, lo, hi - lo, s, u_token, lane);
                    if (lane == 0) {
                        ibox[4] = g0 + j;
                        ibox[5] = zt;
                        ibox[6] = hi > lo ? G.group_tok[lo] : 0;  // stand-in if the group has no token with mass
                    }
                }
            }
        }
        __syncthreads();
        gsel = ibox[4];
        z = ibox[5];
        if (gsel >= 0 && z < 0) {  // the drawn group has no token with target mass (non-finite inputs)
            flags |= PCG_FLAG_NONFINITE;
            z = ibox[6];
        }
    } else if (residual) {
        // a rejection whose residual vanished (P == Q to rounding): draw from P instead
        flags |= PCG_FLAG_ZERO_RESIDUAL;
        gsel = slow_target_group_draw<T, NT>(G, trow, s, rs_target, u_group, dscratch, ibox);
        if (gsel >= 0) z = block_token_in_group<T>(G, trow, gsel, s, u_token, ibox, flags);
    }
    if (gsel < 0) {  // no mass anywhere (non-finite inputs): emit group 0 / token 0 and flag it
        gsel = 0;
        z = 0;
        flags |= PCG_FLAG_NONFINITE;
    }
}

// One block per sequence: pick_group_and_token on the sums the sparse product left, then the outputs.
template <typename T>
__global__ void __launch_bounds__(kPickThreads) terminal_pick_kernel(PickArgs a, GroupsDev G) {
    constexpr int NT = kPickThreads;
    __shared__ double dscratch[32];
    __shared__ int ibox[8];
    const int M = G.M, V = G.V, K = a.K, NP = G.nparts;
    const int b = blockIdx.x, tid = threadIdx.x;
    // inputs of the call (not results of the kernels before): fetched before those are waited for
    // (everything read ahead of the wait is read from L2, not through the L1: a line an earlier kernel left in this
    // SM's L1 must not stand in for what was written since)
    const float u_group = __ldcg(a.uniforms + ((int64_t)b * (K + 1) + K) * 2);
    const float u_token = __ldcg(a.uniforms + ((int64_t)b * (K + 1) + K) * 2 + 1);
    // the terminal position and its statistics were left by the transposed-operand kernel, which has completed
    // by the time a block of this kernel runs (the sparse product between the two releases its dependents only
    // after its own wait): read ahead of the wait as well
    const int n = __ldcg(a.term_n + b);
    int flags = __ldcg(a.term_flags + b);
    const float rs_target = __ldcg(&a.term_stats[b].x);
    pdl_enter();
    const T *trow = reinterpret_cast<const T *>(a.target) + ((int64_t)b * (K + 1) + n) * V;
    const int c = b / a.chunk, colb = b - c * a.chunk;
    const size_t cs = (size_t)a.chunk;
    const float *Rt = a.Rt + (size_t)c * M * cs + colb;    // group g of this sequence: Rt[g * chunk]
    const float *Ps = a.Psum + (size_t)c * NP * cs + colb;  // part p of this sequence: Ps[p * chunk]
    int gsel, z;
    pick_group_and_token<T, NT>(G, trow, a.s, rs_target, n < K, u_group, u_token, Rt, cs, Ps, cs, dscratch, ibox, flags, gsel, z);
    emit_sequence<NT>(G, b, K, n, z, gsel, flags, a.draft_tokens, a.labels, a.out_accept_len, a.out_tokens, a.out_groups,
                      a.out_flags);
    // The transposed operand has been consumed (workspace contents are of no interest after the call):
    // dropping its dirty lines from L2 spares the write-back that would otherwise compete with the next call's
    // streaming reads.  Last, so that it does not delay the draw.
    if (a.spent)
        for (size_t l = (size_t)b * NT + tid; l < a.spent_lines; l += (size_t)gridDim.x * NT)
            asm volatile("discard.global.L2 [%0], 128;" ::"l"(a.spent + l * 32) : "memory");
}

struct DrawArgs {
    const void *target;
    const int32_t *draft_tokens;
    const float *uniforms;
    int K;
    float s;
    const int32_t *labels;
    const int32_t *term_n;
    const int32_t *term_flags;
    float *own_rows;   // M too large for shared memory: [B, M] staging rows, else null
    int own_in_smem;   // 1: the M clamped masses of a sequence are staged in shared memory, 0: in global memory
    const float *Pws;  // [B*(K+1), M] target group masses
    const float *Qws;  // [B*K, M] draft group masses
    int32_t *out_accept_len;
    int32_t *out_tokens;
    int32_t *out_groups;  // may be null
    int32_t *out_flags;   // may be null
};

__device__ __forceinline__ int own_slot(int j) { return j + (j >> 5); }  // one pad word per 32: chunked reads spread over banks

// Dense mode: terminal draw from the stored group masses of every position.  One block per sequence.  Shared
// memory: the M clamped residual masses (padded), then scratch.
template <typename T>
__global__ void __launch_bounds__(kDrawThreads) terminal_draw_kernel(DrawArgs a, GroupsDev G) {
    pdl_enter();
    constexpr int NT = kDrawThreads;
    extern __shared__ __align__(16) unsigned char raw[];
    const int M = G.M, V = G.V, K = a.K;
    const int b = blockIdx.x, tid = threadIdx.x;
    // The M clamped masses of the sequence: in (padded) shared memory when they fit, else in a row of global memory;
    // `slot` maps a group to its place.
    const bool in_smem = a.own_in_smem;
    float *own = in_smem ? reinterpret_cast<float *>(raw) : a.own_rows + (size_t)b * M;
    auto slot = [&](int j) { return in_smem ? own_slot(j) : j; };
    unsigned char *tail = raw + (in_smem ? (((size_t)own_slot(M) + 1) * 4 + 15) / 16 * 16 : 0);
    double *dscratch = reinterpret_cast<double *>(tail);      // 32 doubles
    float *scratch = reinterpret_cast<float *>(dscratch + 32);  // 64 floats
    int *ibox = reinterpret_cast<int *>(scratch + 64);          // 8 ints
    const int n = a.term_n[b];
    int flags = a.term_flags[b];
    const T *trow = reinterpret_cast<const T *>(a.target) + ((int64_t)b * (K + 1) + n) * V;
    const float u_group = a.uniforms[((int64_t)b * (K + 1) + K) * 2];
    const float u_token = a.uniforms[((int64_t)b * (K + 1) + K) * 2 + 1];
    bool residual = n < K;  // false: draw from the target's coarse distribution itself (bonus token)
    const float *Pn = a.Pws + ((size_t)b * (K + 1) + n) * M;
    const float *Qn = a.Qws + ((size_t)b * K + min(n, K - 1)) * M;

    const int per = (M + NT - 1) / NT;
    const int i0 = min(M, tid * per), i1 = min(M, i0 + per);
    double Ztot = 0.0, my_excl = 0.0, my_incl = 0.0, my_sum = 0.0;
    int my_last = -1;  // last group with mass in this thread's chunk
    if (tid == 0) {
        ibox[2] = NT;  // selected thread (minimum)
        ibox[3] = -1;  // last group with mass (maximum)
        ibox[4] = -1;  // drawn group
    }
    for (int attempt = 0; attempt < 2; ++attempt) {
        for (int g = tid; g < M; g += NT)
            own[slot(g)] = fmaxf(residual ? Pn[g] - Qn[g] : Pn[g], 0.f);  // (P - Q)_+ ; NaN becomes 0
        __syncthreads();
        // ---- prefix sums over the groups (double): a contiguous chunk per thread, then a block scan ----
        my_sum = 0.0;
        my_last = -1;
        for (int j = i0; j < i1; ++j) {
            const float v = own[slot(j)];
            my_sum += (double)v;
            if (v > 0.f) my_last = j;
        }
        block_scan<NT>(my_sum, dscratch, &my_excl, &my_incl, &Ztot);
        if (Ztot > 0.0 || !residual) break;
        // a rejection whose residual vanished (P == Q to rounding): draw from P instead
        flags |= PCG_FLAG_ZERO_RESIDUAL;
        residual = false;
        __syncthreads();
    }

    // ---- group draw: first group whose inclusive prefix exceeds u * Z ----
    const double target = (double)u_group * Ztot;  // (ibox was initialised before the barriers of the scan)
    if (my_last >= 0) atomicMax(&ibox[3], my_last);
    if (my_sum > 0.0 && my_incl > target) atomicMin(&ibox[2], tid);
    __syncthreads();
    if (ibox[2] == tid) {
        double loc = 0.0;
        int pick = my_last;
        for (int j = i0; j < i1; ++j) {
            loc += (double)own[slot(j)];
            if (my_excl + loc > target) {
                pick = j;
                break;
            }
        }
        ibox[4] = pick;
    }
    __syncthreads();
    int gsel = ibox[4] >= 0 ? ibox[4] : ibox[3];  // rounding left no prefix above the target: last group with mass
    int z = 0;
    if (gsel < 0) {  // no mass anywhere (non-finite inputs): emit group 0 / token 0 and flag it
        gsel = 0;
        flags |= PCG_FLAG_NONFINITE;
    } else {
        z = block_token_in_group<T>(G, trow, gsel, a.s, u_token, ibox, flags);
    }
    emit_sequence<NT>(G, b, K, n, z, gsel, flags, a.draft_tokens, a.labels, a.out_accept_len, a.out_tokens, a.out_groups,
                      a.out_flags);
}

// ---------------------------------------------------------------- dense mode: accept test from full P, Q -----
struct DenseAcceptArgs {
    const int32_t *draft_tokens;
    const float *uniforms;
    int B, K;
    const float *Pws;  // [B*(K+1), M]
    const float *Qws;  // [B*K, M]
    float bias;        // constant added to the acceptance ratio (0 for PCG)
    int32_t *accept, *labels, *posflags;
};

// One thread per drafted position: label draw, then u < min(1, P[g]/Q[g]) on the stored group masses.
__global__ void dense_accept_kernel(DenseAcceptArgs a, GroupsDev G) {
    const int pos = blockIdx.x * blockDim.x + threadIdx.x;
    if (pos >= a.B * a.K) return;
    const int b = pos / a.K, i = pos - b * a.K;
    int x = a.draft_tokens[pos], flag = 0;
    if (x < 0 || x >= G.V) {
        x = 0;
        flag = PCG_FLAG_BAD_DRAFT_TOKEN;
    }
    const float *u = a.uniforms + ((int64_t)b * (a.K + 1) + i) * 2;
    const int r0 = G.rev_ptr[x];
    const int g = draw_label(G, r0, G.rev_ptr[x + 1] - r0, u[0]);
    const float P = a.Pws[((size_t)b * (a.K + 1) + i) * G.M + g], Q = a.Qws[(size_t)pos * G.M + g];
    if (isnan(P) || isnan(Q)) flag |= PCG_FLAG_NONFINITE;
    a.accept[pos] = (P >= Q) || (u[1] * Q < __fmaf_rn(a.bias, Q, P));
    a.labels[pos] = g;
    a.posflags[pos] = flag;
}

// ================================================================ host side ================================

// Launch behind the previous kernel of the stream with programmatic stream serialisation (see pdl_enter).
template <typename... KArgs, typename... Args>
static cudaError_t launch_after(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

static pcg_status check_common(const pcg_groups *groups, pcg_dtype dtype, float temperature, const char *who) {
    if (!groups) {
        set_error("%s: null group handle", who);
        return PCG_ERR_INVALID_ARG;
    }
    if (!valid_dtype(dtype)) {
        set_error("%s: dtype must be PCG_F32, PCG_BF16 or PCG_F16", who);
        return PCG_ERR_INVALID_ARG;
    }
    if (!(temperature >= 1e-6f) || !std::isfinite(temperature)) {
        set_error("%s: temperature must be finite and at least 1e-6", who);
        return PCG_ERR_INVALID_ARG;
    }
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev != groups->device) {
        set_error("%s: the handle lives on device %d but device %d is current", who, groups->device, dev);
        return PCG_ERR_INVALID_ARG;
    }
    return PCG_OK;
}

template <typename Kern, typename Args>
static cudaError_t launch_cluster(Kern kern, int blocks, int cluster, size_t smem, cudaStream_t stream, Args args,
                                  const GroupsDev &G) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3(kAggThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    // (no programmatic stream serialisation here: measured slower with cluster launches, 35 against 31 us per
    // call at B = 64, K = 8, V = 8192)
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, args, G);
}

constexpr size_t kDtBudgetBytes = (size_t)64 << 20;  // Dt of one chunk of sequences must stay inside the L2

// Sequences per lane of the sparse product: 8 (one 256-bit load per token and lane) from 256 sequences on if
// that many fit the budget of the transposed operand, kSpmmWide (4) from 128 on, else 1.
static int spmm_lanes(int B, int V) {
    if (B >= 256 && kDtBudgetBytes / ((size_t)V * 4) >= 256) return 8;
    return B >= 32 * kSpmmWide ? kSpmmWide : 1;
}

// Sequences per chunk of the batched terminal stage: a multiple of what one warp of the sparse product covers
// (32 sequences per lane-sequence).
static int terminal_chunk(int B, int V) {
    const int64_t unit = 32 * spmm_lanes(B, V);
    const int64_t bpad = ((int64_t)B + unit - 1) / unit * unit;
    int64_t fit = (int64_t)(kDtBudgetBytes / ((size_t)V * 4)) / unit * unit;
    if (fit < unit) fit = unit;
    return (int)std::max<int64_t>(unit, fit < bpad ? fit : bpad);
}

static size_t draw_smem_bytes(int M) { return (((size_t)M + (size_t)(M >> 5) + 1) * 4 + 15) / 16 * 16 + 32 * 8 + 64 * 4 + 8 * 4; }

struct VerifyWorkspace {
    int32_t *accept, *labels, *posflags, *term_n, *term_flags, *bonus_flags;
    float4 *stats, *term_stats, *bonus_stats;
    float *Dt, *Rt, *Psum;  // default mode
    float *Pws, *Qws;       // dense mode
    float *own_rows;        // dense mode, M beyond the draw kernel's shared memory
    void *probs_scratch;    // dense mode: scratch of the two group-probability passes
    size_t bytes;
};

static VerifyWorkspace carve_workspace(void *base, int64_t B, int64_t K, int64_t V, int64_t M, uint32_t mode) {
    VerifyWorkspace w = {};
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t at = off;
        off = (off + bytes + 255) & ~(size_t)255;
        return at;
    };
    char *p = (char *)base;
    const int64_t positions = B * K;
    w.stats = (float4 *)(p + take((size_t)positions * 16));
    w.accept = (int32_t *)(p + take((size_t)positions * 4));
    w.labels = (int32_t *)(p + take((size_t)positions * 4));
    w.posflags = (int32_t *)(p + take((size_t)positions * 4));
    w.term_stats = (float4 *)(p + take((size_t)B * 16));
    w.term_n = (int32_t *)(p + take((size_t)B * 4));
    w.term_flags = (int32_t *)(p + take((size_t)B * 4));
    if (mode == PCG_VERIFY_DENSE) {
        w.Pws = (float *)(p + take((size_t)(B * (K + 1) * M) * 4));
        w.Qws = (float *)(p + take((size_t)(B * K * M) * 4));
        if (draw_smem_bytes((int)M) > kMaxDynSmem) w.own_rows = (float *)(p + take((size_t)(B * M) * 4));
        w.probs_scratch = p + take(pcg_group_probs_workspace_bytes((int32_t)V, (int32_t)M));
    } else if (mode != PCG_VERIFY_CLUSTER_TERMINAL) {
        const int64_t chunk = terminal_chunk((int)B, (int)V);
        const int64_t chunks = (B + chunk - 1) / chunk;
        w.bonus_stats = (float4 *)(p + take((size_t)B * 16));
        w.bonus_flags = (int32_t *)(p + take((size_t)B * 4));
        w.Dt = (float *)(p + take((size_t)V * (size_t)chunk * 4));
        w.Rt = (float *)(p + take((size_t)(chunks * chunk * M) * 4));
        w.Psum = (float *)(p + take((size_t)(chunks * chunk * M) * 4));  // (a part holds at least one group)
    }
    w.bytes = off ? off : 256;
    return w;
}

// Threads of a position block: rows of at most 64 KB are streamed by 128 threads (four or more batches per row even
// at V = 16384, so that the dependent-load chain towards the label group stays hidden, and eight blocks per SM).
static int position_threads(int V, pcg_dtype dtype) {
    return (size_t)V * dtype_bytes(dtype) <= kPosSmallRowBytes ? kPosThreadsSmall : kPosThreads;
}
// (Launched with programmatic stream serialisation like the kernels behind it: after whatever precedes the call on
// the stream -- in a decoding loop the previous call's last kernel -- its blocks are scheduled during that kernel's
// drain and wait at the top, pdl_enter, until it has completed.)
static void launch_position(pcg_dtype dtype, const PositionArgs &pa, const GroupsDev &G, int positions, cudaStream_t cs) {
    if (position_threads(G.V, dtype) == kPosThreadsSmall)
        PCG_DISPATCH_DTYPE(dtype, launch_after(position_kernel<LogitT, kPosThreadsSmall>, dim3((unsigned)positions),
                                               dim3(kPosThreadsSmall), 0, cs, pa, G));
    else
        PCG_DISPATCH_DTYPE(dtype, launch_after(position_kernel<LogitT, kPosThreads>, dim3((unsigned)positions),
                                               dim3(kPosThreads), 0, cs, pa, G));
}

// The transposed-operand kernel over nb batches of 32 sequences: two resident blocks per SM, shared out
// over the batches, each walking a run of its batch's rows.
template <typename T>
static cudaError_t launch_transpose(const TransposeArgs &tr, int nb, const GroupsDev &G, int sm_count, cudaStream_t cs) {
    constexpr int ch = 64 / (int)sizeof(T);  // tokens per step of a lane
    const int nsteps = (G.V + ch - 1) / ch;
    // a block's run: at least 4 steps per warp, so that finding the terminal positions is paid for; at most what
    // fills the two block slots of every SM exactly once (at B = 256, V = 65536: 37 blocks per batch, 296 in all;
    // with 32 per batch the kernel ran in 0.86 waves and the call took 2 us longer)
    const int per_batch = std::max(1, std::min((nsteps + 31) / 32, 2 * sm_count / std::max(nb, 1)));
    const dim3 grid((unsigned)per_batch, (unsigned)nb);
    return launch_after(residual_transpose_kernel<T>, grid, dim3(kTrThreads), 0, cs, tr, G);
}

// The sparse product over nb batches of 32 sequences (nb a multiple of `lanes`, the sequences per lane: 8, 4 or 1).
template <bool PSUM>
static cudaError_t launch_spmm(const SpmmArgs &sp, int nb, int lanes, const GroupsDev &G, cudaStream_t cs) {
    const bool has_w = G.pair_w != nullptr;
    const dim3 grid((unsigned)((G.nparts + kSpmmThreads / 32 - 1) / (kSpmmThreads / 32)), (unsigned)(nb / lanes));
    auto go = [&](auto kern) { return launch_after(kern, grid, dim3(kSpmmThreads), 0, cs, sp, G); };
    if (lanes == 8) return has_w ? go(group_spmm_kernel<8, 4, true, PSUM>) : go(group_spmm_kernel<8, 4, false, PSUM>);
    if (lanes == kSpmmWide)
        return has_w ? go(group_spmm_kernel<kSpmmWide, kSpmmDepth, true, PSUM>)
                     : go(group_spmm_kernel<kSpmmWide, kSpmmDepth, false, PSUM>);
    return has_w ? go(group_spmm_kernel<1, 16, true, PSUM>) : go(group_spmm_kernel<1, 16, false, PSUM>);
}

#include "pcg_thinning.cuh"

}  // namespace pcg

using namespace pcg;

namespace pcg {
struct ProbsScratch {
    float4 *stats;  // [probs_stats_rows]
    float *dt;      // [chunk / 32][V][32]
    float *rt;      // [M][chunk] group-major sums of one chunk of rows
    size_t bytes;
};
static ProbsScratch carve_probs_scratch(void *base, int V, int M) {
    const size_t chunk = (size_t)probs_chunk_rows(V);
    ProbsScratch w;
    char *p = (char *)base;
    w.stats = (float4 *)p;
    size_t off = ((size_t)probs_stats_rows(V) * 16 + 255) & ~(size_t)255;
    w.dt = (float *)(p + off);
    off += ((size_t)V * chunk * 4 + 255) & ~(size_t)255;
    w.rt = (float *)(p + off);
    off += ((size_t)M * chunk * 4 + 255) & ~(size_t)255;
    w.bytes = off;
    return w;
}

static pcg_status group_probs_impl(const void *logits, pcg_dtype dtype, int64_t rows, float temperature,
                                   const pcg_groups *groups, float *out, const ProbsScratch *scratch, cudaStream_t cs,
                                   const char *who) {
    pcg_status st = check_common(groups, dtype, temperature, who);
    if (st != PCG_OK) return st;
    if (rows < 0 || (rows > 0 && (!logits || !out))) {
        set_error("%s: null pointer or negative row count", who);
        return PCG_ERR_INVALID_ARG;
    }
    if (rows == 0) return PCG_OK;
    const GroupsDev &G = groups->dev;
    if (rows * (int64_t)G.slices > INT32_MAX) {
        set_error("%s: too many rows for one launch", who);
        return PCG_ERR_UNSUPPORTED;
    }
    const float s = (float)((double)kLog2e / (double)temperature);
    cudaError_t e;
    if (rows >= kProbsBatchedRows || !groups->has_sweep) {
        // many rows: the same transposed-operand / sparse-product kernels as the per-sequence stage of pcg_verify,
        // a chunk of rows at a time through the scratch (row statistics, then p(t) w in place of p - q)
        const int chunk = probs_chunk_rows(G.V);  // a multiple of 128
        const int stats_rows = probs_stats_rows(G.V);
        for (int64_t r0 = 0; r0 < rows; r0 += chunk) {
            const int nr = (int)std::min<int64_t>(chunk, rows - r0);
            const char *base = (const char *)logits + (size_t)r0 * G.V * dtype_bytes(dtype);
            const int64_t rs = r0 % stats_rows;  // this chunk's place in the statistics of its run of chunks
            if (rs == 0) {  // the statistics of the next stats_rows rows, one block per row
                const int ns = (int)std::min<int64_t>(stats_rows, rows - r0);
                PCG_DISPATCH_DTYPE(dtype, e = launch_after(row_stats_kernel<LogitT>, dim3((unsigned)ns), dim3(kPrepThreads), 0, cs,
                                                           (const void *)base, s, scratch->stats, G));
                if (e != cudaSuccess) return cuda_fail(e, "launching row_stats_kernel");
            }
            const int lanes = (chunk % 256 == 0 && nr >= 256) ? 8 : kSpmmWide;      // rows per lane of the sparse product
            const int nb = (nr + 32 * lanes - 1) / (32 * lanes) * lanes;          // batches of 32 rows, whole warps of it
            // every row is "a sequence whose only row is accepted": K = 0 makes the kernel form p alone
            TransposeArgs tr{};
            tr.target = tr.draft = base;
            tr.B = nr;
            tr.s = s;
            tr.from_accept = 2;
            tr.term_stats = scratch->stats + rs;
            tr.Dt = scratch->dt;
            PCG_DISPATCH_DTYPE(dtype, e = launch_transpose<LogitT>(tr, nb, G, groups->sm_count, cs));
            if (e != cudaSuccess) return cuda_fail(e, "launching residual_transpose_kernel");
            e = launch_spmm<false>(SpmmArgs{scratch->dt, nr, 0, chunk, scratch->rt, nullptr}, nb, lanes, G, cs);
            if (e != cudaSuccess) return cuda_fail(e, "launching group_spmm_kernel");
            e = launch_after(rows_from_groups_kernel, dim3((unsigned)((G.M + 31) / 32), (unsigned)((nr + 31) / 32)), dim3(32, 8), 0,
                             cs, (const float *)scratch->rt, chunk, nr, G.M, out + (size_t)r0 * G.M);
            if (e != cudaSuccess) return cuda_fail(e, "launching rows_from_groups_kernel");
        }
        return PCG_OK;
    }
    ProbsArgs a{logits, out, s};
    PCG_DISPATCH_DTYPE(dtype, e = launch_cluster(group_probs_kernel<LogitT>, (int)(rows * G.slices), G.slices,
                                                 groups->agg_smem_bytes, cs, a, G));
    if (e != cudaSuccess) return cuda_fail(e, "launching group_probs_kernel");
    return PCG_OK;
}
}  // namespace pcg

extern "C" pcg_status pcg_group_probs(const void *logits, pcg_dtype dtype, int64_t rows, float temperature,
                                      const pcg_groups *groups, float *out, pcg_stream stream) {
    ProbsScratch own = {};
    if (groups) {  // the scratch that belongs to the handle
        own.stats = groups->probs_stats;
        own.dt = groups->probs_dt;
        own.rt = groups->probs_rt;
    }
    return group_probs_impl(logits, dtype, rows, temperature, groups, out, &own, (cudaStream_t)stream, "pcg_group_probs");
}

extern "C" size_t pcg_group_probs_workspace_bytes(int32_t V, int32_t M) {
    return (V < 1 || M < 1) ? 256 : carve_probs_scratch(nullptr, V, M).bytes;
}

extern "C" pcg_status pcg_group_probs_ws(const void *logits, pcg_dtype dtype, int64_t rows, float temperature,
                                         const pcg_groups *groups, float *out, void *workspace, size_t workspace_bytes,
                                         pcg_stream stream) {
    if (!groups) {
        set_error("pcg_group_probs_ws: null group handle");
        return PCG_ERR_INVALID_ARG;
    }
    const size_t need = pcg_group_probs_workspace_bytes(groups->dev.V, groups->dev.M);
    if (!workspace || ((uintptr_t)workspace & 255u) || workspace_bytes < need) {
        set_error("pcg_group_probs_ws: workspace must be 256-byte aligned and hold %zu bytes (got %zu)", need, workspace_bytes);
        return PCG_ERR_WORKSPACE;
    }
    const ProbsScratch ws = carve_probs_scratch(workspace, groups->dev.V, groups->dev.M);
    return group_probs_impl(logits, dtype, rows, temperature, groups, out, &ws, (cudaStream_t)stream, "pcg_group_probs_ws");
}

extern "C" size_t pcg_verify_workspace_bytes(int32_t B, int32_t K, int32_t V, int32_t M, pcg_dtype dtype,
                                             uint32_t mode) {
    (void)dtype;
    if (B < 0 || K < 0 || V < 1 || M < 1) return 256;
    return carve_workspace(nullptr, B, K, V, M, mode).bytes;
}

extern "C" pcg_status pcg_verify(const void *target_logits, const void *draft_logits, pcg_dtype dtype, int32_t B,
                                 int32_t K, const int32_t *draft_tokens, const pcg_groups *groups,
                                 const float *uniforms, float temperature, int32_t *out_accept_len,
                                 int32_t *out_tokens, int32_t *out_groups, int32_t *out_flags, void *workspace,
                                 size_t workspace_bytes, uint32_t mode, pcg_stream stream,
                                 const pcg_event *stage_events) {
    pcg_status st = check_common(groups, dtype, temperature, "pcg_verify");
    if (st != PCG_OK) return st;
    if (B < 0 || K < 1) {
        set_error("pcg_verify: need B >= 0 and K >= 1 (B=%d K=%d)", B, K);
        return PCG_ERR_INVALID_ARG;
    }
    if (K > 1024) {
        set_error("pcg_verify: K=%d exceeds the supported 1024 drafted positions per sequence", K);
        return PCG_ERR_UNSUPPORTED;
    }
    if (mode != PCG_VERIFY_DEFAULT && mode != PCG_VERIFY_DENSE && mode != PCG_VERIFY_CLUSTER_TERMINAL &&
        mode != PCG_VERIFY_BATCHED_TERMINAL) {
        set_error("pcg_verify: unknown or contradictory mode bits 0x%x", mode);
        return PCG_ERR_INVALID_ARG;
    }
    if (B == 0) return PCG_OK;
    if (!target_logits || !draft_logits || !draft_tokens || !uniforms || !out_accept_len || !out_tokens) {
        set_error("pcg_verify: null pointer");
        return PCG_ERR_INVALID_ARG;
    }
    const GroupsDev &G = groups->dev;
    const size_t esz = dtype_bytes(dtype);
    if (((uintptr_t)target_logits % esz) || ((uintptr_t)draft_logits % esz)) {
        set_error("pcg_verify: logits pointers must be aligned to their element size");
        return PCG_ERR_INVALID_ARG;
    }
    if ((int64_t)B * (K + 1) > INT32_MAX / 8) {
        set_error("pcg_verify: B*K too large for one launch");
        return PCG_ERR_UNSUPPORTED;
    }
    const size_t need = pcg_verify_workspace_bytes(B, K, G.V, G.M, dtype, mode);
    if (!workspace || ((uintptr_t)workspace & 255u) || workspace_bytes < need) {
        set_error("pcg_verify: workspace must be 256-byte aligned and hold %zu bytes (got %zu)", need,
                  workspace_bytes);
        return PCG_ERR_WORKSPACE;
    }
    const bool dense = mode == PCG_VERIFY_DENSE;
    // Default: one cluster per sequence while all clusters are resident in about one wave (a handful of
    // sequences: fewer launches, lower latency), the batched kernels beyond that.
    const bool cluster_terminal = mode == PCG_VERIFY_CLUSTER_TERMINAL ||
                                  (mode == PCG_VERIFY_DEFAULT && groups->has_sweep &&
                                   (int64_t)B * G.slices <= 2 * (int64_t)groups->sm_count);
    if (cluster_terminal && !groups->has_sweep) {
        set_error("pcg_verify: this handle has no sweep layout (M=%d, V=%d), so the cluster terminal is unavailable", G.M,
                  G.V);
        return PCG_ERR_UNSUPPORTED;
    }
    const bool own_in_smem = draw_smem_bytes(G.M) <= kMaxDynSmem;
    const size_t draw_smem = own_in_smem ? draw_smem_bytes(G.M) : 1024;
    cudaStream_t cs = (cudaStream_t)stream;
    const VerifyWorkspace w = carve_workspace(workspace, B, K, G.V, G.M, mode);
    const float s = (float)((double)kLog2e / (double)temperature);
    cudaError_t e = cudaSuccess;
    if (stage_events) e = cudaEventRecord((cudaEvent_t)stage_events[0], cs);
    if (e != cudaSuccess) return cuda_fail(e, "cudaEventRecord");

    // ---- per-position stage: statistics, label, accept bit ----
    if (dense) {
        // P and Q of ALL groups at EVERY position, then the accept test on the stored masses
        const ProbsScratch ps = carve_probs_scratch(w.probs_scratch, G.V, G.M);
        pcg_status st2 = group_probs_impl(target_logits, dtype, (int64_t)B * (K + 1), temperature, groups, w.Pws, &ps, cs, "pcg_verify");
        if (st2 == PCG_OK) st2 = group_probs_impl(draft_logits, dtype, (int64_t)B * K, temperature, groups, w.Qws, &ps, cs, "pcg_verify");
        if (st2 != PCG_OK) return st2;
        DenseAcceptArgs da{draft_tokens, uniforms, B, K, w.Pws, w.Qws, groups->accept_bias, w.accept, w.labels, w.posflags};
        dense_accept_kernel<<<(B * K + 127) / 128, 128, 0, cs>>>(da, G);
        e = cudaGetLastError();
        if (e != cudaSuccess) return cuda_fail(e, "launching dense_accept_kernel");
    } else {
        // (the batched per-sequence stage takes the bonus row's statistics from this kernel)
        PositionArgs pa{target_logits, draft_logits, draft_tokens, uniforms, K, s, groups->accept_bias,
                        w.accept,      w.labels,     w.posflags,   w.stats,  nullptr,
                        cluster_terminal ? nullptr : w.bonus_stats, cluster_terminal ? nullptr : w.bonus_flags, nullptr, 0};
        launch_position(dtype, pa, G, B * K, cs);
        e = cudaGetLastError();
        if (e != cudaSuccess) return cuda_fail(e, "launching position_kernel");
    }
    if (stage_events) {
        e = cudaEventRecord((cudaEvent_t)stage_events[1], cs);
        if (e != cudaSuccess) return cuda_fail(e, "cudaEventRecord");
    }

    // ---- per-sequence stage: first rejection, residual over all groups, group and token draw ----
    if (cluster_terminal) {
        TerminalArgs ta{target_logits, draft_logits, draft_tokens, uniforms,       K,          s,         w.accept,
                        w.labels,      w.posflags,   w.stats,      out_accept_len, out_tokens, out_groups, out_flags};
        PCG_DISPATCH_DTYPE(dtype, e = launch_cluster(terminal_kernel<LogitT>, B * G.slices, G.slices,
                                                     groups->agg_smem_bytes, cs, ta, G));
        if (e != cudaSuccess) return cuda_fail(e, "launching terminal_kernel");
    } else if (dense) {
        PrepareArgs pr{target_logits, K, s, 0, w.accept, w.posflags, w.stats, w.term_n, w.term_flags, w.term_stats};
        PCG_DISPATCH_DTYPE(dtype, launch_after(terminal_prepare_kernel<LogitT>, dim3((unsigned)B), dim3(kPrepThreads), 0, cs, pr, G));
        e = cudaGetLastError();
        if (e != cudaSuccess) return cuda_fail(e, "launching terminal_prepare_kernel");
        DrawArgs dr{target_logits, draft_tokens, uniforms, K, s, w.labels, w.term_n, w.term_flags, w.own_rows,
                    own_in_smem ? 1 : 0, w.Pws, w.Qws, out_accept_len, out_tokens, out_groups, out_flags};
        auto launch_draw = [&](auto kern) -> cudaError_t {
            cudaError_t le = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)draw_smem);
            if (le != cudaSuccess) return le;
            return launch_after(kern, dim3((unsigned)B), dim3(kDrawThreads), draw_smem, cs, dr, G);
        };
        PCG_DISPATCH_DTYPE(dtype, e = launch_draw(terminal_draw_kernel<LogitT>));
        if (e != cudaSuccess) return cuda_fail(e, "launching terminal_draw_kernel");
    } else {
        const int chunk = terminal_chunk(B, G.V);
        const int lanes = spmm_lanes(B, G.V);  // sequences per lane in the sparse product
        for (int b0 = 0, ci = 0; b0 < B; b0 += chunk, ++ci) {
            // batches of 32 sequences in this chunk, rounded up to what one warp of the sparse product reads
            const int unit = 32 * lanes;
            const int nb = (std::min(B - b0, chunk) + unit - 1) / unit * (unit / 32);
            TransposeArgs tr{target_logits, draft_logits, B,        K,         b0,          s,           1,
                             w.accept,      w.posflags,   w.stats,  w.bonus_stats, w.bonus_flags, w.term_n, w.term_flags,
                             w.term_stats,  w.Dt};
            PCG_DISPATCH_DTYPE(dtype, e = launch_transpose<LogitT>(tr, nb, G, groups->sm_count, cs));
            if (e != cudaSuccess) return cuda_fail(e, "launching residual_transpose_kernel");
            e = launch_spmm<true>(SpmmArgs{w.Dt, B, b0, chunk, w.Rt + (size_t)ci * G.M * chunk,
                                            w.Psum + (size_t)ci * G.nparts * chunk},
                                   nb, lanes, G, cs);
            if (e != cudaSuccess) return cuda_fail(e, "launching group_spmm_kernel");
        }
        PickArgs pk{target_logits, draft_tokens, uniforms,   K,          s,         w.labels, w.term_n, w.term_flags, w.term_stats,
                    w.Rt,          w.Psum,       chunk,      out_accept_len, out_tokens, out_groups, out_flags,
                    w.Dt,          (size_t)G.V * (size_t)chunk * 4 / 128};
        PCG_DISPATCH_DTYPE(dtype, e = launch_after(terminal_pick_kernel<LogitT>, dim3((unsigned)B), dim3(kPickThreads), 0, cs, pk, G));
        if (e != cudaSuccess) return cuda_fail(e, "launching terminal_pick_kernel");
    }
    if (stage_events) {
        e = cudaEventRecord((cudaEvent_t)stage_events[2], cs);
        if (e != cudaSuccess) return cuda_fail(e, "cudaEventRecord");
    }
    return PCG_OK;
}

// ================================================================ verification with the thinning sampler ====

namespace pcg {
struct ThinWorkspace {
    int32_t *accept, *labels, *posflags, *exh, *exh_meta;
    float4 *stats, *exh_stats;
    float *fallback_rows, *exh_psum;
    float2 *strata;
    size_t bytes;
};
static ThinWorkspace carve_thin_workspace(void *base, int64_t B, int64_t K, int64_t M) {
    ThinWorkspace w = {};
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t at = off;
        off = (off + bytes + 255) & ~(size_t)255;
        return at;
    };
    char *p = (char *)base;
    w.stats = (float4 *)(p + take((size_t)(B * K) * 16));
    w.accept = (int32_t *)(p + take((size_t)(B * K) * 4));
    w.labels = (int32_t *)(p + take((size_t)(B * K) * 4));
    w.posflags = (int32_t *)(p + take((size_t)(B * K) * 4));
    w.fallback_rows = (float *)(p + take((size_t)(B * M) * 4));
    w.exh_psum = (float *)(p + take((size_t)(B * M) * 4));  // (a part holds at least one group)
    w.exh = (int32_t *)(p + take((size_t)(B + 2) * 4));
    w.exh_meta = (int32_t *)(p + take((size_t)B * 8));
    w.exh_stats = (float4 *)(p + take((size_t)B * 16));
    w.strata = (float2 *)(p + take((size_t)(B * K) * kPosThreads * 8));  // (128 pairs per position are used for short rows)
    w.bytes = off ? off : 256;
    return w;
}
}  // namespace pcg

extern "C" size_t pcg_verify_thinning_workspace_bytes(int32_t B, int32_t K, int32_t V, int32_t M, pcg_dtype dtype) {
    (void)dtype;
    if (B < 0 || K < 0 || V < 1 || M < 1) return 256;
    return carve_thin_workspace(nullptr, B, K, M).bytes;
}

extern "C" pcg_status pcg_verify_thinning(const void *target_logits, const void *draft_logits, pcg_dtype dtype, int32_t B,
                                          int32_t K, const int32_t *draft_tokens, const pcg_groups *groups,
                                          const float *uniforms, const float *thin_uniforms, int32_t n_trials,
                                          float temperature, int32_t *out_accept_len, int32_t *out_tokens,
                                          int32_t *out_groups, int32_t *out_flags, int32_t *out_trials, void *workspace,
                                          size_t workspace_bytes, pcg_stream stream, const pcg_event *stage_events) {
    pcg_status st = check_common(groups, dtype, temperature, "pcg_verify_thinning");
    if (st != PCG_OK) return st;
    if (B < 0 || K < 1 || n_trials < 1) {
        set_error("pcg_verify_thinning: need B >= 0, K >= 1 and n_trials >= 1 (B=%d K=%d n_trials=%d)", B, K, n_trials);
        return PCG_ERR_INVALID_ARG;
    }
    if (K > 1024 || n_trials > 65536) {
        set_error("pcg_verify_thinning: K=%d or n_trials=%d exceeds the supported 1024 positions / 65536 trials", K, n_trials);
        return PCG_ERR_UNSUPPORTED;
    }
    if (B == 0) return PCG_OK;
    if (!target_logits || !draft_logits || !draft_tokens || !uniforms || !thin_uniforms || !out_accept_len || !out_tokens) {
        set_error("pcg_verify_thinning: null pointer");
        return PCG_ERR_INVALID_ARG;
    }
    const GroupsDev &G = groups->dev;
    const size_t esz = dtype_bytes(dtype);
    if (((uintptr_t)target_logits % esz) || ((uintptr_t)draft_logits % esz)) {
        set_error("pcg_verify_thinning: logits pointers must be aligned to their element size");
        return PCG_ERR_INVALID_ARG;
    }
    if ((int64_t)B * (K + 1) > INT32_MAX / 8) {
        set_error("pcg_verify_thinning: B*K too large for one launch");
        return PCG_ERR_UNSUPPORTED;
    }
    const size_t smem = thin_smem_bytes();
    const size_t need = pcg_verify_thinning_workspace_bytes(B, K, G.V, G.M, dtype);
    if (!workspace || ((uintptr_t)workspace & 255u) || workspace_bytes < need) {
        set_error("pcg_verify_thinning: workspace must be 256-byte aligned and hold %zu bytes (got %zu)", need,
                  workspace_bytes);
        return PCG_ERR_WORKSPACE;
    }
    cudaStream_t cs = (cudaStream_t)stream;
    const ThinWorkspace w = carve_thin_workspace(workspace, B, K, G.M);
    const float s = (float)((double)kLog2e / (double)temperature);
    cudaError_t e = cudaSuccess;
    if (stage_events) e = cudaEventRecord((cudaEvent_t)stage_events[0], cs);
    if (e != cudaSuccess) return cuda_fail(e, "cudaEventRecord");
    // Rows that start on 16-byte boundaries and consist of whole 16-byte words: the partial sums the position
    // kernel's threads hold anyway are exactly the slot masses the candidate draw needs (slot of token t =
    // (t div W) mod 128), so the thinning kernel needs no pass of its own over the row.
    const bool strata = ((uintptr_t)target_logits & 15u) == 0 && ((size_t)G.V * esz) % 16 == 0;
    PositionArgs pa{target_logits, draft_logits, draft_tokens, uniforms, K, s, groups->accept_bias,
                    w.accept,      w.labels,     w.posflags,   w.stats,  strata ? w.strata : nullptr, nullptr, nullptr, w.exh, 2};
    launch_position(dtype, pa, G, B * K, cs);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "launching position_kernel");
    if (stage_events) {
        e = cudaEventRecord((cudaEvent_t)stage_events[1], cs);
        if (e != cudaSuccess) return cuda_fail(e, "cudaEventRecord");
    }
    ThinArgs ta{target_logits, draft_logits, draft_tokens, uniforms,        thin_uniforms, n_trials,
                K,             s,            w.accept,     w.labels,        w.posflags,    w.stats,
                w.fallback_rows, out_accept_len, out_tokens, out_groups,    out_flags,     out_trials,
                strata ? w.strata : nullptr, position_threads(G.V, dtype), w.exh, w.exh_stats, w.exh_meta, w.exh_psum,
                n_trials < kEnumBelowTrials ? 1 : 0};
    auto launch = [&](auto kern) -> cudaError_t {
        cudaError_t le = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (le != cudaSuccess) return le;
        return launch_after(kern, dim3((unsigned)B), dim3(kThinThreads), smem, cs, ta, G);
    };
    PCG_DISPATCH_DTYPE(dtype, e = launch(thinning_kernel<LogitT>));
    if (e != cudaSuccess) return cuda_fail(e, "launching thinning_kernel");
    // the shared enumeration for sequences whose trials ran out (returns at once when there is none): only where
    // running out is likely enough to pay for the launch
    if (ta.coop) {
        const dim3 egrid((unsigned)((G.nparts + kEnumThreads / 32 - 1) / (kEnumThreads / 32)));
        PCG_DISPATCH_DTYPE(dtype, e = launch_after(thinning_enumerate_kernel<LogitT>, egrid, dim3(kEnumThreads), 0, cs, ta, G));
        if (e != cudaSuccess) return cuda_fail(e, "launching thinning_enumerate_kernel");
    }
    if (stage_events) {
        e = cudaEventRecord((cudaEvent_t)stage_events[2], cs);
        if (e != cudaSuccess) return cuda_fail(e, "cudaEventRecord");
    }
    return PCG_OK;
}

// ================================================================ verification without caller scratch ======
//
// Built-in scratch of pcg_verify_static: one array per GPU that loads the library, held until the process
// exits.  In host code `g_static_scratch` is only a stand-in for the symbol, never a device address; the
// address a kernel may use comes from cudaGetSymbolAddress, asked once per device and remembered here.
namespace pcg {
constexpr size_t kStaticScratchBytes = (size_t)1 << 20;  // built-in scratch of pcg_verify_static, per GPU
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
constexpr int kMaxStaticDevices = 64;
static void *g_static_scratch_addr[kMaxStaticDevices];  // zero-initialised; written once per device
static std::mutex g_static_scratch_mutex;
}  // namespace pcg

extern "C" pcg_status pcg_verify_static(const void *target_logits, const void *draft_logits, pcg_dtype dtype,
                                        int32_t B, int32_t K, const int32_t *draft_tokens, const pcg_groups *groups,
                                        const float *uniforms, float temperature, int32_t *out_accept_len,
                                        int32_t *out_tokens, int32_t *out_groups, int32_t *out_flags,
                                        pcg_stream stream) {
    if (!groups) {
        set_error("pcg_verify_static: null group handle");
        return PCG_ERR_INVALID_ARG;
    }
    if (B < 0 || K < 1) {
        set_error("pcg_verify_static: need B >= 0 and K >= 1 (B=%d K=%d)", B, K);
        return PCG_ERR_INVALID_ARG;
    }
    if (!groups->has_sweep) {
        set_error("pcg_verify_static: this handle has no sweep layout (M=%d), which the scratch-free mode needs",
                  groups->dev.M);
        return PCG_ERR_UNSUPPORTED;
    }
    const uint32_t mode = PCG_VERIFY_CLUSTER_TERMINAL;  // the mode whose scratch is a few bytes per position
    const size_t need = pcg_verify_workspace_bytes(B, K, groups->dev.V, groups->dev.M, dtype, mode);
    if (need > kStaticScratchBytes) {
        set_error("pcg_verify_static: B=%d, K=%d need %zu bytes of scratch but the built-in array holds %zu "
                  "(about %zu positions); use pcg_verify with a workspace of your own",
                  B, K, need, kStaticScratchBytes, kStaticScratchBytes / 29);
        return PCG_ERR_UNSUPPORTED;
    }
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev < 0 || dev >= kMaxStaticDevices) {
        set_error("pcg_verify_static: device ordinal %d is beyond the %d devices the address table covers", dev,
                  kMaxStaticDevices);
        return PCG_ERR_UNSUPPORTED;
    }
    void *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
        if (!g_static_scratch_addr[dev]) {  // first call on this device: resolve the symbol with it current
            void *addr = nullptr;
            e = cudaGetSymbolAddress(&addr, g_static_scratch);
            if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress (built-in scratch)");
            g_static_scratch_addr[dev] = addr;
        }
        scratch = g_static_scratch_addr[dev];
    }
    // Nothing in the scratch has to start at zero: every field a kernel reads is written earlier in the same call.
    return pcg_verify(target_logits, draft_logits, dtype, B, K, draft_tokens, groups, uniforms, temperature,
                      out_accept_len, out_tokens, out_groups, out_flags, scratch, kStaticScratchBytes, mode, stream,
                      nullptr);
}
