// Kernels and entry points of libpcg: PCG group-level verification on sm_100a.
//
// Two kernels make up pcg_verify:
//   position_kernel  one thread block per drafted position (b,i).  Streams the target and the draft row once
//                    (online max/sum softmax statistics, 128-bit loads), draws the group label of the draft
//                    token, forms the label group's target and draft mass from a handful of gathered logits and
//                    takes the accept decision.  This kernel moves ~all of the bytes.
//   terminal_kernel  one thread-block cluster per sequence.  Finds the first rejected position with a warp
//                    ballot, re-reads that position's rows, builds the residual (P-Q)_+ (or P for the bonus
//                    token) of ALL groups with a token-sliced segmented reduction in shared memory, combines the
//                    slices over distributed shared memory, scans it, draws the group, draws the token inside
//                    it and writes the outputs.
// pcg_group_probs uses the same token-sliced aggregation to write P of every row.
#include <cooperative_groups.h>

#include <algorithm>
#include <cmath>

#include "pcg_common.cuh"

namespace cg = cooperative_groups;

namespace pcg {

constexpr float kLog2e = 1.4426950408889634f;

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
// A block handles one drafted position: its first half streams the target row, its second half the draft row,
// with 128-bit loads issued one batch (kBatch vectors per thread) ahead of the arithmetic.  The chain of
// dependent loads that leads from the draft token to the label group's logits (token -> its groups -> label ->
// group's token list -> logits) is spread over the streaming loop, one hop per batch, so its latency is hidden.

constexpr int kPosThreads = 256;
constexpr int kHalf = kPosThreads / 2;
constexpr int kBatch = 4;
constexpr float kRefInit = -1.0e30f;     // "no logit seen yet": finite, so that -inf logits give 2^-inf = 0, not NaN
constexpr float kVecSumLimit = 4294967296.f;  // 2^32

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
    int32_t *accept;         // [B*K] 1 = accepted
    int32_t *labels;         // [B*K] group label of the draft token
    int32_t *posflags;       // [B*K]
    float4 *stats;           // [B*K] (RS_p, 1/Z_p, RS_q, 1/Z_q): scaled reference and reciprocal normaliser
};

template <typename T>
__global__ void __launch_bounds__(kPosThreads, 4) position_kernel(PositionArgs a, GroupsDev G) {
    constexpr int NT = kPosThreads, H = kHalf, NW = NT / 32, HW = H / 32;
    constexpr int NV = Elem<T>::kPerVec;
    constexpr int U = kBatch;
    constexpr int kChainSteps = 6;
    __shared__ float red_z[2 * NW];
    __shared__ float red_s[NW];
    const int tid = threadIdx.x;
    const int half = tid / H, htid = tid - half * H;  // 0: target row, 1: draft row (warp-uniform)
    const int V = G.V, K = a.K;
    const float s = a.s;
    const int pos = blockIdx.x;
    const int b = pos / K, i = pos - b * K;
    const T *row = half ? reinterpret_cast<const T *>(a.draft) + (int64_t)pos * V
                        : reinterpret_cast<const T *>(a.target) + ((int64_t)b * (K + 1) + i) * V;
    const float *u = a.uniforms + ((int64_t)b * (K + 1) + i) * 2;

    // ---- dependent-load chain towards the label group's logits (every thread, redundantly) ----
    int c_x = 0, c_r0 = 0, c_n = 1, c_g = 0, c_lo = 0, c_hi = 0, c_t = 0, c_flag = 0;
    float c_u0 = 0.f, c_u1 = 0.f, c_l = kNegInf, c_w = 0.f;
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
            case 2: {
                // group-label coupling: the label is drawn from the groups of the draft token
                int j;
                if (!G.rev_w) {
                    j = (int)floor((double)c_u0 * (double)c_n);  // exact: float times small integer in double
                    j = min(max(j, 0), c_n - 1);
                } else {
                    double tot = 0.0, run = 0.0;
                    for (int e = 0; e < c_n; ++e) tot += (double)G.rev_w[c_r0 + e];
                    const double target = (double)c_u0 * tot;
                    j = -1;
                    int last_pos = 0;
                    for (int e = 0; e < c_n; ++e) {
                        const double w = (double)G.rev_w[c_r0 + e];
                        if (w > 0.0) last_pos = e;
                        run += w;
                        if (run > target) {
                            j = e;
                            break;
                        }
                    }
                    if (j < 0) j = last_pos;
                }
                c_g = G.rev_grp[c_r0 + j];
                break;
            }
            case 3:
                c_lo = G.group_ptr[c_g];
                c_hi = G.group_ptr[c_g + 1];
                break;
            case 4:
                if (c_lo + htid < c_hi) c_t = G.group_tok[c_lo + htid];
                break;
            case 5:
                if (c_lo + htid < c_hi) {
                    c_l = Elem<T>::widen(row[c_t]);
                    c_w = G.pair_w ? G.pair_w[c_lo + htid] : G.inv_deg[c_t];
                }
                break;
        }
    };

    // ---- stream the row: elements before the first 16-byte boundary, whole vectors, the rest ----
    RefSum st{kRefInit * s, 0.f};
    int chained = 0;
    int head = (int)(((16u - (unsigned)((uintptr_t)row & 15u)) & 15u) / sizeof(T));
    if (head > V) head = V;
    const int nvec = (V - head) / NV;
    const int nfull = nvec / (H * U);  // batches in which every thread has all U vectors
    {
        const uint4 *p = reinterpret_cast<const uint4 *>(row + head) + htid;
        uint4 cur[U], nxt[U];
        if (nfull > 0) {
#pragma unroll
            for (int j = 0; j < U; ++j) cur[j] = ld_stream(p + j * H);
        }
        for (int bi = 0; bi < nfull; ++bi) {
            p += H * U;
            if (bi + 1 < nfull) {
#pragma unroll
                for (int j = 0; j < U; ++j) nxt[j] = ld_stream(p + j * H);
            }
            if (chained < kChainSteps) chain(chained++);
#pragma unroll
            for (int j = 0; j < U; ++j) {
                float v[NV];
                Elem<T>::unpack(cur[j], v);
                absorb<NV>(st, v, s);
            }
#pragma unroll
            for (int j = 0; j < U; ++j) cur[j] = nxt[j];
        }
        // remaining whole vectors (fewer than H*U), then the scalar head and tail
        for (int idx = nfull * H * U + htid; idx < nvec; idx += H) {
            float v[NV];
            Elem<T>::unpack(ld_stream(reinterpret_cast<const uint4 *>(row + head) + idx), v);
            absorb<NV>(st, v, s);
        }
        for (int t = htid; t < head; t += H) absorb1(st, Elem<T>::widen(row[t]), s);
        for (int t = head + nvec * NV + htid; t < V; t += H) absorb1(st, Elem<T>::widen(row[t]), s);
    }
    while (chained < kChainSteps) chain(chained++);

    // ---- per-row (rs, Z): xor butterfly inside a warp, then a fixed-order pass over each half's warps ----
    float rs = st.rs, Z = st.acc;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) merge(rs, Z, __shfl_xor_sync(0xffffffffu, rs, o), __shfl_xor_sync(0xffffffffu, Z, o));
    if ((tid & 31) == 0) {
        red_z[2 * (tid >> 5)] = rs;
        red_z[2 * (tid >> 5) + 1] = Z;
    }
    __syncthreads();
    float rs_p = red_z[0], Zp = red_z[1], rs_q = red_z[2 * HW], Zq = red_z[2 * HW + 1];
#pragma unroll
    for (int w = 1; w < HW; ++w) {
        merge(rs_p, Zp, red_z[2 * w], red_z[2 * w + 1]);
        merge(rs_q, Zq, red_z[2 * (HW + w)], red_z[2 * (HW + w) + 1]);
    }

    // ---- mass of the label group under this half's row (first element prefetched by the chain) ----
    const float rs_mine = half ? rs_q : rs_p;
    float part = __fmul_rn(ex2(__fmaf_rn(c_l, s, -rs_mine)), c_w);
    for (int k = c_lo + htid + H; k < c_hi; k += H) {  // groups larger than half a block
        const int t = G.group_tok[k];
        const float w = G.pair_w ? G.pair_w[k] : G.inv_deg[t];
        part += __fmul_rn(ex2(__fmaf_rn(Elem<T>::widen(row[t]), s, -rs_mine)), w);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
    if ((tid & 31) == 0) red_s[tid >> 5] = part;
    __syncthreads();

    if (tid == 0) {
        float Sp = red_s[0], Sq = red_s[HW];
        for (int w = 1; w < HW; ++w) {
            Sp += red_s[w];
            Sq += red_s[HW + w];
        }
        // acceptance u < min(1, P/Q) without a division: P = Sp/Zp, Q = Sq/Zq
        const float lhs = Sp * Zq, rhs = Sq * Zp;
        const int acc = (lhs >= rhs) || (c_u1 * rhs < lhs);
        int flag = c_flag;
        if (!(Zp > 0.f) || !(Zq > 0.f) || isinf(Zp) || isinf(Zq) || isinf(rs_p) || isinf(rs_q))
            flag |= PCG_FLAG_NONFINITE;
        a.accept[pos] = acc;
        a.labels[pos] = c_g;
        a.posflags[pos] = flag;
        a.stats[pos] = make_float4(rs_p, 1.0f / Zp, rs_q, 1.0f / Zq);
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
    constexpr int NT = kAggThreads;
    extern __shared__ __align__(16) unsigned char raw[];
    AggSmem sm = carve_smem(raw, G);
    cg::cluster_group cluster = cg::this_cluster();
    const int C = G.slices, K = a.K, V = G.V, M = G.M;
    const int c = (int)cluster.block_rank();
    const int b = blockIdx.x / C;
    const int tid = threadIdx.x;

    // ---- first rejected position: one ballot over the K <= 32 accept bits ----
    if (tid < 32) {
        const int rej = (tid < K) && (a.accept[b * K + tid] == 0);
        const unsigned mask = __ballot_sync(0xffffffffu, rej);
        const int n = mask ? (__ffs(mask) - 1) : K;
        const int f = (tid < K && tid <= n) ? a.posflags[b * K + tid] : 0;
        const int flags = __reduce_or_sync(0xffffffffu, f);
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
        if (tid <= K) {
            int tok = -1, grp = -1;
            if (tid < n) {
                tok = a.draft_tokens[b * K + tid];
                if (tok < 0 || tok >= V) tok = 0;  // verified as token 0 (and flagged), so emitted as token 0
                grp = a.labels[b * K + tid];
            } else if (tid == n) {
                tok = z;
                grp = gsel;
            }
            a.out_tokens[(int64_t)b * (K + 1) + tid] = tok;
            if (a.out_groups) a.out_groups[(int64_t)b * (K + 1) + tid] = grp;
        }
        if (tid == 0) {
            a.out_accept_len[b] = n;
            if (a.out_flags) a.out_flags[b] = flags;
        }
    }
    cluster.sync();  // no block may exit while another still reads its shared memory
}

// ================================================================ host side ================================

static pcg_status check_common(const pcg_groups *groups, pcg_dtype dtype, float temperature, const char *who) {
    if (!groups) {
        set_error("%s: null group handle", who);
        return PCG_ERR_INVALID_ARG;
    }
    if (dtype != PCG_F32 && dtype != PCG_BF16) {
        set_error("%s: dtype must be PCG_F32 or PCG_BF16", who);
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
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, args, G);
}

struct VerifyWorkspace {
    int32_t *accept, *labels, *posflags;
    float4 *stats;
    size_t bytes;
};

static VerifyWorkspace carve_workspace(void *base, int64_t positions) {
    VerifyWorkspace w;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t at = off;
        off = (off + bytes + 255) & ~(size_t)255;
        return at;
    };
    char *p = (char *)base;
    w.stats = (float4 *)(p + take((size_t)positions * 16));
    w.accept = (int32_t *)(p + take((size_t)positions * 4));
    w.labels = (int32_t *)(p + take((size_t)positions * 4));
    w.posflags = (int32_t *)(p + take((size_t)positions * 4));
    w.bytes = off ? off : 256;
    return w;
}

}  // namespace pcg

using namespace pcg;

extern "C" pcg_status pcg_group_probs(const void *logits, pcg_dtype dtype, int64_t rows, float temperature,
                                      const pcg_groups *groups, float *out, pcg_stream stream) {
    pcg_status st = check_common(groups, dtype, temperature, "pcg_group_probs");
    if (st != PCG_OK) return st;
    if (rows < 0 || (rows > 0 && (!logits || !out))) {
        set_error("pcg_group_probs: null pointer or negative row count");
        return PCG_ERR_INVALID_ARG;
    }
    if (rows == 0) return PCG_OK;
    const GroupsDev &G = groups->dev;
    if (rows * (int64_t)G.slices > INT32_MAX) {
        set_error("pcg_group_probs: too many rows for one launch");
        return PCG_ERR_UNSUPPORTED;
    }
    ProbsArgs a{logits, out, (float)((double)kLog2e / (double)temperature)};
    cudaError_t e;
    if (dtype == PCG_F32)
        e = launch_cluster(group_probs_kernel<float>, (int)(rows * G.slices), G.slices, groups->agg_smem_bytes,
                           (cudaStream_t)stream, a, G);
    else
        e = launch_cluster(group_probs_kernel<uint16_t>, (int)(rows * G.slices), G.slices, groups->agg_smem_bytes,
                           (cudaStream_t)stream, a, G);
    if (e != cudaSuccess) return cuda_fail(e, "launching group_probs_kernel");
    return PCG_OK;
}

extern "C" size_t pcg_verify_workspace_bytes(int32_t B, int32_t K, int32_t V, int32_t M, pcg_dtype dtype,
                                             uint32_t mode) {
    (void)V;
    (void)M;
    (void)dtype;
    (void)mode;
    if (B < 0 || K < 0) return 256;
    return carve_workspace(nullptr, (int64_t)B * K).bytes;
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
    if (K > 32) {
        set_error("pcg_verify: K=%d exceeds the 32 positions one ballot covers", K);
        return PCG_ERR_UNSUPPORTED;
    }
    if (mode & ~PCG_VERIFY_DENSE) {
        set_error("pcg_verify: unknown mode bits 0x%x", mode);
        return PCG_ERR_INVALID_ARG;
    }
    if (B == 0) return PCG_OK;
    if (!target_logits || !draft_logits || !draft_tokens || !uniforms || !out_accept_len || !out_tokens) {
        set_error("pcg_verify: null pointer");
        return PCG_ERR_INVALID_ARG;
    }
    const GroupsDev &G = groups->dev;
    const size_t esz = dtype == PCG_F32 ? 4 : 2;
    if (((uintptr_t)target_logits % esz) || ((uintptr_t)draft_logits % esz)) {
        set_error("pcg_verify: logits pointers must be aligned to their element size");
        return PCG_ERR_INVALID_ARG;
    }
    if ((int64_t)B * K > INT32_MAX / 8) {
        set_error("pcg_verify: B*K too large for one launch");
        return PCG_ERR_UNSUPPORTED;
    }
    const size_t need = pcg_verify_workspace_bytes(B, K, G.V, G.M, dtype, mode);
    if (!workspace || ((uintptr_t)workspace & 255u) || workspace_bytes < need) {
        set_error("pcg_verify: workspace must be 256-byte aligned and hold %zu bytes (got %zu)", need,
                  workspace_bytes);
        return PCG_ERR_WORKSPACE;
    }
    if (mode & PCG_VERIFY_DENSE) {
        set_error("pcg_verify: dense mode is not built yet");
        return PCG_ERR_UNSUPPORTED;
    }
    cudaStream_t cs = (cudaStream_t)stream;
    const VerifyWorkspace w = carve_workspace(workspace, (int64_t)B * K);
    const float s = (float)((double)kLog2e / (double)temperature);
    cudaError_t e = cudaSuccess;
    if (stage_events) e = cudaEventRecord((cudaEvent_t)stage_events[0], cs);
    if (e != cudaSuccess) return cuda_fail(e, "cudaEventRecord");

    PositionArgs pa{target_logits, draft_logits, draft_tokens, uniforms, K, s, w.accept, w.labels, w.posflags, w.stats};
    if (dtype == PCG_F32)
        position_kernel<float><<<B * K, kPosThreads, 0, cs>>>(pa, G);
    else
        position_kernel<uint16_t><<<B * K, kPosThreads, 0, cs>>>(pa, G);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "launching position_kernel");
    if (stage_events) {
        e = cudaEventRecord((cudaEvent_t)stage_events[1], cs);
        if (e != cudaSuccess) return cuda_fail(e, "cudaEventRecord");
    }

    TerminalArgs ta{target_logits, draft_logits, draft_tokens, uniforms,       K,          s,         w.accept,
                    w.labels,      w.posflags,   w.stats,      out_accept_len, out_tokens, out_groups, out_flags};
    if (dtype == PCG_F32)
        e = launch_cluster(terminal_kernel<float>, B * G.slices, G.slices, groups->agg_smem_bytes, cs, ta, G);
    else
        e = launch_cluster(terminal_kernel<uint16_t>, B * G.slices, G.slices, groups->agg_smem_bytes, cs, ta, G);
    if (e != cudaSuccess) return cuda_fail(e, "launching terminal_kernel");
    if (stage_events) {
        e = cudaEventRecord((cudaEvent_t)stage_events[2], cs);
        if (e != cudaSuccess) return cuda_fail(e, "cudaEventRecord");
    }
    return PCG_OK;
}
