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

#include <cmath>

#include "pcg_common.cuh"

namespace cg = cooperative_groups;

namespace pcg {

constexpr int kPosThreads = 256;
constexpr float kLog2e = 1.4426950408889634f;

// ================================================================ position kernel ==========================
//
// Per row the kernel needs Z = sum_t 2^(l_t*s - RS) for SOME reference RS (any value works as long as the same
// RS is used for the group masses: it cancels in P = S/Z), so each thread keeps a lazy reference: the largest
// logit of its first vector, raised only when a later logit exceeds it by more than 32/s (a factor 2^32 of
// headroom).  After the first vector the rescale branch is practically never taken, which keeps the special-
// function unit at exactly one ex2 per logit.  Logits travel global -> shared through a per-thread ring of
// 16-byte cp.async copies (kStages deep) so that many loads stay in flight without holding registers.

constexpr int kStages = 8;
constexpr float kRefInit = -1.0e30f;  // "no logit seen yet"; finite so that -inf logits give 2^-inf = 0, not NaN

struct RefSum {
    float r;    // raw-logit reference
    float rs;   // r * s as computed once (the exponent actually subtracted)
    float thr;  // r + 32/s: logits above this raise the reference
    float acc;  // sum of 2^(l*s - rs)
};

__device__ __forceinline__ void raise_ref(RefSum &st, float vm, float s, float headroom) {
    const float nrs = vm * s;
    st.acc *= ex2(st.rs - nrs);
    st.r = vm;
    st.rs = nrs;
    st.thr = vm + headroom;
}

template <int NV>
__device__ __forceinline__ void absorb(RefSum &st, const float (&v)[NV], float s, float headroom) {
    float vm = v[0];
#pragma unroll
    for (int i = 1; i < NV; ++i) vm = fmaxf(vm, v[i]);
    if (vm > st.thr) raise_ref(st, vm, s, headroom);
#pragma unroll
    for (int i = 0; i < NV; ++i) st.acc += ex2(__fmaf_rn(v[i], s, -st.rs));
}

__device__ __forceinline__ void absorb1(RefSum &st, float l, float s, float headroom) {
    if (l > st.thr) raise_ref(st, l, s, headroom);
    st.acc += ex2(__fmaf_rn(l, s, -st.rs));
}

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src) {
    const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// Where the 16-byte vectors of a row start and how many there are.
template <typename T>
struct RowSplit {
    int head, nvec;
    const uint4 *vp;
    __device__ __forceinline__ RowSplit(const T *row, int V) {
        head = (int)(((16u - (unsigned)((uintptr_t)row & 15u)) & 15u) / sizeof(T));
        if (head > V) head = V;
        nvec = (V - head) / Elem<T>::kPerVec;
        vp = reinterpret_cast<const uint4 *>(row + head);
    }
};

// Deterministic block-wide combine of (rs, acc) pairs of TWO rows at once: xor butterfly inside a warp, then a
// fixed-order pass over the warps.  `scratch` holds 4*NWARPS floats.  Every thread returns the same values.
__device__ __forceinline__ void merge(float &rs, float &acc, float rs2, float acc2) {
    const float m = fmaxf(rs, rs2);
    acc = acc * ex2(rs - m) + acc2 * ex2(rs2 - m);
    rs = m;
}

template <int NT>
__device__ __forceinline__ void block_combine2(float &rs_a, float &acc_a, float &rs_b, float &acc_b, float *scratch) {
    constexpr int NW = NT / 32;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        merge(rs_a, acc_a, __shfl_xor_sync(0xffffffffu, rs_a, o), __shfl_xor_sync(0xffffffffu, acc_a, o));
        merge(rs_b, acc_b, __shfl_xor_sync(0xffffffffu, rs_b, o), __shfl_xor_sync(0xffffffffu, acc_b, o));
    }
    __syncthreads();
    if ((threadIdx.x & 31) == 0) {
        float *p = scratch + 4 * (threadIdx.x >> 5);
        p[0] = rs_a, p[1] = acc_a, p[2] = rs_b, p[3] = acc_b;
    }
    __syncthreads();
    rs_a = scratch[0], acc_a = scratch[1], rs_b = scratch[2], acc_b = scratch[3];
#pragma unroll
    for (int w = 1; w < NW; ++w) {
        merge(rs_a, acc_a, scratch[4 * w], scratch[4 * w + 1]);
        merge(rs_b, acc_b, scratch[4 * w + 2], scratch[4 * w + 3]);
    }
}

template <int NT>
__device__ __forceinline__ void block_sum2(float &a, float &b, float *scratch) {
    constexpr int NW = NT / 32;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        a += __shfl_xor_sync(0xffffffffu, a, o);
        b += __shfl_xor_sync(0xffffffffu, b, o);
    }
    __syncthreads();
    if ((threadIdx.x & 31) == 0) {
        scratch[2 * (threadIdx.x >> 5)] = a;
        scratch[2 * (threadIdx.x >> 5) + 1] = b;
    }
    __syncthreads();
    a = scratch[0], b = scratch[1];
#pragma unroll
    for (int w = 1; w < NW; ++w) a += scratch[2 * w], b += scratch[2 * w + 1];
}

struct PositionArgs {
    const void *target;      // [B, K+1, V]
    const void *draft;       // [B, K, V]
    const int32_t *draft_tokens;  // [B, K]
    const float *uniforms;   // [B, K+1, 2]
    int K;
    float s;                 // log2(e) / temperature
    float headroom;          // 32 / s
    int32_t *accept;         // [B*K] 1 = accepted
    int32_t *labels;         // [B*K] group label of the draft token
    int32_t *posflags;       // [B*K]
    float4 *stats;           // [B*K] (RS_p, 1/Z_p, RS_q, 1/Z_q): scaled reference and reciprocal normaliser
};

template <typename T>
__global__ void __launch_bounds__(kPosThreads, 5) position_kernel(PositionArgs a, GroupsDev G) {
    constexpr int NT = kPosThreads;
    constexpr int NV = Elem<T>::kPerVec;
    constexpr int S = kStages;
    __shared__ uint4 ring[S][NT];
    __shared__ float scratch[4 * (NT / 32)];
    __shared__ int sh_label, sh_flag;
    const int tid = threadIdx.x;
    const int pos = blockIdx.x;
    const int b = pos / a.K, i = pos - b * a.K;
    const int V = G.V;
    const T *trow = reinterpret_cast<const T *>(a.target) + ((int64_t)b * (a.K + 1) + i) * V;
    const T *qrow = reinterpret_cast<const T *>(a.draft) + (int64_t)pos * V;
    const float *u = a.uniforms + ((int64_t)b * (a.K + 1) + i) * 2;
    const float s = a.s, headroom = a.headroom;

    // ---- start streaming: the two rows form one sequence of 2*nk vector slots per thread ----
    const RowSplit<T> ts(trow, V), qs(qrow, V);
    const int nk_t = (ts.nvec + NT - 1) / NT, nk_q = (qs.nvec + NT - 1) / NT, nk = nk_t + nk_q;
    auto issue = [&](int k) {
        if (k < nk) {
            const bool second = k >= nk_t;
            const int idx = tid + (second ? k - nk_t : k) * NT;
            if (idx < (second ? qs.nvec : ts.nvec)) cp_async16(&ring[k % S][tid], (second ? qs.vp : ts.vp) + idx);
        }
        cp_async_commit();
    };
#pragma unroll
    for (int k = 0; k < S - 1; ++k) issue(k);

    if (tid == 0) {
        // group-label coupling: the label is drawn from the groups of the draft token with its split weights
        int x = a.draft_tokens[pos], flag = 0;
        if (x < 0 || x >= V) {
            x = 0;
            flag = PCG_FLAG_BAD_DRAFT_TOKEN;
        }
        const int r0 = G.rev_ptr[x], N = G.rev_ptr[x + 1] - r0;
        int j;
        if (!G.rev_w) {
            j = (int)floor((double)u[0] * (double)N);  // exact: a float times a small integer fits a double
            j = min(max(j, 0), N - 1);
        } else {
            double tot = 0.0, run = 0.0;
            for (int e = 0; e < N; ++e) tot += (double)G.rev_w[r0 + e];
            const double target = (double)u[0] * tot;
            j = -1;
            int last_pos = 0;
            for (int e = 0; e < N; ++e) {
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
        sh_label = G.rev_grp[r0 + j];
        sh_flag = flag;
    }

    RefSum st_t{kRefInit, kRefInit * s, kRefInit, 0.f}, st_q = st_t;
    for (int k = 0; k < nk; ++k) {
        issue(k + S - 1);
        cp_async_wait<S - 1>();
        const bool second = k >= nk_t;
        const int idx = tid + (second ? k - nk_t : k) * NT;
        if (idx < (second ? qs.nvec : ts.nvec)) {
            float v[NV];
            Elem<T>::unpack(ring[k % S][tid], v);
            if (second)
                absorb<NV>(st_q, v, s, headroom);
            else
                absorb<NV>(st_t, v, s, headroom);
        }
    }
    // elements before the first and after the last whole 16-byte vector of each row
    for (int t = tid; t < ts.head; t += NT) absorb1(st_t, Elem<T>::widen(trow[t]), s, headroom);
    for (int t = ts.head + ts.nvec * NV + tid; t < V; t += NT) absorb1(st_t, Elem<T>::widen(trow[t]), s, headroom);
    for (int t = tid; t < qs.head; t += NT) absorb1(st_q, Elem<T>::widen(qrow[t]), s, headroom);
    for (int t = qs.head + qs.nvec * NV + tid; t < V; t += NT) absorb1(st_q, Elem<T>::widen(qrow[t]), s, headroom);

    float rs_p = st_t.rs, Zp = st_t.acc, rs_q = st_q.rs, Zq = st_q.acc;
    block_combine2<NT>(rs_p, Zp, rs_q, Zq, scratch);  // its barriers also publish sh_label

    // ---- masses of the label group under both rows: a handful of gathered logits ----
    const int g = sh_label;
    const int lo = G.group_ptr[g], hi = G.group_ptr[g + 1];
    float Sp = 0.f, Sq = 0.f;
    for (int k = lo + tid; k < hi; k += NT) {
        const int t = G.group_tok[k];
        const float w = G.pair_w ? G.pair_w[k] : G.inv_deg[t];
        Sp += __fmul_rn(ex2(__fmaf_rn(Elem<T>::widen(trow[t]), s, -rs_p)), w);
        Sq += __fmul_rn(ex2(__fmaf_rn(Elem<T>::widen(qrow[t]), s, -rs_q)), w);
    }
    block_sum2<NT>(Sp, Sq, scratch);

    if (tid == 0) {
        // acceptance u < min(1, P/Q) without a division: P = Sp/Zp, Q = Sq/Zq
        const float lhs = Sp * Zq, rhs = Sq * Zp;
        const int acc = (lhs >= rhs) || (u[1] * rhs < lhs);
        int flag = sh_flag;
        if (!(Zp > 0.f) || !(Zq > 0.f) || isinf(Zp) || isinf(Zq) || isinf(rs_p) || isinf(rs_q))
            flag |= PCG_FLAG_NONFINITE;
        a.accept[pos] = acc;
        a.labels[pos] = g;
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

    PositionArgs pa{target_logits, draft_logits, draft_tokens, uniforms, K,       s,
                    32.0f / s,     w.accept,     w.labels,     w.posflags, w.stats};
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
