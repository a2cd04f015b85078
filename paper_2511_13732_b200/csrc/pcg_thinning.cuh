// Terminal group by thinning (the thinning paragraph of Sec. 2.2) -- included by pcg_kernels.cu inside
// namespace pcg, after the helpers of the batched terminal stage.
//
// The paper's sampler never enumerates the groups: a candidate (y, k) is drawn with y ~ target and k ~ w_{.,y}
// (so k follows the target's coarse distribution) and kept with probability [1 - Q(k)/P(k)]_+, which needs the
// two masses of group k only.  The candidate token is drawn by inverse CDF over the tokens taken slot by slot:
// the slot of token t is (t div W) mod 128, W = logits per 16 bytes, tokens ascending inside a slot.  That is the
// order in which the position kernel's 128 target-row threads sum the row, so the 128 slot masses are a free
// by-product of that kernel and no pass over the row is needed here.  One block per sequence:
//   1. first rejection n from the accept bits (warp ballots); row statistics from the position kernel, or, when
//      every position was accepted, one pass over the bonus row;
//   2. the 128 slot masses of the target row of position n -- from the position kernel's threads, or (bonus row,
//      rows that are not made of aligned 16-byte words) summed here -- and their inclusive prefix in double;
//   3. trials, one WARP per trial and all warps at once: binary search for the slot, scan of the slot's words
//      (32 at a time, 2 KB apart) for y, label k, the two masses of group k by a warp gather, keep test, token
//      inside a kept group.  The first kept candidate in trial order wins, so the result is the sequential
//      sampler's although several trials run side by side;
//   4. outputs.
// If all supplied trials of a sequence are turned down, the residual is enumerated after all and the group drawn
// from it with the sequence's terminal-group uniform: same law, flagged PCG_FLAG_THINNING_EXHAUSTED.  Calls with
// many supplied trials (where that is rare) do it in the sequence's own block (one thread per group, staged in a
// row of the workspace: 0.47 ms at C5).  Calls with fewer than kEnumBelowTrials trials run thinning_enumerate_kernel
// behind this kernel (an empty launch costs them about 3 us): the exhausted sequences are put on a list and
// enumerated by ALL its blocks (a warp per part of the groups, as in the sparse product): 15 us for one.

constexpr int kThinThreads = 512;
constexpr int kEnumBelowTrials = 24;  // that kernel is launched for calls with fewer supplied trials than this

struct ThinArgs {
    const void *target;           // [B, K+1, V]
    const void *draft;            // [B, K, V]
    const int32_t *draft_tokens;  // [B, K]
    const float *uniforms;        // [B, K+1, 2]
    const float *thin;            // [B, n_trials, 3]: token, label and keep uniform of every trial
    int n_trials;
    int K;
    float s;
    const int32_t *accept, *labels, *posflags;  // [B*K] from the position kernel
    const float4 *stats;                        // [B*K]
    float *fallback_rows;                       // [B, M] staging for sequences whose trials ran out
    int32_t *out_accept_len, *out_tokens, *out_groups, *out_flags, *out_trials;
    const float2 *strata;  // [B*K, strata_threads] (reference, sum) of every thread of the position kernel's target-row pass, or null
    int strata_threads;    // threads of a position block: kThinSlots or 2 * kThinSlots
    // Sequences whose trials all failed are handed to thinning_enumerate_kernel (below) through these:
    int32_t *exh;          // [2 + B], [0] and [1] zero on entry: [0] how many, [1] blocks of that kernel that are done,
                           // [2 + j] the j-th such sequence
    float4 *exh_stats;     // [B] (RS_p, 1/Z_p, RS_q, 1/Z_q) of its rejected position
    int32_t *exh_meta;     // [2B] (n, flags) of the sequence
    float *exh_psum;       // [B, nparts] part sums written by that kernel (group sums go to fallback_rows[j, M])
    int coop;              // 1: thinning_enumerate_kernel runs behind this kernel
};

constexpr int kThinSlots = 128;  // slots of the candidate order (the interface's rule: slot of token t = (t div W) mod 128)
static_assert(kPosThreads == 2 * kThinSlots && kPosThreadsSmall == kThinSlots,
              "a slot is the words of one thread of the position kernel (short rows) or of two (long rows)");
static_assert(kThinThreads % kThinSlots == 0, "the block sums the slots with a whole number of threads per slot");

static size_t thin_smem_bytes() {
    return kThinSlots * 8 + 32 * 8 + 64 * 4 + 8 * 4 + 2 * (kThinThreads / 32) * 4 + (kThinThreads / kThinSlots) * kThinSlots * 4;
}

// 2^(l s - rs) of the 16-byte word `word` of `row` (NV logits); zero past the end of the row.
template <typename T>
__device__ __forceinline__ void thin_word_terms(const T *row, int V, int word, bool vec_ok, float s, float rs,
                                                float (&e)[Elem<T>::kPerVec]) {
    constexpr int NV = Elem<T>::kPerVec;
    const int t0 = word * NV;
    if (vec_ok && t0 + NV <= V) {
        float v[NV];
        Elem<T>::unpack(ld_stream(reinterpret_cast<const uint4 *>(row + t0)), v);
#pragma unroll
        for (int i = 0; i < NV; ++i) e[i] = ex2(__fmaf_rn(v[i], s, -rs));
    } else {
#pragma unroll
        for (int i = 0; i < NV; ++i) e[i] = t0 + i < V ? ex2(__fmaf_rn(Elem<T>::widen(row[t0 + i]), s, -rs)) : 0.f;
    }
}

template <int NV>
__device__ __forceinline__ float thin_lane_sum(const float (&e)[NV]) {
    float v = e[0];
#pragma unroll
    for (int i = 1; i < NV; ++i) v += e[i];
    return v;
}

template <typename T>
__global__ void __launch_bounds__(kThinThreads, 2) thinning_kernel(ThinArgs a, GroupsDev G) {
    constexpr int NT = kThinThreads, NW = NT / 32, NV = Elem<T>::kPerVec, S = kThinSlots, SUB = NT / S;
    extern __shared__ __align__(16) unsigned char raw[];
    __shared__ int s_n, s_flags;
    __shared__ float4 s_stats;
    const int V = G.V, M = G.M, K = a.K;
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nwords = (V + NV - 1) / NV;                       // 16-byte words of a row (the last may be partial)
    double *slot_incl = reinterpret_cast<double *>(raw);        // [S] inclusive prefix of the slot masses
    double *dscratch = slot_incl + S;                           // 32 doubles
    float *scratch = reinterpret_cast<float *>(dscratch + 32);  // 64 floats
    int *ibox = reinterpret_cast<int *>(scratch + 64);          // 8 ints
    int *cand = ibox + 8;                                       // NW ints: group kept by each warp's trial, or -1
    int *cand_tok = cand + NW;                                  // NW ints: the token drawn inside that group
    float *part = reinterpret_cast<float *>(cand_tok + NW);     // [SUB][S] partial slot sums of the pass below

    // the first trial of this warp: its uniforms are inputs of the call, so they can be fetched before the
    // position kernel's results are waited for
    const float *tu = a.thin + (size_t)b * a.n_trials * 3;
    float u_first[3] = {0.f, 0.f, 0.f};
    if (warp < a.n_trials) {
#pragma unroll
        for (int j = 0; j < 3; ++j) u_first[j] = __ldcg(tu + 3 * warp + j);  // (from L2: ahead of the wait nothing vouches for this SM's L1)
    }
    const float u_token = __ldcg(a.uniforms + ((int64_t)b * (K + 1) + K) * 2 + 1);
    const int pre_tok = tid < K ? __ldcg(a.draft_tokens + b * K + tid) : -1;  // for the emission at the end
    pdl_enter();  // everything above may overlap the tail of the position kernel; none of its results is read before here

    // ---- 1. first rejected position and the flags of the positions up to it ----
    if (tid < 32) {
        int n = K, flags = 0;
        // the statistics of the first 32 positions travel with their accept bits (one hop fewer for most sequences)
        const float4 early = tid < K ? a.stats[b * K + tid] : make_float4(0.f, 0.f, 0.f, 0.f);
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
        const int src = n < 32 ? n : 0;
        float4 st;
        st.x = __shfl_sync(0xffffffffu, early.x, src);
        st.y = __shfl_sync(0xffffffffu, early.y, src);
        st.z = __shfl_sync(0xffffffffu, early.z, src);
        st.w = __shfl_sync(0xffffffffu, early.w, src);
        if (tid == 0) {
            s_n = n;
            s_flags = flags;
            s_stats = (n < K && n >= 32) ? a.stats[b * K + n] : st;
        }
    }
    __syncthreads();
    const int n = s_n;
    int flags = s_flags;
    const bool residual = n < K;  // false: every position accepted, the terminal draw is the bonus token
    const T *trow = reinterpret_cast<const T *>(a.target) + ((int64_t)b * (K + 1) + n) * V;
    const T *qrow = reinterpret_cast<const T *>(a.draft) + ((int64_t)b * K + min(n, K - 1)) * V;
    const bool vec_ok = ((uintptr_t)trow & 15u) == 0;
    float rs_p, iz_p, rs_q = 0.f, iz_q = 0.f;
    if (residual) {
        const float4 st = s_stats;
        rs_p = st.x, iz_p = st.y, rs_q = st.z, iz_q = st.w;
    } else {
        // statistics of the bonus row: one pass with a per-thread reference, merged over the block
        RefSum st{kRefInit * a.s, 0.f};
        for (int word = tid; word < nwords; word += NT) {
            const int t0 = word * NV;
            if (vec_ok && t0 + NV <= V) {
                float v[NV];
                Elem<T>::unpack(ld_stream(reinterpret_cast<const uint4 *>(trow + t0)), v);
                absorb<NV>(st, v, a.s);
            } else {
                for (int i = 0; i < NV && t0 + i < V; ++i) absorb1(st, Elem<T>::widen(trow[t0 + i]), a.s);
            }
        }
        float rs = st.rs, Z = st.acc;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) merge(rs, Z, __shfl_xor_sync(0xffffffffu, rs, o), __shfl_xor_sync(0xffffffffu, Z, o));
        if (lane == 0) {
            scratch[2 * warp] = rs;
            scratch[2 * warp + 1] = Z;
        }
        __syncthreads();
        rs = scratch[0];
        Z = scratch[1];
        for (int w = 1; w < NW; ++w) merge(rs, Z, scratch[2 * w], scratch[2 * w + 1]);
        __syncthreads();
        if (!(Z > 0.f) || isinf(Z) || isinf(rs)) flags |= PCG_FLAG_NONFINITE;
        rs_p = rs;
        iz_p = 1.0f / Z;
    }

    // ---- 2. the slot masses of the target row (slot of token t = (t div NV) mod S), then their prefix ----
    float mass = 0.f;  // of slot tid, in threads tid < S
    if (a.strata && residual) {
        // the position kernel's thread h (short rows: S threads per block) or its threads h and h + S between them
        // (long rows: words h, h + 2S, ... and h + S, h + 3S, ...) summed exactly slot h, each relative to a reference
        // of its own that is at most the row's final one
        if (tid < S) {
            const float2 *pairs = a.strata + (size_t)(b * K + n) * a.strata_threads;
            const float2 v0 = pairs[tid];
            mass = __fmul_rn(v0.y, ex2(v0.x - rs_p));
            if (a.strata_threads == 2 * S) {
                const float2 v1 = pairs[S + tid];
                mass += __fmul_rn(v1.y, ex2(v1.x - rs_p));
            }
        }
    } else {
        // SUB threads per slot walk the slot's words, four loads in flight each; partial sums added in fixed order
        const int h = tid % S, sub = tid / S;
        float acc = 0.f;
        for (int w0 = h + S * sub; w0 < nwords; w0 += 4 * S * SUB) {
            float e[4][NV];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int word = w0 + j * S * SUB;
                if (word < nwords) {
                    thin_word_terms<T>(trow, V, word, vec_ok, a.s, rs_p, e[j]);
                } else {
#pragma unroll
                    for (int i = 0; i < NV; ++i) e[j][i] = 0.f;
                }
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) acc += thin_lane_sum<NV>(e[j]);
        }
        part[sub * S + h] = acc;
        __syncthreads();
        if (tid < S)
            for (int j = 0; j < SUB; ++j) mass += part[j * S + tid];
    }
    double Ztot;
    {
        double excl, incl;
        block_scan<NT>(tid < S ? (double)mass : 0.0, dscratch, &excl, &incl, &Ztot);
        if (tid < S) slot_incl[tid] = incl;
    }
    __syncthreads();

    // ---- 3. trials: warp w of round r0 runs trial r0 + w; the first kept candidate in trial order wins ----
    int gsel = -1, used = 0, z = -1;
    const bool usable = Ztot > 0.0 && Ztot < (double)__builtin_huge_valf();
    if (!usable) flags |= PCG_FLAG_NONFINITE;
    const int max_trials = usable ? (residual ? a.n_trials : 1) : 0;
    // trials of the first round (every trial reads its slot's words, scattered over the whole row: fewer side by
    // side means less traffic, more means fewer sequences need a second round)
    constexpr int kFirstRound = 8;
    for (int r0 = 0, width = kFirstRound; r0 < max_trials && gsel < 0; r0 += width, width = NW) {
        const int r = r0 + warp;
        int kept = -1;
        if (warp < width && r < max_trials) {
            const float u_tok = r0 ? tu[3 * r] : u_first[0], u_lab = r0 ? tu[3 * r + 1] : u_first[1];
            const float u_keep = r0 ? tu[3 * r + 2] : u_first[2];
            // token y ~ target: slot by binary search over the prefix, then a scan over the slot's words in token
            // order, 32 words (each S words apart) at a time with the next 32 already loading
            const double target = (double)u_tok * Ztot;
            int lo = 0, hi = S - 1;  // the last slot's prefix is the total, which exceeds u * total for u < 1
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (slot_incl[mid] > target)
                    hi = mid;
                else
                    lo = mid + 1;
            }
            const int h = lo;
            const double tl = target - (h > 0 ? slot_incl[h - 1] : 0.0);
            const int cnt = h < nwords ? (nwords - h + S - 1) / S : 0;  // words of slot h
            double carry = 0.0;
            int y = -1, y_last = -1;
            float e[NV], e_next[NV];
            if (lane < cnt) thin_word_terms<T>(trow, V, h + S * lane, vec_ok, a.s, rs_p, e);
            for (int base = 0; base < cnt && y < 0; base += 32) {
                const int m = base + lane;
                if (m >= cnt) {
#pragma unroll
                    for (int i = 0; i < NV; ++i) e[i] = 0.f;
                }
                if (m + 32 < cnt) thin_word_terms<T>(trow, V, h + S * (m + 32), vec_ok, a.s, rs_p, e_next);
                const float lsum = thin_lane_sum<NV>(e);
                double inc = (double)lsum;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const double up = __shfl_up_sync(0xffffffffu, inc, o);
                    if (lane >= o) inc += up;
                }
                const unsigned above = __ballot_sync(0xffffffffu, lsum > 0.f && carry + inc > tl);
                const unsigned massy = __ballot_sync(0xffffffffu, lsum > 0.f);
                // the lane that holds the answer of this chunk (if any), and the last lane with mass for the case
                // that rounding leaves no prefix above the target
                const int L = above ? __ffs(above) - 1 : (massy ? 31 - __clz(massy) : -1);
                if (L >= 0) {
                    int pick = 0;
                    if (lane == L) {
                        double loc = carry + inc - (double)lsum;
                        int first_above = -1, last = 0;
#pragma unroll
                        for (int i = 0; i < NV; ++i) {
                            loc += (double)e[i];
                            if (e[i] > 0.f) {
                                last = i;
                                if (first_above < 0 && loc > tl) first_above = i;
                            }
                        }
                        pick = first_above >= 0 ? first_above : last;
                    }
                    pick = __shfl_sync(0xffffffffu, pick, L);
                    const int tok = (h + S * (base + L)) * NV + pick;
                    if (above)
                        y = tok;
                    else
                        y_last = tok;
                }
                carry += __shfl_sync(0xffffffffu, inc, 31);
#pragma unroll
                for (int i = 0; i < NV; ++i) e[i] = e_next[i];
            }
            if (y < 0) y = y_last >= 0 ? y_last : min(h * NV, V - 1);
            if (y >= V) y = V - 1;
            // label k ~ w_{.,y}
            const int rv0 = G.rev_ptr[y];
            const int g = draw_label(G, rv0, G.rev_ptr[y + 1] - rv0, u_lab);
            bool keep = true;
            if (residual) {
                // the two masses of group g (a warp gather over its tokens), then u < [1 - Q/P]_+ without a division
                const int k_lo = G.group_ptr[g], k_hi = G.group_ptr[g + 1];
                float Sp = 0.f, Sq = 0.f;
                for (int k = k_lo + lane; k < k_hi; k += 32) {
                    const int t = G.group_tok[k];
                    const float w = G.pair_w ? G.pair_w[k] : G.inv_deg[t];
                    Sp += __fmul_rn(ex2(__fmaf_rn(Elem<T>::widen(trow[t]), a.s, -rs_p)), w);
                    Sq += __fmul_rn(ex2(__fmaf_rn(Elem<T>::widen(qrow[t]), a.s, -rs_q)), w);
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    Sp += __shfl_xor_sync(0xffffffffu, Sp, o);
                    Sq += __shfl_xor_sync(0xffffffffu, Sq, o);
                }
                const float P = __fmul_rn(Sp, iz_p), Q = __fmul_rn(Sq, iz_q);
                keep = __fmul_rn(u_keep, P) < P - Q;
            }
            kept = keep ? g : -1;
            if (keep) {  // the token inside the kept group, by this warp (used only if this trial wins)
                const int zt = warp_token_in_group<T>(G, trow, g, a.s, u_token, lane);
                if (lane == 0) cand_tok[warp] = zt;
            }
        }
        if (lane == 0) cand[warp] = kept;
        __syncthreads();
        used = min(r0 + width, max_trials);
        for (int w = 0; w < NW; ++w)
            if (cand[w] >= 0) {
                gsel = cand[w];
                z = cand_tok[w];
                used = r0 + w + 1;
                break;
            }
        __syncthreads();
    }

    // ---- every supplied trial was turned down ----
    // With the enumeration kernel behind this one (a.coop) the sequence is handed to it: all blocks of the GPU then
    // share its enumeration.  Without, it is enumerated right here by its own block.  (One route per call, so that
    // a sequence's result never depends on which other sequences ran out.)
    if (usable && gsel < 0 && a.coop) {
        if (tid == 0) {
            const int slot = atomicAdd(&a.exh[0], 1);
            a.exh[2 + slot] = b;
            a.exh_stats[b] = make_float4(rs_p, iz_p, rs_q, iz_q);
            a.exh_meta[2 * b] = n;
            a.exh_meta[2 * b + 1] = flags | PCG_FLAG_THINNING_EXHAUSTED;
            if (a.out_trials) a.out_trials[b] = used;
        }
        return;  // (block-uniform) that kernel draws group and token and writes the sequence's outputs
    }
    // ---- enumerate the residual in this block and invert its CDF (same law) ----
    if (usable && gsel < 0) {
        flags |= PCG_FLAG_THINNING_EXHAUSTED;
        float *own = a.fallback_rows + (size_t)b * M;
        const float u_group = a.uniforms[((int64_t)b * (K + 1) + K) * 2];
        const int per = (M + NT - 1) / NT;
        const int i0 = min(M, tid * per), i1 = min(M, i0 + per);
        double Zr = 0.0, excl = 0.0, incl = 0.0, my = 0.0;
        bool minus_q = true;
        for (int attempt = 0; attempt < 2; ++attempt) {
            // one thread per group, its tokens eight at a time: ids first, then the gathers they address, then the
            // sum in CSR order (the dependent loads of a batch are in flight together)
            constexpr int FB = 8;
            for (int g = tid; g < M; g += NT) {
                float acc = 0.f;
                const int k_end = G.group_ptr[g + 1];
                for (int k = G.group_ptr[g]; k < k_end; k += FB) {
                    int t[FB];
                    float lp[FB], lq[FB], w[FB];
#pragma unroll
                    for (int j = 0; j < FB; ++j) t[j] = k + j < k_end ? G.group_tok[k + j] : -1;
#pragma unroll
                    for (int j = 0; j < FB; ++j) {
                        lp[j] = lq[j] = kNegInf;
                        w[j] = 0.f;
                        if (t[j] >= 0) {
                            lp[j] = Elem<T>::widen(trow[t[j]]);
                            if (minus_q) lq[j] = Elem<T>::widen(qrow[t[j]]);
                            w[j] = G.pair_w ? G.pair_w[k + j] : G.inv_deg[t[j]];
                        }
                    }
#pragma unroll
                    for (int j = 0; j < FB; ++j) {
                        if (t[j] < 0) continue;
                        float d = __fmul_rn(ex2(__fmaf_rn(lp[j], a.s, -rs_p)), iz_p);
                        if (minus_q) d -= __fmul_rn(ex2(__fmaf_rn(lq[j], a.s, -rs_q)), iz_q);
                        acc += __fmul_rn(d, w[j]);
                    }
                }
                own[g] = fmaxf(acc, 0.f);
            }
            __syncthreads();
            my = 0.0;
            for (int j = i0; j < i1; ++j) my += (double)own[j];
            block_scan<NT>(my, dscratch, &excl, &incl, &Zr);
            if (Zr > 0.0 || !minus_q) break;
            flags |= PCG_FLAG_ZERO_RESIDUAL;  // the residual vanished (P == Q to rounding): draw from P instead
            minus_q = false;
            __syncthreads();
        }
        const double target = (double)u_group * Zr;
        if (tid == 0) {
            ibox[2] = NT;
            ibox[3] = -1;
            ibox[4] = -1;
        }
        __syncthreads();
        int my_last = -1;
        for (int j = i0; j < i1; ++j)
            if (own[j] > 0.f) my_last = j;
        if (my_last >= 0) atomicMax(&ibox[3], my_last);
        if (my > 0.0 && incl > target) atomicMin(&ibox[2], tid);
        __syncthreads();
        if (ibox[2] == tid) {
            double loc = 0.0;
            int pick = my_last;
            for (int j = i0; j < i1; ++j) {
                loc += (double)own[j];
                if (excl + loc > target) {
                    pick = j;
                    break;
                }
            }
            ibox[4] = pick;
        }
        __syncthreads();
        gsel = ibox[4] >= 0 ? ibox[4] : ibox[3];
        __syncthreads();
    }

    // ---- 4. outputs (the token was drawn by the winning warp; block-wide after the enumerated fallback) ----
    if (gsel < 0) {  // no mass anywhere (non-finite inputs): emit group 0 / token 0 and flag it
        gsel = 0;
        z = 0;
        flags |= PCG_FLAG_NONFINITE;
    } else if (z < 0) {
        z = block_token_in_group<T>(G, trow, gsel, a.s, u_token, ibox, flags);
    }
    for (int i = tid; i <= K; i += NT) {
        int tok = -1, grp = -1;
        if (i < n) {
            tok = i == tid ? pre_tok : a.draft_tokens[b * K + i];
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
        if (a.out_trials) a.out_trials[b] = used;
    }
}

// Enumerated residual for the sequences whose thinning trials ran out (a.exh), by the whole grid.
// Grid: ceil(nparts / 4) blocks of 4 warps, as the sparse product.  Nothing to do (the usual case): every block
// returns right after the wait.  Otherwise warp = one part of the groups: for every listed sequence it gathers the
// two logits of each of its stored pairs straight from the rows (lane = pair, 32 at a time), forms
// (p - q) w, adds the terms group by group (per-lane partial sums, then a butterfly: a fixed order), writes the
// group sums to fallback_rows[j, g] and the sum of their positive parts to exh_psum[j, part].  The block that
// finishes last (a counter; nobody waits for anybody) then draws group and token of every listed sequence with
// pick_group_and_token and writes its outputs.  (A counter per sequence, so that the draws spread over the blocks,
// was slower: 740 additions to one word per sequence.)
constexpr int kEnumThreads = 128;

template <typename T>
__global__ void __launch_bounds__(kEnumThreads) thinning_enumerate_kernel(ThinArgs a, GroupsDev G) {
    constexpr int NT = kEnumThreads;
    __shared__ double dscratch[32];
    __shared__ int ibox[8];
    pdl_enter();
    const int ne = a.exh[0];
    if (ne == 0) return;
    const int V = G.V, M = G.M, K = a.K, NP = G.nparts;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int part = blockIdx.x * (NT / 32) + warp;
    const bool working = part < NP;  // (warp-uniform; the last block may have warps without a part)
    const int g0 = working ? G.part_ptr[part] : 0, ng = working ? G.part_ptr[part + 1] - g0 : 0;  // at most kPartMaxGroups
    const int ptr_l = (working && lane <= ng) ? G.group_ptr[g0 + lane] : 0;                          // lane i: group_ptr[g0 + i]
    const int e0 = __shfl_sync(0xffffffffu, ptr_l, 0), e1 = __shfl_sync(0xffffffffu, ptr_l, ng);
    for (int j = 0; j < ne; ++j) {
        if (working) {
            const int b = a.exh[2 + j];
            const float4 st = a.exh_stats[b];
            const int n = a.exh_meta[2 * b];
            const T *trow = reinterpret_cast<const T *>(a.target) + ((int64_t)b * (K + 1) + n) * V;
            const T *qrow = reinterpret_cast<const T *>(a.draft) + ((int64_t)b * K + min(n, K - 1)) * V;
            float gsum[kPartMaxGroups];
#pragma unroll
            for (int gi = 0; gi < kPartMaxGroups; ++gi) gsum[gi] = 0.f;
            for (int k0 = e0; k0 < e1; k0 += 32) {
                const int k = k0 + lane;
                float d = 0.f;
                if (k < e1) {
                    const int t = G.group_tok[k];
                    const float w = G.pair_w ? G.pair_w[k] : G.inv_deg[t];
                    float v = __fmul_rn(ex2(__fmaf_rn(Elem<T>::widen(trow[t]), a.s, -st.x)), st.y);
                    v -= __fmul_rn(ex2(__fmaf_rn(Elem<T>::widen(qrow[t]), a.s, -st.z)), st.w);
                    d = __fmul_rn(v, w);
                }
#pragma unroll
                for (int gi = 0; gi < kPartMaxGroups; ++gi) {
                    const int lo = __shfl_sync(0xffffffffu, ptr_l, gi), hi = __shfl_sync(0xffffffffu, ptr_l, gi + 1);
                    if (gi < ng && k >= lo && k < hi) gsum[gi] += d;
                }
            }
            float pos = 0.f;
#pragma unroll
            for (int gi = 0; gi < kPartMaxGroups; ++gi) {
                float r = gsum[gi];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) r += __shfl_xor_sync(0xffffffffu, r, o);
                if (gi < ng) {
                    if (lane == 0) a.fallback_rows[(size_t)j * M + g0 + gi] = r;
                    pos += fmaxf(r, 0.f);  // (P - Q)_+ ; NaN counts as 0
                }
            }
            if (lane == 0) a.exh_psum[(size_t)j * NP + part] = pos;
        }
    }
    // ---- the block that finishes last draws for the listed sequences (a counter; nobody waits for anybody) ----
    __threadfence();
    __syncthreads();
    if (tid == 0) ibox[7] = atomicAdd(&a.exh[1], 1);
    __syncthreads();
    if (ibox[7] != (int)gridDim.x - 1) return;
    __threadfence();
    for (int j = 0; j < ne; ++j) {
        const int b = a.exh[2 + j];
        const int n = a.exh_meta[2 * b];
        int flags = a.exh_meta[2 * b + 1];
        const float rs_p = a.exh_stats[b].x;
        const T *trow = reinterpret_cast<const T *>(a.target) + ((int64_t)b * (K + 1) + n) * V;
        const float u_group = a.uniforms[((int64_t)b * (K + 1) + K) * 2];
        const float u_token = a.uniforms[((int64_t)b * (K + 1) + K) * 2 + 1];
        int gsel, z;
        pick_group_and_token<T, NT>(G, trow, a.s, rs_p, true, u_group, u_token, a.fallback_rows + (size_t)j * M, 1,
                                    a.exh_psum + (size_t)j * NP, 1, dscratch, ibox, flags, gsel, z);
        emit_sequence<NT>(G, b, K, n, z, gsel, flags, a.draft_tokens, a.labels, a.out_accept_len, a.out_tokens, a.out_groups,
                          a.out_flags);
        __syncthreads();
    }
}
