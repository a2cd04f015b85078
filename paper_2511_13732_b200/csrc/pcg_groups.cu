// Group handle: host-side validation of the membership CSR and construction of the device layouts.
// One-time set-up (the groups are precomputed once and cached); not part of the verification hot path.
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <algorithm>
#include <new>
#include <queue>
#include <vector>

#include "pcg_common.cuh"

namespace pcg {

static thread_local char g_error[512] = "";

void set_error(const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_error, sizeof g_error, fmt, ap);
    va_end(ap);
}

pcg_status cuda_fail(cudaError_t e, const char *what) {
    set_error("%s: %s", what, cudaGetErrorString(e));
    return PCG_ERR_CUDA;
}

constexpr size_t kMaxSmem = 227 * 1024;
constexpr size_t kAggScratch = 2048;

size_t agg_smem_bytes(int slice_len, int M, int slices) {
    size_t mc = (size_t)(M + slices - 1) / slices;
    return ((size_t)slice_len + 32) * 4 + (size_t)M * 4 + mc * 4 + kAggScratch;
}

}  // namespace pcg

extern "C" const char *pcg_status_string(pcg_status s) {
    switch (s) {
        case PCG_OK: return "ok";
        case PCG_ERR_INVALID_ARG: return "invalid argument";
        case PCG_ERR_INVALID_GROUPS: return "invalid group membership";
        case PCG_ERR_UNSUPPORTED: return "unsupported size";
        case PCG_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case PCG_ERR_CUDA: return "CUDA error";
    }
    return "unknown status";
}

extern "C" const char *pcg_last_error(void) { return pcg::g_error; }

namespace {

struct Carver {  // lays arrays out in one allocation, 256-byte aligned
    size_t off = 0;
    size_t take(size_t bytes) {
        size_t at = off;
        off = (off + bytes + 255) & ~(size_t)255;
        return at;
    }
};

template <typename T>
cudaError_t upload(char *base, size_t at, const std::vector<T> &v) {
    if (v.empty()) return cudaSuccess;
    return cudaMemcpy(base + at, v.data(), v.size() * sizeof(T), cudaMemcpyHostToDevice);
}

}  // namespace

extern "C" pcg_status pcg_groups_create(const pcg_csr *csr, int slices_hint, pcg_groups **out) {
    using namespace pcg;
    if (out) *out = nullptr;
    if (!csr || !out || !csr->group_ptr || !csr->tok_degree || (csr->nnz > 0 && !csr->group_tok)) {
        set_error("pcg_groups_create: null argument");
        return PCG_ERR_INVALID_ARG;
    }
    const int V = csr->V, M = csr->M;
    const int64_t nnz = csr->nnz;
    if (V < 1 || M < 1 || nnz < 0 || nnz > INT32_MAX) {
        set_error("pcg_groups_create: need V >= 1, M >= 1, 0 <= nnz < 2^31 (V=%d M=%d nnz=%lld)", V, M, (long long)nnz);
        return PCG_ERR_INVALID_ARG;
    }
    if (slices_hint != 0 && slices_hint != 1 && slices_hint != 2 && slices_hint != 4 && slices_hint != 8) {
        set_error("pcg_groups_create: slices_hint must be 0, 1, 2, 4 or 8");
        return PCG_ERR_INVALID_ARG;
    }
    // Without a usable CUDA device the arrays are taken to be host memory, so that the validation below
    // still reports what is wrong with them; the call then fails with PCG_ERR_CUDA at the allocation.
    int device = 0;
    cudaError_t e = cudaGetDevice(&device);
    const bool have_device = (e == cudaSuccess);
    if (!have_device) (void)cudaGetLastError();

    // ---- bring the CSR to the host (with a device present the arrays may be host or device memory) ----
    std::vector<int32_t> gptr((size_t)M + 1), gtok((size_t)nnz), deg((size_t)V);
    std::vector<float> w;
    if (csr->weights && nnz) w.resize((size_t)nnz);
    if (have_device) {
        e = cudaMemcpy(gptr.data(), csr->group_ptr, gptr.size() * 4, cudaMemcpyDefault);
        if (e == cudaSuccess && nnz) e = cudaMemcpy(gtok.data(), csr->group_tok, gtok.size() * 4, cudaMemcpyDefault);
        if (e == cudaSuccess) e = cudaMemcpy(deg.data(), csr->tok_degree, deg.size() * 4, cudaMemcpyDefault);
        if (e == cudaSuccess && !w.empty()) e = cudaMemcpy(w.data(), csr->weights, w.size() * 4, cudaMemcpyDefault);
        if (e != cudaSuccess) return cuda_fail(e, "copying the membership CSR");
    } else {
        memcpy(gptr.data(), csr->group_ptr, gptr.size() * 4);
        if (nnz) memcpy(gtok.data(), csr->group_tok, gtok.size() * 4);
        memcpy(deg.data(), csr->tok_degree, deg.size() * 4);
        if (!w.empty()) memcpy(w.data(), csr->weights, w.size() * 4);
    }

    // ---- validate ----
    if (gptr[0] != 0 || gptr[M] != nnz) {
        set_error("group_ptr[0] must be 0 and group_ptr[M] must equal nnz");
        return PCG_ERR_INVALID_GROUPS;
    }
    // the whole pointer array first: 0 <= group_ptr[g] <= group_ptr[g+1] <= nnz, so that no token list read below
    // can leave the copy of group_tok
    for (int g = 0; g < M; ++g) {
        if (gptr[g] < 0 || gptr[g + 1] < gptr[g] || (int64_t)gptr[g + 1] > nnz) {
            set_error("group_ptr decreases or leaves [0, nnz] at group %d", g);
            return PCG_ERR_INVALID_GROUPS;
        }
    }
    std::vector<int32_t> count((size_t)V, 0);
    int max_group = 0;
    for (int g = 0; g < M; ++g) {
        for (int32_t k = gptr[g]; k < gptr[g + 1]; ++k) {
            int32_t t = gtok[k];
            if (t < 0 || t >= V) {
                set_error("token id %d of group %d is outside [0,%d)", t, g, V);
                return PCG_ERR_INVALID_GROUPS;
            }
            if (k > gptr[g] && gtok[k - 1] >= t) {
                set_error("tokens of group %d are not strictly ascending", g);
                return PCG_ERR_INVALID_GROUPS;
            }
            count[t]++;
        }
        max_group = std::max(max_group, gptr[g + 1] - gptr[g]);
    }
    int max_deg = 0;
    for (int t = 0; t < V; ++t) {
        if (deg[t] != count[t] || deg[t] < 1) {
            set_error("tok_degree[%d] = %d but the token is listed by %d groups (every token needs >= 1)", t, deg[t],
                      count[t]);
            return PCG_ERR_INVALID_GROUPS;
        }
        max_deg = std::max(max_deg, deg[t]);
    }

    // ---- reverse membership S(t), ascending group id (counting sort over the CSR) ----
    std::vector<int32_t> rptr((size_t)V + 1, 0), rgrp((size_t)nnz);
    std::vector<float> rw;
    for (int t = 0; t < V; ++t) rptr[t + 1] = rptr[t] + deg[t];
    {
        std::vector<int32_t> fill(rptr.begin(), rptr.end() - 1);
        if (!w.empty()) rw.resize((size_t)nnz);
        for (int g = 0; g < M; ++g)
            for (int32_t k = gptr[g]; k < gptr[g + 1]; ++k) {
                int32_t at = fill[gtok[k]]++;
                rgrp[at] = g;
                if (!w.empty()) rw[at] = w[k];
            }
    }
    if (!w.empty()) {
        for (int64_t k = 0; k < nnz; ++k)
            if (!(w[k] >= 0.f) || !std::isfinite(w[k])) {
                set_error("weights[%lld] is negative or not finite", (long long)k);
                return PCG_ERR_INVALID_GROUPS;
            }
        for (int t = 0; t < V; ++t) {
            double s = 0;
            for (int32_t k = rptr[t]; k < rptr[t + 1]; ++k) s += rw[k];
            if (std::fabs(s - 1.0) > 1e-4) {
                set_error("weights of token %d sum to %.6f over its groups, not 1", t, s);
                return PCG_ERR_INVALID_GROUPS;
            }
        }
    }

    // ---- choose the token slicing ----
    int C = slices_hint ? slices_hint : 1;
    if (!slices_hint)
        while (C < 8 && (V + C - 1) / C > 8192) C *= 2;
    // Beyond 65534 groups (the sweep entries hold group ids in 16 bits) or when a token slice plus the per-group
    // partial sums cannot fit in shared memory, the handle carries no sweep layout: the kernels that need it (the
    // per-row cluster kernel of pcg_group_probs, PCG_VERIFY_CLUSTER_TERMINAL) are then unavailable and the batched
    // kernels are used throughout.
    bool has_sweep = M < (int)kNoGroup;
    int SL = 0;
    for (; has_sweep; C *= 2) {
        SL = (((V + C - 1) / C) + 63) / 64 * 64;
        if (SL <= 65472 && agg_smem_bytes(SL, M, C) <= kMaxSmem) break;
        if (C >= 8) has_sweep = false;
    }
    if (!has_sweep) {
        if (slices_hint) {
            set_error("V=%d, M=%d: no sweep layout is possible, so slices_hint must be 0", V, M);
            return PCG_ERR_UNSUPPORTED;
        }
        C = 1;
        SL = ((V + 63) / 64) * 64;
    }

    // ---- token-sliced sweep layout (see GroupsDev::ent) ----
    // Per slice, the groups' sub-lists are dealt to the kAggThreads threads longest first, each to the thread
    // with the least work so far (ties: lowest thread id), so that the columns are balanced.
    std::vector<int32_t> eoff((size_t)C + 1, 0);
    std::vector<uint32_t> ent;
    std::vector<float> entw;
    {
        constexpr int NT = kAggThreads;
        std::vector<int32_t> cursor(gptr.begin(), gptr.end() - 1);  // tokens ascend, so each slice is a sub-range
        std::vector<int32_t> sub_lo((size_t)M), sub_hi((size_t)M), order((size_t)M);
        std::vector<std::vector<int32_t>> owned(NT);
        for (int c = 0; c < C && has_sweep; ++c) {
            const int32_t t_end = (int32_t)std::min<int64_t>((int64_t)(c + 1) * SL, V);
            for (int g = 0; g < M; ++g) {
                int32_t k = cursor[g];
                sub_lo[g] = k;
                while (k < gptr[g + 1] && gtok[k] < t_end) ++k;
                sub_hi[g] = cursor[g] = k;
                order[g] = g;
            }
            std::stable_sort(order.begin(), order.end(), [&](int32_t x, int32_t y) {
                return sub_hi[x] - sub_lo[x] > sub_hi[y] - sub_lo[y];
            });
            std::priority_queue<std::pair<int64_t, int>, std::vector<std::pair<int64_t, int>>,
                                std::greater<std::pair<int64_t, int>>> load;
            for (int t = 0; t < NT; ++t) {
                owned[t].clear();
                load.push({0, t});
            }
            for (int32_t g : order) {
                const int32_t len = sub_hi[g] - sub_lo[g];
                if (len == 0) break;  // the rest is empty in this slice (partial[] is zero-filled by the kernel)
                auto top = load.top();
                load.pop();
                owned[top.second].push_back(g);
                load.push({top.first + len, top.second});
            }
            int64_t rows = 0;
            for (int t = 0; t < NT; ++t) {
                int64_t n = 0;
                for (int32_t g : owned[t]) n += sub_hi[g] - sub_lo[g];
                rows = std::max(rows, n);
            }
            const size_t base = ent.size();
            if ((int64_t)base + rows * NT > INT32_MAX) {
                set_error("membership too large for the sweep layout");
                return PCG_ERR_UNSUPPORTED;
            }
            ent.resize(base + (size_t)rows * NT);
            if (!w.empty()) entw.resize(ent.size(), 0.f);
            for (int t = 0; t < NT; ++t) {
                int64_t j = 0;
                uint32_t last_group = kNoGroup;
                for (int32_t g : owned[t]) {
                    last_group = (uint32_t)g;
                    for (int32_t k = sub_lo[g]; k < sub_hi[g]; ++k, ++j) {
                        ent[base + (size_t)j * NT + t] = ((uint32_t)g << 16) | (uint32_t)(gtok[k] - c * SL);
                        if (!w.empty()) entw[base + (size_t)j * NT + t] = w[k];
                    }
                }
                for (; j < rows; ++j) ent[base + (size_t)j * NT + t] = (last_group << 16) | (uint32_t)SL;
            }
            eoff[c + 1] = (int32_t)ent.size();
        }
    }
    std::vector<float> inv((size_t)V);
    for (int t = 0; t < V; ++t) inv[t] = 1.0f / (float)deg[t];

    // ---- partition of the groups for the sparse product (see GroupsDev::part_ptr) ----
    // Cut points are the group boundaries nearest to the quantiles k * nnz / parts of the pair index, so that parts
    // differ by at most about one group's size; runs of more than kPartMaxGroups (small) groups are cut further.
    int sm_count = 148;
    if (have_device) cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, device);
    std::vector<int32_t> part_ptr;
    {
        const int64_t want = std::max<int64_t>(1, std::min<int64_t>((int64_t)sm_count * kPartWarpsPerSM, nnz / 32));
        part_ptr.push_back(0);
        int g = 0;
        for (int64_t k = 1; k <= want && g < M; ++k) {
            int gend = M;
            if (k < want) {
                const int64_t target = k * nnz / want;
                int hi = (int)(std::lower_bound(gptr.begin() + g, gptr.end(), (int32_t)target) - gptr.begin());
                hi = std::min(hi, M);
                const int lo = std::max(hi - 1, g);
                gend = (target - gptr[lo] <= (int64_t)gptr[hi] - target) ? lo : hi;
                if (gend <= g) continue;  // the quantile falls inside a group larger than a part
            }
            while (gend - g > kPartMaxGroups) {
                g += kPartMaxGroups;
                part_ptr.push_back(g);
            }
            g = gend;
            part_ptr.push_back(g);
        }
    }

    // ---- one device allocation for everything ----
    Carver cv;
    const size_t o_gptr = cv.take(gptr.size() * 4), o_gtok = cv.take(gtok.size() * 4), o_inv = cv.take(inv.size() * 4);
    const size_t o_rptr = cv.take(rptr.size() * 4), o_rgrp = cv.take(rgrp.size() * 4);
    const size_t o_eoff = cv.take(eoff.size() * 4), o_ent = cv.take(ent.size() * 4);
    const size_t o_w = cv.take(w.size() * 4), o_entw = cv.take(entw.size() * 4), o_rw = cv.take(rw.size() * 4);
    std::vector<int32_t> part_ent(part_ptr.size());
    for (size_t k = 0; k < part_ptr.size(); ++k) part_ent[k] = gptr[part_ptr[k]];
    const size_t o_part = cv.take(part_ptr.size() * 4), o_pent = cv.take(part_ent.size() * 4);
    // scratch of the batched route of pcg_group_probs: 128 rows per chunk, more while Dt stays within 64 MB
    const int probs_chunk = probs_chunk_rows(V);
    const size_t o_pdt = cv.take((size_t)V * probs_chunk * 4), o_pst = cv.take((size_t)probs_stats_rows(V) * 16);
    const size_t o_prt = cv.take((size_t)M * probs_chunk * 4);
    const size_t total = cv.off ? cv.off : 256;
    void *mem = nullptr;
    if (!have_device) {
        set_error("no usable CUDA device (the membership itself is valid)");
        return PCG_ERR_CUDA;
    }
    e = cudaMalloc(&mem, total);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMalloc (group handle)");
    char *base = (char *)mem;
    e = upload(base, o_gptr, gptr);
    if (e == cudaSuccess) e = upload(base, o_gtok, gtok);
    if (e == cudaSuccess) e = upload(base, o_inv, inv);
    if (e == cudaSuccess) e = upload(base, o_rptr, rptr);
    if (e == cudaSuccess) e = upload(base, o_rgrp, rgrp);
    if (e == cudaSuccess) e = upload(base, o_eoff, eoff);
    if (e == cudaSuccess) e = upload(base, o_ent, ent);
    if (e == cudaSuccess) e = upload(base, o_w, w);
    if (e == cudaSuccess) e = upload(base, o_entw, entw);
    if (e == cudaSuccess) e = upload(base, o_rw, rw);
    if (e == cudaSuccess) e = upload(base, o_part, part_ptr);
    if (e == cudaSuccess) e = upload(base, o_pent, part_ent);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        cudaFree(mem);
        return cuda_fail(e, "uploading the group handle");
    }
    pcg_groups *h = new (std::nothrow) pcg_groups();
    if (!h) {
        cudaFree(mem);
        set_error("out of host memory");
        return PCG_ERR_INVALID_ARG;
    }
    h->dev.V = V;
    h->dev.M = M;
    h->dev.slices = C;
    h->dev.slice_len = SL;
    h->dev.groups_per_slice = (M + C - 1) / C;
    h->dev.group_ptr = (const int32_t *)(base + o_gptr);
    h->dev.group_tok = (const int32_t *)(base + o_gtok);
    h->dev.inv_deg = (const float *)(base + o_inv);
    h->dev.rev_ptr = (const int32_t *)(base + o_rptr);
    h->dev.rev_grp = (const int32_t *)(base + o_rgrp);
    h->dev.ent_off = (const int32_t *)(base + o_eoff);
    h->dev.ent = (const uint32_t *)(base + o_ent);
    h->dev.pair_w = w.empty() ? nullptr : (const float *)(base + o_w);
    h->dev.ent_w = w.empty() ? nullptr : (const float *)(base + o_entw);
    h->dev.rev_w = w.empty() ? nullptr : (const float *)(base + o_rw);
    h->dev.part_ptr = (const int32_t *)(base + o_part);
    h->dev.part_ent = (const int32_t *)(base + o_pent);
    h->dev.nparts = (int32_t)part_ptr.size() - 1;
    h->nnz = nnz;
    h->device = device;
    h->sm_count = sm_count;
    h->max_group_size = max_group;
    h->max_degree = max_deg;
    h->device_bytes = (int64_t)total;
    h->allocation = mem;
    h->agg_smem_bytes = has_sweep ? agg_smem_bytes(SL, M, C) : 0;
    h->has_sweep = has_sweep;
    h->accept_bias = 0.f;
    h->probs_chunk = probs_chunk;
    h->probs_dt = (float *)(base + o_pdt);
    h->probs_stats = (float4 *)(base + o_pst);
    h->probs_rt = (float *)(base + o_prt);
    *out = h;
    return PCG_OK;
}

extern "C" void pcg_groups_destroy(pcg_groups *groups) {
    if (!groups) return;
    cudaFree(groups->allocation);
    delete groups;
}

extern "C" pcg_status pcg_groups_info(const pcg_groups *groups, pcg_groups_info_t *out) {
    if (!groups || !out) {
        pcg::set_error("pcg_groups_info: null argument");
        return PCG_ERR_INVALID_ARG;
    }
    out->V = groups->dev.V;
    out->M = groups->dev.M;
    out->nnz = groups->nnz;
    out->slices = groups->has_sweep ? groups->dev.slices : 0;
    out->slice_len = groups->dev.slice_len;
    out->max_group_size = groups->max_group_size;
    out->max_degree = groups->max_degree;
    out->device = groups->device;
    out->has_weights = groups->dev.pair_w != nullptr;
    out->device_bytes = groups->device_bytes;
    return PCG_OK;
}

extern "C" pcg_status pcg_groups_set_accept_bias(pcg_groups *groups, float bias) {
    if (!groups || !std::isfinite(bias) || bias < 0.f) {
        pcg::set_error("pcg_groups_set_accept_bias: null handle, or a bias that is negative or not finite");
        return PCG_ERR_INVALID_ARG;
    }
    groups->accept_bias = bias;
    return PCG_OK;
}
