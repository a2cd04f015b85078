// Group construction on the GPU: cosine-threshold neighbourhoods of an embedding table, distinct sets, CSR.
// One-time set-up (the groups are precomputed once and cached); not part of the verification hot path.
//
// Stages (all on the device):
//   asg_prepare_kernel      rows to bfloat16 (zero-padded to a multiple of 32 columns and 128 rows), 1/|row| in fp32
//   asg_similarity_tc_kernel  E * E^T on the tensor cores (tcgen05, TMA; asg_similarity_kernel is the mma.sync form);
//                           the epilogue turns each dot product into cos = dot * rn_i * rn_j, compares with theta
//                           and packs the decisions into a V x V BIT matrix (the similarities are never stored);
//                           the tensor-core form computes only the tiles on or right of the diagonal blocks
//   asg_mirror_kernel       (tensor-core form) the lower triangle of the bit matrix as the transpose of the upper
//   asg_row_kernel          per row: population count and a position-aware 64-bit hash of its bit row
//   asg_representative_kernel  rep(t) = smallest t' with G(t') == G(t).  Such a t' is itself a member of G(t)
//                           (t' is in G(t') = G(t)), so only the set bits below t are candidates: hash, then
//                           a full comparison of the two bit rows
//   scans, asg_fill_kernel  group numbers by ascending representative, group_ptr, token lists from the bit rows,
//                           token degrees by counting
#include <cuda.h>  // CUtensorMap and its enums only; the encoder is fetched through the runtime, not linked
#include <cuda_bf16.h>

#include <algorithm>
#include <cmath>
#include <new>
#include <vector>

#include "pcg_common.cuh"

struct pcg_asg {
    int32_t V, M;
    int64_t nnz;
    int32_t max_group_size, max_degree;
    float similarity_ms, total_ms;
    int32_t *group_ptr, *group_tok, *tok_degree;  // device
    int32_t tensor_path;                          // 1 = tcgen05, 0 = mma.sync
};

namespace pcg {

constexpr int kAsgTile = 128;  // rows and columns of a similarity tile
constexpr int kAsgBK = 32;     // embedding columns per pipeline step
constexpr int kAsgLd = 40;     // shared-memory row stride in bf16 (80 bytes: 16-byte aligned, conflict-free ldmatrix)
constexpr int kAsgThreads = 256;

// ---------------------------------------------------------------------------------------------- prepare
// One warp per padded row.  out[r, :] = bf16(emb[r, :]) (exact for bf16 input), zero beyond d and beyond V;
// rnorm[r] = 1 / sqrt(sum of squares of the bf16 values) in fp32, 0 for a zero row.
template <typename T>
__global__ void asg_prepare_kernel(const T *emb, int V, int d, int dp, int Vp, __nv_bfloat16 *out, float *rnorm) {
    const int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (r >= Vp) return;
    float ss = 0.f;
    for (int c = lane; c < dp; c += 32) {
        __nv_bfloat16 v = __float2bfloat16_rn(0.f);
        if (r < V && c < d) {
            if (sizeof(T) == 2)
                v = reinterpret_cast<const __nv_bfloat16 *>(emb)[(size_t)r * d + c];
            else
                v = __float2bfloat16_rn(reinterpret_cast<const float *>(emb)[(size_t)r * d + c]);
        }
        out[(size_t)r * dp + c] = v;
        const float f = __bfloat162float(v);
        ss = __fmaf_rn(f, f, ss);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if (lane == 0) rnorm[r] = ss > 0.f ? 1.0f / sqrtf(ss) : 0.f;
}

// ---------------------------------------------------------------------------------------------- similarity
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void *smem) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"((uint32_t)__cvta_generic_to_shared(smem)));
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void asg_cp_async16(void *smem, const void *g) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem)), "l"(g)
                 : "memory");
}

// Grid (Vp/128, Vp/128), 256 threads = 8 warps as 2 x 4; a warp owns 64 x 32 of the tile (4 x 4 mma tiles).
// Both operands are row blocks of the same matrix E (the "B" operand is E^T, i.e. rows of E with the
// embedding index contiguous, which is the column-major form mma expects).  bits[V, W]: bit j of word w of row i
// says j' = 32 w + j is in G(i).
__global__ void __launch_bounds__(kAsgThreads) asg_similarity_kernel(const __nv_bfloat16 *E, const float *rnorm, int V,
                                                                    int dp, float theta, int W, uint32_t *bits) {
    constexpr int T = kAsgTile, BK = kAsgBK, LD = kAsgLd;
    __shared__ __align__(16) unsigned char smem_raw[2 * 2 * T * LD * 2];  // [stage][A|B][T][LD] bf16; reused for the decisions
    __nv_bfloat16 *sm = reinterpret_cast<__nv_bfloat16 *>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int wm = warp >> 2, wn = warp & 3;
    const int i0 = blockIdx.y * T, j0 = blockIdx.x * T;
    auto tile_ptr = [&](int stage, int which) { return sm + ((size_t)stage * 2 + which) * T * LD; };
    auto load_stage = [&](int stage, int k0) {
        // 128 rows x 32 bf16 = 4 chunks of 16 bytes per row, per operand: 512 chunks, 2 per thread
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            const int idx = tid + c * kAsgThreads, row = idx >> 2, ch = idx & 3;
            asg_cp_async16(tile_ptr(stage, 0) + row * LD + ch * 8, E + (size_t)(i0 + row) * dp + k0 + ch * 8);
            asg_cp_async16(tile_ptr(stage, 1) + row * LD + ch * 8, E + (size_t)(j0 + row) * dp + k0 + ch * 8);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    float acc[4][4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[a][b][c] = 0.f;
    const int nk = dp / BK;
    load_stage(0, 0);
    for (int kt = 0; kt < nk; ++kt) {
        if (kt + 1 < nk) {
            load_stage((kt + 1) & 1, (kt + 1) * BK);
            asm volatile("cp.async.wait_group 1;" ::: "memory");
        } else {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        __syncthreads();
        const __nv_bfloat16 *A = tile_ptr(kt & 1, 0) + (wm * 64) * LD, *B = tile_ptr(kt & 1, 1) + (wn * 32) * LD;
#pragma unroll
        for (int ks = 0; ks < BK; ks += 16) {
            uint32_t af[4][4], bf[2][4];
#pragma unroll
            for (int mi = 0; mi < 4; ++mi) ldmatrix_x4(af[mi], A + (mi * 16 + (lane & 15)) * LD + ks + (lane >> 4) * 8);
#pragma unroll
            for (int nj = 0; nj < 2; ++nj)  // two n8 tiles per ldmatrix: lanes 0-15 first tile (k 0-7, 8-15), 16-31 second
                ldmatrix_x4(bf[nj], B + (nj * 16 + (lane >> 4) * 8 + (lane & 7)) * LD + ks + ((lane >> 3) & 1) * 8);
#pragma unroll
            for (int mi = 0; mi < 4; ++mi)
#pragma unroll
                for (int ni = 0; ni < 4; ++ni) mma_bf16_16816(acc[mi][ni], af[mi], bf[ni >> 1][(ni & 1) * 2], bf[ni >> 1][(ni & 1) * 2 + 1]);
        }
        __syncthreads();  // the stage is overwritten by the load after next
    }
    // ---- decisions: one byte per (row, column) of the tile in shared memory, then 32 of them per word ----
    constexpr int PS = T + 16;  // byte stride of a decision row
    unsigned char *dec = smem_raw;
    float rni[4][2], rnj[4][2];
#pragma unroll
    for (int mi = 0; mi < 4; ++mi) {
        rni[mi][0] = rnorm[i0 + wm * 64 + mi * 16 + (lane >> 2)];
        rni[mi][1] = rnorm[i0 + wm * 64 + mi * 16 + (lane >> 2) + 8];
    }
#pragma unroll
    for (int ni = 0; ni < 4; ++ni) {
        rnj[ni][0] = rnorm[j0 + wn * 32 + ni * 8 + (lane & 3) * 2];
        rnj[ni][1] = rnorm[j0 + wn * 32 + ni * 8 + (lane & 3) * 2 + 1];
    }
#pragma unroll
    for (int mi = 0; mi < 4; ++mi)
#pragma unroll
        for (int ni = 0; ni < 4; ++ni)
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int r = wm * 64 + mi * 16 + (lane >> 2) + (c >> 1) * 8;
                const int q = wn * 32 + ni * 8 + (lane & 3) * 2 + (c & 1);
                const float cosv = __fmul_rn(__fmul_rn(acc[mi][ni][c], rni[mi][c >> 1]), rnj[ni][c & 1]);
                const bool in = (j0 + q < V) && (cosv > theta || i0 + r == j0 + q);
                dec[r * PS + q] = in ? 1 : 0;
            }
    __syncthreads();
    {
        const int r = tid >> 1;
        if (i0 + r < V) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int w = (tid & 1) * 2 + h;
                const uint4 *p = reinterpret_cast<const uint4 *>(dec + r * PS + w * 32);
                uint32_t word = 0;
#pragma unroll
                for (int v = 0; v < 2; ++v) {
                    const uint4 x = p[v];
                    const uint32_t q4[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                    for (int k = 0; k < 4; ++k)
#pragma unroll
                        for (int bb = 0; bb < 4; ++bb) word |= ((q4[k] >> (8 * bb)) & 1u) << (v * 16 + k * 4 + bb);
                }
                bits[(size_t)(i0 + r) * W + (j0 >> 5) + w] = word;
            }
        }
    }
}


// ---------------------------------------------------------------------------------------------- similarity, tcgen05
// Persistent, warp-specialised tiles on the 5th-generation tensor cores.  One block per SM walks the 128 x 256
// tiles of E * E^T; its warps have fixed roles that meet only through mbarriers:
//   warps 0-7  epilogue: read a finished 128 x 256 fp32 accumulator from tensor memory (tcgen05.ld, a warp may
//              touch the 32 lanes given by its index modulo 4; thread = accumulator row), turn it into 256
//              decisions cos > theta and write them as eight 32-bit words
//   warp 8     producer: one thread fetches the operands of the next K step (64 bf16 per row: a 128-row box of A and
//              two 128-row boxes of B) with TMA (cp.async.bulk.tensor, 128-byte swizzle) into a ring of stages; the
//              copies complete the stage's "full" barrier by byte count (expect_tx / complete_tx)
//   warp 9     one thread issues tcgen05.mma (M = 128, N = 256, K = 16, four per stage), hands each stage back to
//              the producers with tcgen05.commit on its "empty" barrier, and commits the tile's last K step on the
//              accumulator's "full" barrier
// The two 128 x 256 accumulators fill the SM's 512 columns of tensor memory, so the epilogue of one tile runs
// under the MMAs of the next.
//
// Shared-memory operand layout: the canonical K-major 128-byte-swizzle layout that TMA writes -- row r of a box at
// byte r * 128, its eight 16-byte chunks XOR-permuted by r % 8; groups of 8 rows are 1024 bytes apart (the
// descriptor's stride byte offset), every stage starts on a 1024-byte boundary, and a K step of 16 bf16 advances
// the descriptor's start address by 32 bytes inside the swizzled row.
// Every wait on an mbarrier is a bounded poll that also watches a block-wide failure flag: on a time-out the
// waiting role raises the flag, every role leaves its loop, the block drains its copies, frees its tensor memory,
// records an error code and returns.
constexpr int kTcBK = 64;        // bf16 per row and stage
constexpr int kTcTile = 256;     // columns of a tile (rows of the B operand); Vp is a multiple of it
constexpr int kTcRows = 128;     // rows of a tile (rows of the A operand) = lanes of tensor memory
constexpr int kTcStages = 4;     // stages of the operand ring
constexpr int kTcEpilogueWarps = 8, kTcProducerWarps = 1;
constexpr int kTcRasterRows = 16, kTcRasterCols = 8;  // tiles are visited in blocks of 16 x 8 (see tile_origin)
constexpr int kTcThreads = 32 * (kTcEpilogueWarps + kTcProducerWarps + 1);
constexpr int kTcABytes = kTcRows * kTcBK * 2, kTcBBytes = kTcTile * kTcBK * 2;
constexpr int kTcStageBytes = kTcABytes + kTcBBytes;
constexpr uint32_t kTcSpinLimit = 1u << 22;  // polls of about 50 ns each: gives up after a fraction of a second

// false = gave up (time-out, or another role raised the failure flag)
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, volatile int *failed) {
    for (uint32_t i = 0; i < kTcSpinLimit; ++i) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(bar), "r"(parity)
            : "memory");
        if (done) return true;
        if (*failed) return false;
        __nanosleep(20);
    }
    *failed = 1;
    return false;
}
__device__ __forceinline__ uint64_t umma_desc_kmajor_sw128(uint32_t smem_addr) {
    // start address >> 4 | leading byte offset field 1 (not used by swizzled K-major layouts) at bit 16 |
    // stride byte offset (1024: one group of 8 rows) >> 4 at bit 32 | descriptor version 1 at bit 46 |
    // layout type 2 (128-byte swizzle) at bit 61
    return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
           (2ull << 61);
}
// kind::f16 instruction descriptor: D = fp32 (1 << 4), A = B = bf16 (1 << 7, 1 << 10), both K-major,
// N = 256 (256 >> 3 at bit 17), M = 128 (128 >> 4 at bit 24)
constexpr uint32_t kTcIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((256u >> 3) << 17) | ((128u >> 4) << 24);

__global__ void __launch_bounds__(kTcThreads, 1) asg_similarity_tc_kernel(const __grid_constant__ CUtensorMap tmap,
                                                                         const float *rnorm, int V, int Vp, int dp,
                                                                         float theta, int W, uint32_t *bits,
                                                                         int *error) {
    constexpr int S = kTcStages, BK = kTcBK;
    extern __shared__ unsigned char tc_smem_raw[];  // [S][A 128 rows | B 256 rows][128 bytes per row], 1024-aligned below
    __shared__ __align__(8) uint64_t bars[2 * S + 5];          // full[S], empty[S], acc_full[2], acc_empty[2], drain
    __shared__ uint32_t tmem_slot;
    __shared__ int failed_flag;
    volatile int *failed = &failed_flag;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t smem_base = ((uint32_t)__cvta_generic_to_shared(tc_smem_raw) + 1023u) & ~1023u;
    const uint32_t bar0 = (uint32_t)__cvta_generic_to_shared(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (S + s); };
    auto acc_full_bar = [&](int b) { return bar0 + 8u * (2 * S + b); };
    auto acc_empty_bar = [&](int b) { return bar0 + 8u * (2 * S + 2 + b); };
    const uint32_t drain_bar = bar0 + 8u * (2 * S + 4);  // failure path only: all issued MMAs have retired
    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(full_bar(s)));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(empty_bar(s)));
        }
        for (int b = 0; b < 2; ++b) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(acc_full_bar(b)));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(acc_empty_bar(b)), "r"(32 * kTcEpilogueWarps));
        }
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(drain_bar));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        failed_flag = 0;
    }
    if (warp == 0) {  // tensor memory: all 512 columns (two 128 x 256 accumulators), allocated and freed by warp 0
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                         (uint32_t)__cvta_generic_to_shared(&tmem_slot)),
                     "r"(512));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = tmem_slot;
    const int nI = Vp / kTcRows, nJ = Vp / kTcTile, nk = dp / BK;
    // Tile numbers run through blocks of 16 row blocks x 8 column blocks (128 tiles, about one wave of the
    // persistent grid), so the tiles in flight at any time share 4096 rows of E (4 MB at d = 512) and the operands
    // come out of L2 rather than HBM; numbers that fall outside the matrix are skipped by every role alike.
    const int sbI = (nI + kTcRasterRows - 1) / kTcRasterRows, sbJ = (nJ + kTcRasterCols - 1) / kTcRasterCols;
    const int ntiles = sbI * sbJ * kTcRasterRows * kTcRasterCols;
    auto tile_origin = [&](int tile, int &i0, int &j0) -> bool {
        const int sb = tile / (kTcRasterRows * kTcRasterCols), local = tile % (kTcRasterRows * kTcRasterCols);
        const int ti = (sb / sbJ) * kTcRasterRows + local % kTcRasterRows;
        const int tj = (sb % sbJ) * kTcRasterCols + local / kTcRasterRows;
        i0 = ti * kTcRows;
        j0 = tj * kTcTile;
        // The cosine is symmetric: only tiles that reach the diagonal block of 256 columns of their rows, or lie to
        // its right, are computed (column block tj >= row block ti / 2); asg_mirror_kernel fills in the rest.
        return ti < nI && tj < nJ && tj >= ti * kTcRows / kTcTile;
    };

    if (warp < kTcEpilogueWarps) {
        // ------------------------------------------------------------------ epilogue warps
        // warps 0-3 take columns 0-127 of the accumulator, warps 4-7 columns 128-255; a warp may only touch the 32
        // lanes of tensor memory given by its index modulo 4.  Thread = accumulator row, 128 decisions = 4 words.
        const int quarter = warp & 3, chalf = warp >> 2;
        int tcount = 0;
        for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
            int i0, j0;
            if (!tile_origin(tile, i0, j0)) continue;
            const int buf = tcount & 1;
            const int r = quarter * 32 + lane, c0 = chalf * 128;
            const float rni = rnorm[i0 + r];
            float rnq[4];  // 1/|column| of columns c0 + 32 q + lane, handed round by shuffle below
#pragma unroll
            for (int q = 0; q < 4; ++q) rnq[q] = rnorm[j0 + c0 + q * 32 + lane];
            const bool ready = mbar_wait_bounded(acc_full_bar(buf), (tcount >> 1) & 1, failed);
            if (!__all_sync(0xffffffffu, ready)) break;  // warp-uniform: tcgen05.ld below needs the whole warp
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            uint32_t words[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint32_t v[32];
                const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * 256 + c0 + q * 32);
                asm volatile(
                    "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, "
                    "%14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                    : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                      "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]),
                      "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]),
                      "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]),
                      "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                    : "r"(taddr));
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                uint32_t word = 0;
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    const float rnc = __shfl_sync(0xffffffffu, rnq[q], c);
                    const float cosv = __fmul_rn(__fmul_rn(__uint_as_float(v[c]), rni), rnc);
                    word |= (cosv > theta ? 1u : 0u) << c;
                }
                // t is always a member of G(t); columns past the end of the vocabulary are never members
                const int first = j0 + c0 + q * 32, diag = i0 + r - first;
                if (diag >= 0 && diag < 32) word |= 1u << diag;
                const int valid = V - first;
                if (valid < 32) word = valid <= 0 ? 0u : (word & ((1u << valid) - 1u));
                words[q] = word;
            }
            // the accumulator may be overwritten: hand it back to the MMA warp before the stores
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(acc_empty_bar(buf)) : "memory");
            if (i0 + r < V)
                *reinterpret_cast<uint4 *>(bits + (size_t)(i0 + r) * W + ((j0 + c0) >> 5)) =
                    make_uint4(words[0], words[1], words[2], words[3]);
            ++tcount;
        }
    } else if (warp < kTcEpilogueWarps + kTcProducerWarps) {
        // ------------------------------------------------------------------ producer (one thread)
        if (lane == 0) {
            const uint64_t map = reinterpret_cast<uint64_t>(&tmap);
            int it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
                int i0, j0;
                if (!tile_origin(tile, i0, j0)) continue;
                for (int kt = 0; kt < nk; ++kt, ++it) {
                    const int s = it % S;
                    if (it >= S && !mbar_wait_bounded(empty_bar(s), ((it / S) - 1) & 1, failed)) {
                        ok = false;
                        break;
                    }
                    const uint32_t a = smem_base + (uint32_t)(s * kTcStageBytes), b = a + kTcABytes, bar = full_bar(s);
                    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(kTcStageBytes)
                                 : "memory");
                    const int k0 = kt * BK;  // inner coordinate: a multiple of 64 elements = 128 bytes
                    auto tma_box = [&](uint32_t dst, int row) {  // 128 rows x 64 bf16 of E starting at (row, k0)
                        asm volatile(
                            "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, "
                            "%3}], [%4];" ::"r"(dst),
                            "l"(map), "r"(k0), "r"(row), "r"(bar)
                            : "memory");
                    };
                    tma_box(a, i0);
                    tma_box(b, j0);
                    tma_box(b + kTcABytes, j0 + 128);
                }
            }
            if (*failed) {
                // Giving up: copies already requested may still be landing in shared memory.  Wait (bounded, and no
                // longer cut short by the failure flag) for the last S armed stages before the block may end.
                for (int back = 1; back <= S && back <= it; ++back) {
                    const int j = it - back, s = j % S;
                    for (uint32_t spin = 0; spin < kTcSpinLimit; ++spin) {
                        uint32_t done;
                        asm volatile(
                            "{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                            : "=r"(done)
                            : "r"(full_bar(s)), "r"((uint32_t)((j / S) & 1))
                            : "memory");
                        if (done) break;
                        __nanosleep(20);
                    }
                }
            }
        }
    } else if (warp == kTcEpilogueWarps + kTcProducerWarps && lane == 0) {
        // ------------------------------------------------------------------ MMA issuer (one thread)
        int it = 0, tcount = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
            int i0, j0;
            if (!tile_origin(tile, i0, j0)) continue;
            const int buf = tcount & 1;
            if (tcount >= 2 && !mbar_wait_bounded(acc_empty_bar(buf), ((tcount >> 1) - 1) & 1, failed)) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            for (int kt = 0; kt < nk; ++kt, ++it) {
                const int s = it % S;
                if (!mbar_wait_bounded(full_bar(s), (it / S) & 1, failed)) {
                    ok = false;
                    break;
                }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t a = smem_base + (uint32_t)(s * kTcStageBytes), b = a + kTcABytes;
#pragma unroll
                for (int kk = 0; kk < BK / 16; ++kk) {
                    const uint64_t da = umma_desc_kmajor_sw128(a + kk * 32), db = umma_desc_kmajor_sw128(b + kk * 32);
                    const uint32_t accumulate = (kt > 0 || kk > 0) ? 1u : 0u;
                    asm volatile(
                        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
                        :
                        : "r"(tmem + buf * 256), "l"(da), "l"(db), "r"(kTcIdesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u),
                          "r"(0u)
                        : "memory");
                }
                // arrives when every MMA issued so far has finished reading the stage: the producers may refill it
                asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(empty_bar(s))
                             : "memory");
            }
            if (ok)  // ... and when the tile's accumulator is complete
                asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                                 acc_full_bar(buf))
                             : "memory");
            ++tcount;
        }
        if (*failed) {
            // Giving up: MMAs already issued may still be writing tensor memory.  One more commit arrives on a
            // barrier of its own when all of them have retired; wait for it (bounded) before the memory is freed.
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(drain_bar)
                         : "memory");
            for (uint32_t spin = 0; spin < kTcSpinLimit; ++spin) {
                uint32_t done;
                asm volatile(
                    "{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                    : "=r"(done)
                    : "r"(drain_bar), "r"(0u)
                    : "memory");
                if (done) break;
                __nanosleep(20);
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (tid == 0 && failed_flag) atomicMax(error, 1);
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512));
}

// The lower triangle of the bit matrix from the upper one (cos is symmetric, so t' in G(t) iff t in G(t')): the
// block of 256 rows x 256 columns at (TR, TC), TC < TR, is the transpose of the block at (TC, TR).  One thread block
// per such pair: 256 rows x 32 bytes in (whole sectors), the 256 x 256 bits turned 32 x 32 at a time by exchanges
// between lanes (lane = input row before, output row after), 256 rows x 32 bytes out.
constexpr int kMirrorBits = 256;
static_assert(kMirrorBits == kTcTile, "the tensor-core kernel computes whole diagonal blocks of this size");
__global__ void __launch_bounds__(kMirrorBits) asg_mirror_kernel(uint32_t *bits, int V, int W) {
    const int TR = blockIdx.y, TC = blockIdx.x;
    if (TC >= TR) return;
    constexpr int WB = kMirrorBits / 32;  // words per block row
    __shared__ uint32_t win[kMirrorBits][WB + 1], wout[kMirrorBits][WB + 1];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    {
        const int row = TC * kMirrorBits + tid;
        uint4 a = make_uint4(0u, 0u, 0u, 0u), b = a;
        if (row < V) {
            const uint4 *src = reinterpret_cast<const uint4 *>(bits + (size_t)row * W + (size_t)TR * WB);
            a = src[0];
            b = src[1];
        }
        win[tid][0] = a.x, win[tid][1] = a.y, win[tid][2] = a.z, win[tid][3] = a.w;
        win[tid][4] = b.x, win[tid][5] = b.y, win[tid][6] = b.z, win[tid][7] = b.w;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < WB; ++k) {
        // lane = input row 32 warp + lane, bits = columns 32 k .. 32 k + 31: the 32 x 32 bit block is transposed across
        // the lanes in five exchange steps (blocks of 16, 8, 4, 2, 1 swapped across the diagonal)
        uint32_t x = win[32 * warp + lane][k];
#pragma unroll
        for (int j = 16; j > 0; j >>= 1) {
            const uint32_t m = j == 16 ? 0x0000ffffu : j == 8 ? 0x00ff00ffu : j == 4 ? 0x0f0f0f0fu : j == 2 ? 0x33333333u : 0x55555555u;
            const uint32_t partner = __shfl_xor_sync(0xffffffffu, x, j);
            x = (lane & j) ? ((x & ~m) | ((partner & ~m) >> j)) : ((x & m) | ((partner & m) << j));
        }
        wout[32 * k + lane][warp] = x;  // output row 32 k + lane, columns 32 warp .. 32 warp + 31
    }
    __syncthreads();
    {
        const int row = TR * kMirrorBits + tid;
        if (row < V) {
            uint4 *dst = reinterpret_cast<uint4 *>(bits + (size_t)row * W + (size_t)TC * WB);
            dst[0] = make_uint4(wout[tid][0], wout[tid][1], wout[tid][2], wout[tid][3]);
            dst[1] = make_uint4(wout[tid][4], wout[tid][5], wout[tid][6], wout[tid][7]);
        }
    }
}

// ---------------------------------------------------------------------------------------------- rows
__device__ __forceinline__ uint64_t mix64(uint64_t x) {  // splitmix64 finaliser
    x ^= x >> 30;
    x *= 0xbf58476d1ce4e5b9ull;
    x ^= x >> 27;
    x *= 0x94d049bb133111ebull;
    x ^= x >> 31;
    return x;
}

// One warp per row: number of members and a hash of the bit row (sum of mixed (word, position) pairs, so it
// does not depend on the order in which the lanes visit the words).
__global__ void asg_row_kernel(const uint32_t *bits, int V, int W, int32_t *count, uint64_t *hash) {
    const int t = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (t >= V) return;
    const uint32_t *row = bits + (size_t)t * W;
    int n = 0;
    uint64_t h = 0;
    for (int w = lane; w < W; w += 32) {
        const uint32_t x = row[w];
        n += __popc(x);
        if (x) h += mix64(((uint64_t)(uint32_t)w << 32) | x);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        n += __shfl_xor_sync(0xffffffffu, n, o);
        h += __shfl_xor_sync(0xffffffffu, h, o);
    }
    if (lane == 0) {
        count[t] = n;
        hash[t] = h;
    }
}

// One warp per row t: the smallest member t' < t of G(t) whose bit row equals row t, else t itself.
__global__ void asg_representative_kernel(const uint32_t *bits, int V, int W, const int32_t *count,
                                          const uint64_t *hash, int32_t *rep) {
    const int t = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (t >= V) return;
    const uint32_t *row = bits + (size_t)t * W;
    const uint64_t ht = hash[t];
    const int ct = count[t];
    int found = t;
    for (int w0 = 0; w0 * 32 < t && found == t; w0 += 32) {  // 32 words = 1024 candidate tokens per round
        const int w = w0 + lane;
        uint32_t x = (w < W) ? row[w] : 0u;
        if (w * 32 + 31 >= t) {  // keep candidates below t only
            const int keep = t - w * 32;
            x = keep <= 0 ? 0u : (keep >= 32 ? x : (x & ((1u << keep) - 1u)));
        }
        while (true) {
            // smallest remaining candidate of this round whose hash and size match
            int cand = 0x7fffffff;
            while (x) {
                const int j = w * 32 + __ffs(x) - 1;
                if (hash[j] == ht && count[j] == ct) {
                    cand = j;
                    break;
                }
                x &= x - 1;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) cand = min(cand, __shfl_xor_sync(0xffffffffu, cand, o));
            if (cand == 0x7fffffff) break;
            const uint32_t *other = bits + (size_t)cand * W;
            bool same = true;
            for (int k = lane; k < W; k += 32) same = same && (row[k] == other[k]);
            if (__all_sync(0xffffffffu, same)) {
                found = cand;
                break;
            }
            if ((cand >> 5) == w) x &= ~(1u << (cand & 31));  // a hash collision: drop it and look on
        }
    }
    if (lane == 0) rep[t] = found;
}

// Exclusive prefix sum of n ints by one block (set-up sizes: n <= 2^20), total to out[n]: a contiguous run per
// thread, the 1024 run totals scanned by warp shuffles (32 warp scans, then one over the warps' totals).
__global__ void __launch_bounds__(1024) asg_scan_kernel(const int32_t *in, int n, int32_t *out) {
    __shared__ int32_t warp_tot[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, per = (n + 1023) / 1024;
    const int lo = min(n, tid * per), hi = min(n, lo + per);
    int32_t s = 0;
    for (int i = lo; i < hi; ++i) s += in[i];
    int32_t inc = s;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int32_t up = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += up;
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        int32_t w = warp_tot[lane], winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int32_t up = __shfl_up_sync(0xffffffffu, winc, o);
            if (lane >= o) winc += up;
        }
        warp_tot[lane] = winc - w;  // exclusive prefix of the warps' totals
        if (lane == 31) out[n] = winc;
    }
    __syncthreads();
    int32_t run = warp_tot[warp] + inc - s;
    for (int i = lo; i < hi; ++i) {
        const int32_t v = in[i];
        out[i] = run;
        run += v;
    }
}

__global__ void asg_flag_kernel(const int32_t *rep, int V, int32_t *is_rep) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t < V) is_rep[t] = rep[t] == t;
}

// sizes[g] = |G(t)| for the representative t of group g = gid[t]
__global__ void asg_sizes_kernel(const int32_t *rep, const int32_t *gid, const int32_t *count, int V, int32_t *sizes) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t < V && rep[t] == t) sizes[gid[t]] = count[t];
}

// One warp per representative row: its set bits, ascending, into group_tok[group_ptr[g] ...]; degrees by counting.
__global__ void asg_fill_kernel(const uint32_t *bits, int V, int W, const int32_t *rep, const int32_t *gid,
                                const int32_t *group_ptr, int32_t *group_tok, int32_t *degree) {
    const int t = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (t >= V || rep[t] != t) return;
    const uint32_t *row = bits + (size_t)t * W;
    int base = group_ptr[gid[t]];
    for (int w0 = 0; w0 < W; w0 += 32) {
        const int w = w0 + lane;
        uint32_t x = w < W ? row[w] : 0u;
        const int n = __popc(x);
        int incl = n;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += up;
        }
        int at = base + incl - n;
        while (x) {
            const int j = w * 32 + __ffs(x) - 1;
            group_tok[at++] = j;
            atomicAdd(&degree[j], 1);
            x &= x - 1;
        }
        base += __shfl_sync(0xffffffffu, incl, 31);
    }
}

__global__ void asg_max_kernel(const int32_t *a, int n, int32_t *out) {  // out must hold 0 on entry
    int m = 0;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) m = max(m, a[i]);
    atomicMax(out, m);
}

}  // namespace pcg

// ================================================================================================ host side
using namespace pcg;

namespace {
struct DeviceBuffers {  // frees whatever was allocated when it goes out of scope
    std::vector<void *> ptrs;
    cudaError_t alloc(void **p, size_t bytes) {
        cudaError_t e = cudaMalloc(p, bytes ? bytes : 1);
        if (e == cudaSuccess) ptrs.push_back(*p);
        return e;
    }
    void release(void *keep) {  // forget one pointer (it now belongs to the result)
        for (auto &q : ptrs)
            if (q == keep) q = nullptr;
    }
    ~DeviceBuffers() {
        for (void *q : ptrs)
            if (q) cudaFree(q);
    }
};
}  // namespace

extern "C" pcg_status pcg_asg_create(const void *emb, pcg_dtype dtype, int32_t V, int32_t d, float theta,
                                     uint32_t flags, pcg_asg **out) {
    if (out) *out = nullptr;
    if (!emb || !out || V < 1 || d < 1 || (dtype != PCG_F32 && dtype != PCG_BF16) || !std::isfinite(theta)) {
        set_error("pcg_asg_create: null pointer, V < 1, d < 1, bad dtype or a threshold that is not finite");
        return PCG_ERR_INVALID_ARG;
    }
    if (flags & ~PCG_ASG_MMA_SYNC) {
        set_error("pcg_asg_create: unknown flag bits 0x%x", flags);
        return PCG_ERR_INVALID_ARG;
    }
    if (V > (1 << 20)) {
        set_error("pcg_asg_create: V=%d exceeds 2^20 (the bit matrix would need %lld GB)", V,
                  (long long)((int64_t)V * V / 8 >> 30));
        return PCG_ERR_UNSUPPORTED;
    }
    const int Vp = (V + kTcTile - 1) / kTcTile * kTcTile, dp = (d + kTcBK - 1) / kTcBK * kTcBK, W = Vp / 32;
    DeviceBuffers buf;
    __nv_bfloat16 *E = nullptr;
    float *rnorm = nullptr;
    uint32_t *bits = nullptr;
    int32_t *count = nullptr, *rep = nullptr, *flag = nullptr, *gid = nullptr, *sizes = nullptr, *gptr = nullptr;
    int32_t *gtok = nullptr, *deg = nullptr, *maxes = nullptr;
    uint64_t *hash = nullptr;
    cudaError_t e = buf.alloc((void **)&E, (size_t)Vp * dp * 2);
    if (e == cudaSuccess) e = buf.alloc((void **)&rnorm, (size_t)Vp * 4);
    if (e == cudaSuccess) e = buf.alloc((void **)&bits, (size_t)V * W * 4);
    if (e == cudaSuccess) e = buf.alloc((void **)&count, (size_t)V * 4);
    if (e == cudaSuccess) e = buf.alloc((void **)&hash, (size_t)V * 8);
    if (e == cudaSuccess) e = buf.alloc((void **)&rep, (size_t)V * 4);
    if (e == cudaSuccess) e = buf.alloc((void **)&flag, (size_t)V * 4);
    if (e == cudaSuccess) e = buf.alloc((void **)&gid, ((size_t)V + 1) * 4);
    if (e == cudaSuccess) e = buf.alloc((void **)&sizes, (size_t)V * 4);
    if (e == cudaSuccess) e = buf.alloc((void **)&gptr, ((size_t)V + 1) * 4);
    if (e == cudaSuccess) e = buf.alloc((void **)&deg, (size_t)V * 4);
    if (e == cudaSuccess) e = buf.alloc((void **)&maxes, 16);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMalloc (group construction)");
    cudaEvent_t ev[4] = {nullptr, nullptr, nullptr, nullptr};
    for (auto &x : ev)
        if (e == cudaSuccess) e = cudaEventCreate(&x);
    auto drop_events = [&]() {
        for (auto &x : ev)
            if (x) cudaEventDestroy(x);
    };
    if (e != cudaSuccess) {
        drop_events();
        return cuda_fail(e, "cudaEventCreate");
    }
    const int rows_per_block = 8, row_blocks = (V + rows_per_block - 1) / rows_per_block;
    cudaEventRecord(ev[0], 0);
    if (dtype == PCG_BF16)
        asg_prepare_kernel<uint16_t><<<(Vp + 7) / 8, 256>>>((const uint16_t *)emb, V, d, dp, Vp, E, rnorm);
    else
        asg_prepare_kernel<float><<<(Vp + 7) / 8, 256>>>((const float *)emb, V, d, dp, Vp, E, rnorm);
    cudaMemsetAsync(maxes, 0, 16, 0);  // [0] largest group, [1] largest degree, [2] error code of the tensor-core kernel
    cudaEventRecord(ev[1], 0);
    const dim3 tiles(Vp / kAsgTile, Vp / kAsgTile);
    if (flags & PCG_ASG_MMA_SYNC) {
        asg_similarity_kernel<<<tiles, kAsgThreads>>>(E, rnorm, V, dp, theta, W, bits);
    } else {
        // TMA descriptor of E as a [Vp rows, dp columns] bf16 matrix, boxes of 128 rows x 64 columns, 128-byte swizzle
        typedef CUresult (*EncodeTiled)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                        const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                        CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres = cudaDriverEntryPointSymbolNotFound;
        e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
            drop_events();
            set_error("pcg_asg_create: the driver does not provide cuTensorMapEncodeTiled");
            return PCG_ERR_CUDA;
        }
        alignas(64) CUtensorMap tmap;
        const cuuint64_t gdim[2] = {(cuuint64_t)dp, (cuuint64_t)Vp}, gstride[1] = {(cuuint64_t)dp * 2};
        const cuuint32_t box[2] = {(cuuint32_t)kTcBK, 128u}, estride[2] = {1u, 1u};
        const CUresult cr = ((EncodeTiled)fn)(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, E, gdim, gstride, box, estride,
                                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (cr != CUDA_SUCCESS) {
            drop_events();
            set_error("pcg_asg_create: cuTensorMapEncodeTiled failed (%d)", (int)cr);
            return PCG_ERR_CUDA;
        }
        const int smem = kTcStages * kTcStageBytes + 1024;  // room to start the stages on a 1024-byte boundary
        e = cudaFuncSetAttribute(asg_similarity_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) {
            drop_events();
            return cuda_fail(e, "cudaFuncSetAttribute (asg_similarity_tc_kernel)");
        }
        int dev = 0, sms = 1;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        const int ntiles = (Vp / kTcRows) * (Vp / kTcTile);
        asg_similarity_tc_kernel<<<std::min(sms, std::max(1, ntiles)), kTcThreads, smem>>>(tmap, rnorm, V, Vp, dp, theta, W,
                                                                                          bits, maxes + 2);
        const int nT = Vp / kMirrorBits;
        if (nT > 1) asg_mirror_kernel<<<dim3(nT, nT), kMirrorBits>>>(bits, V, W);
    }
    cudaEventRecord(ev[2], 0);
    {
        int32_t tc_error = 0;
        e = cudaMemcpy(&tc_error, maxes + 2, 4, cudaMemcpyDeviceToHost);
        if (e == cudaSuccess && tc_error) {
            drop_events();
            set_error("pcg_asg_create: the tensor-core pipeline gave up waiting on a barrier (code %d)", tc_error);
            return PCG_ERR_CUDA;
        }
        if (e != cudaSuccess) {
            drop_events();
            return cuda_fail(e, "similarity kernel");
        }
    }
    asg_row_kernel<<<row_blocks, 256>>>(bits, V, W, count, hash);
    asg_representative_kernel<<<row_blocks, 256>>>(bits, V, W, count, hash, rep);
    asg_flag_kernel<<<(V + 255) / 256, 256>>>(rep, V, flag);
    asg_scan_kernel<<<1, 1024>>>(flag, V, gid);  // gid[t] = group number of a representative t; gid[V] = M
    int32_t M = 0;
    e = cudaMemcpy(&M, gid + V, 4, cudaMemcpyDeviceToHost);
    if (e == cudaSuccess) {
        asg_sizes_kernel<<<(V + 255) / 256, 256>>>(rep, gid, count, V, sizes);
        asg_scan_kernel<<<1, 1024>>>(sizes, M, gptr);
    }
    int32_t nnz = 0;
    if (e == cudaSuccess) e = cudaMemcpy(&nnz, gptr + M, 4, cudaMemcpyDeviceToHost);
    if (e == cudaSuccess) e = buf.alloc((void **)&gtok, (size_t)nnz * 4);
    if (e == cudaSuccess) e = cudaMemsetAsync(deg, 0, (size_t)V * 4, 0);
    int32_t mx[2] = {0, 0};
    float sim_ms = 0.f, total_ms = 0.f;
    if (e == cudaSuccess) {
        asg_fill_kernel<<<row_blocks, 256>>>(bits, V, W, rep, gid, gptr, gtok, deg);
        asg_max_kernel<<<64, 256>>>(sizes, M, maxes);
        asg_max_kernel<<<64, 256>>>(deg, V, maxes + 1);
        cudaEventRecord(ev[3], 0);
        e = cudaMemcpy(mx, maxes, 8, cudaMemcpyDeviceToHost);
    }
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e == cudaSuccess) {
        cudaEventElapsedTime(&sim_ms, ev[1], ev[2]);
        cudaEventElapsedTime(&total_ms, ev[0], ev[3]);
    }
    drop_events();
    if (e != cudaSuccess) return cuda_fail(e, "group construction");
    // the result keeps exact-size copies of group_ptr; group_tok and the degrees are handed over as they are
    int32_t *gptr_out = nullptr;
    e = buf.alloc((void **)&gptr_out, ((size_t)M + 1) * 4);
    if (e == cudaSuccess) e = cudaMemcpy(gptr_out, gptr, ((size_t)M + 1) * 4, cudaMemcpyDeviceToDevice);
    if (e != cudaSuccess) return cuda_fail(e, "copying group_ptr");
    pcg_asg *r = new (std::nothrow) pcg_asg();
    if (!r) {
        set_error("out of host memory");
        return PCG_ERR_INVALID_ARG;
    }
    r->V = V;
    r->M = M;
    r->nnz = nnz;
    r->max_group_size = mx[0];
    r->max_degree = mx[1];
    r->similarity_ms = sim_ms;
    r->total_ms = total_ms;
    r->tensor_path = (flags & PCG_ASG_MMA_SYNC) ? 0 : 1;
    r->group_ptr = gptr_out;
    r->group_tok = gtok;
    r->tok_degree = deg;
    buf.release(gptr_out);
    buf.release(gtok);
    buf.release(deg);
    *out = r;
    return PCG_OK;
}

extern "C" pcg_status pcg_asg_info(const pcg_asg *asg, pcg_asg_info_t *out) {
    if (!asg || !out) {
        set_error("pcg_asg_info: null argument");
        return PCG_ERR_INVALID_ARG;
    }
    out->V = asg->V;
    out->M = asg->M;
    out->nnz = asg->nnz;
    out->max_group_size = asg->max_group_size;
    out->max_degree = asg->max_degree;
    out->similarity_ms = asg->similarity_ms;
    out->total_ms = asg->total_ms;
    out->tensor_path = asg->tensor_path;
    return PCG_OK;
}

extern "C" pcg_status pcg_asg_csr(const pcg_asg *asg, pcg_csr *out) {
    if (!asg || !out) {
        set_error("pcg_asg_csr: null argument");
        return PCG_ERR_INVALID_ARG;
    }
    out->V = asg->V;
    out->M = asg->M;
    out->nnz = asg->nnz;
    out->group_ptr = asg->group_ptr;
    out->group_tok = asg->group_tok;
    out->tok_degree = asg->tok_degree;
    out->weights = nullptr;
    return PCG_OK;
}

extern "C" void pcg_asg_destroy(pcg_asg *asg) {
    if (!asg) return;
    cudaFree(asg->group_ptr);
    cudaFree(asg->group_tok);
    cudaFree(asg->tok_degree);
    delete asg;
}
