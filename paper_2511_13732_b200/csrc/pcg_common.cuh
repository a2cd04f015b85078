// Shared device helpers and the group handle of libpcg (sm_100a only).
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "pcg.h"

#ifndef __CUDA_ARCH__
#define PCG_HOST_ONLY 1
#endif

namespace pcg {

constexpr float kNegInf = -__builtin_huge_valf();
constexpr int kAggThreads = 512;        // threads per block of the aggregation kernels (fixes the sweep layout)
constexpr uint32_t kNoGroup = 0xffffu;  // group field of sweep entries that belong to no group
constexpr int kPartMaxGroups = 8;       // a part of the sparse product holds at most this many consecutive groups
constexpr int kPartWarpsPerSM = 20;     // parts are sized so that one warp per part fills the GPU about once

// Device-resident membership, built once by pcg_groups_create.
struct GroupsDev {
    int32_t V, M;
    int32_t slices;     // C: token slices per row = cluster size of the aggregation kernels
    int32_t slice_len;  // tokens per slice (multiple of 64)
    int32_t groups_per_slice;  // ceil(M / C): groups whose totals a CTA of the cluster owns
    const int32_t *group_ptr;  // [M+1]   original CSR
    const int32_t *group_tok;  // [nnz]
    const float *inv_deg;      // [V]     1/N(t)
    const int32_t *rev_ptr;    // [V+1]   reverse membership S(t), ascending group id
    const int32_t *rev_grp;    // [nnz]
    // Token-sliced copy of the CSR for the aggregation sweep.  Slice c owns entries [ent_off[c], ent_off[c+1]),
    // a whole number of rows of kAggThreads entries; thread t walks column t (entry j of thread t sits at
    // row j, so a warp reads consecutive words).  An entry is (group id << 16) | in-slice token offset; all
    // entries of one (slice, group) pair are consecutive in one thread's column, in CSR order.  Columns are
    // padded with entries that point at the always-zero slot `slice_len` (group kNoGroup if the thread owns
    // no group in this slice).
    const int32_t *ent_off;    // [C+1]
    const uint32_t *ent;       // [ent_off[C]]
    const float *ent_w;        // [ent_off[C]] weights in the same layout, or nullptr (equal split)
    const float *pair_w;       // [nnz] CSR-order weights w_{g,t} or nullptr (equal split)
    const float *rev_w;        // [nnz] the same in reverse-membership order, or nullptr
    // Partition of the groups for the sparse product: part p is the run of whole groups [part_ptr[p], part_ptr[p+1]),
    // at most kPartMaxGroups of them, cut so that every part holds about the same number of stored pairs.
    const int32_t *part_ptr;   // [nparts+1]
    const int32_t *part_ent;   // [nparts+1] group_ptr[part_ptr[p]]: the first stored pair of part p
    int32_t nparts;
};

}  // namespace pcg

struct pcg_groups {
    pcg::GroupsDev dev;
    int64_t nnz;
    int device;
    int sm_count;
    int max_group_size;
    int max_degree;
    int64_t device_bytes;
    void *allocation;  // single device allocation holding every array
    size_t agg_smem_bytes;  // dynamic shared memory of the aggregation kernels
    float accept_bias;      // constant added to the acceptance ratio (0 = PCG)
    bool has_sweep;         // the token-sliced sweep layout exists (M <= 65534 and it fits in shared memory)
    // scratch of the batched route of pcg_group_probs (inside `allocation`): rows are processed in chunks of
    // probs_chunk; the transposed operand Dt[V, probs_chunk] and per-row statistics
    int probs_chunk;
    float *probs_dt;
    float4 *probs_stats;  // [probs_stats_rows]
    float *probs_rt;  // [M, probs_chunk] group-major sums of one chunk
};

namespace pcg {

void set_error(const char *fmt, ...);
pcg_status cuda_fail(cudaError_t e, const char *what);

inline bool valid_dtype(pcg_dtype d) { return d == PCG_F32 || d == PCG_BF16 || d == PCG_F16; }
inline size_t dtype_bytes(pcg_dtype d) { return d == PCG_F32 ? 4 : 2; }

// Rows per chunk of the batched route of pcg_group_probs: 128, or 256 while the transposed operand of a chunk
// (4 * V bytes per row) stays within 64 MB, so that it remains L2-resident.
inline int probs_chunk_rows(int V) {
    const int64_t fit = ((int64_t)64 << 20) / ((int64_t)V * 4) / 128 * 128;
    return (int)(fit < 128 ? 128 : (fit > 256 ? 256 : fit));
}

// Rows whose softmax statistics the batched route forms in ONE launch ahead of their chunks (a launch per chunk
// of 128 or 256 rows leaves most of the GPU idle): sixteen chunks.
inline int probs_stats_rows(int V) { return 16 * probs_chunk_rows(V); }

// Runs `...` with LogitT bound to the element type of `dtype` (float, uint16_t for bfloat16 bit patterns, f16_t).
#define PCG_DISPATCH_DTYPE(dtype, ...)        \
    do {                                      \
        if ((dtype) == PCG_F32) {             \
            using LogitT = float;             \
            __VA_ARGS__;                      \
        } else if ((dtype) == PCG_BF16) {     \
            using LogitT = uint16_t;          \
            __VA_ARGS__;                      \
        } else {                              \
            using LogitT = pcg::f16_t;        \
            __VA_ARGS__;                      \
        }                                     \
    } while (0)

#ifdef __CUDACC__

// ---- loading 16 bytes of logits and widening them to float -------------------------------------------------
template <typename T>
struct Elem;
template <>
struct Elem<float> {
    static constexpr int kPerVec = 4;
    static __device__ __forceinline__ float widen(float x) { return x; }
    static __device__ __forceinline__ void unpack(const uint4 &r, float (&v)[4]) {
        v[0] = __uint_as_float(r.x);
        v[1] = __uint_as_float(r.y);
        v[2] = __uint_as_float(r.z);
        v[3] = __uint_as_float(r.w);
    }
};
template <>
struct Elem<uint16_t> {  // bfloat16 bit patterns: the upper half of a float
    static constexpr int kPerVec = 8;
    static __device__ __forceinline__ float widen(uint16_t x) { return __uint_as_float(((uint32_t)x) << 16); }
    static __device__ __forceinline__ void unpack(const uint4 &r, float (&v)[8]) {
        v[0] = __uint_as_float(r.x << 16);
        v[1] = __uint_as_float(r.x & 0xffff0000u);
        v[2] = __uint_as_float(r.y << 16);
        v[3] = __uint_as_float(r.y & 0xffff0000u);
        v[4] = __uint_as_float(r.z << 16);
        v[5] = __uint_as_float(r.z & 0xffff0000u);
        v[6] = __uint_as_float(r.w << 16);
        v[7] = __uint_as_float(r.w & 0xffff0000u);
    }
};

struct f16_t {  // IEEE binary16 bit pattern (a tag type: bfloat16 patterns travel as plain uint16_t)
    uint16_t bits;
};
template <>
struct Elem<f16_t> {
    static constexpr int kPerVec = 8;
    static __device__ __forceinline__ float widen(f16_t x) { return __half2float(__ushort_as_half(x.bits)); }
    static __device__ __forceinline__ void unpack(const uint4 &r, float (&v)[8]) {
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w[i]));
            v[2 * i] = f.x;
            v[2 * i + 1] = f.y;
        }
    }
};

// Streaming 128-bit load that does not allocate in L1 (each logit is read once per kernel).
// Programmatic dependent launch.  A kernel launched with cudaLaunchAttributeProgrammaticStreamSerialization may
// be scheduled while the kernel before it on the stream is still draining: pdl_enter() first lets the NEXT kernel
// do the same with respect to this one, then waits until the previous grid has completed and its writes are
// visible.  Nothing a previous kernel wrote may be read before it.  Without the launch attribute both are no-ops.
__device__ __forceinline__ void pdl_enter() {
    asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

__device__ __forceinline__ uint4 ld_stream(const uint4 *p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

// The same with an L2 eviction policy (see l2_evict_first_policy): logits are read once, so their lines should be
// the first to leave the L2 -- not the operands later kernels of the call keep there.
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t pol;
    asm("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ uint4 ld_stream(const uint4 *p, uint64_t pol) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p), "l"(pol));
    return r;
}

__device__ __forceinline__ float ex2(float x) {  // 2^x, MUFU, flushes subnormal results to zero
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int NT>
__device__ __forceinline__ float block_sum(float v, float *scratch) {
    constexpr int NW = NT / 32;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = scratch[0];
#pragma unroll
    for (int w = 1; w < NW; ++w) r += scratch[w];
    return r;
}

template <int NT>
__device__ __forceinline__ float block_max(float v, float *scratch) {
    constexpr int NW = NT / 32;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = scratch[0];
#pragma unroll
    for (int w = 1; w < NW; ++w) r = fmaxf(r, scratch[w]);
    return r;
}

// Prefix sums (in double) of one value per thread, in thread order.  *incl is this thread's inclusive
// prefix and *excl is exactly the previous thread's inclusive prefix (0 for thread 0), so the intervals
// [excl, incl) of consecutive threads tile [0, total) without cracks.  `scratch` holds NWARPS doubles.
template <int NT>
__device__ __forceinline__ void block_scan(double v, double *scratch, double *excl, double *incl, double *total) {
    constexpr int NW = NT / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    double inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        double up = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += up;
    }
    double prev = __shfl_up_sync(0xffffffffu, inc, 1);
    if (lane == 0) prev = 0.0;
    __syncthreads();
    if (lane == 31) scratch[warp] = inc;
    __syncthreads();
    double base = 0.0, tot = 0.0;
#pragma unroll
    for (int w = 0; w < NW; ++w) {
        if (w == warp) base = tot;
        tot += scratch[w];
    }
    *total = tot;
    *excl = base + prev;
    *incl = base + inc;
}

#endif  // __CUDACC__

}  // namespace pcg
