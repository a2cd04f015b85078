// pcg_verify_host: the same verification for callers whose tensors live in host memory.
#include <cmath>

#include "pcg_common.cuh"

namespace {

struct Arena {
    size_t target, draft, tokens, uniforms, accept_len, out_tokens, out_groups, out_flags, workspace, total;
    size_t target_bytes, draft_bytes, tokens_bytes, uniforms_bytes, len_bytes, outtok_bytes, ws_bytes;
};

Arena layout(int32_t B, int32_t K, int32_t V, int32_t M, pcg_dtype dtype, uint32_t mode) {
    Arena a{};
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t at = off;
        off = (off + bytes + 255) & ~(size_t)255;
        return at;
    };
    const size_t esz = pcg::dtype_bytes(dtype);
    const size_t b = B > 0 ? B : 0, k = K > 0 ? K : 0, v = V > 0 ? V : 0;
    a.target_bytes = b * (k + 1) * v * esz;
    a.draft_bytes = b * k * v * esz;
    a.tokens_bytes = b * k * 4;
    a.uniforms_bytes = b * (k + 1) * 2 * 4;
    a.len_bytes = b * 4;
    a.outtok_bytes = b * (k + 1) * 4;
    a.ws_bytes = pcg_verify_workspace_bytes(B, K, V, M, dtype, mode);
    a.target = take(a.target_bytes);
    a.draft = take(a.draft_bytes);
    a.tokens = take(a.tokens_bytes);
    a.uniforms = take(a.uniforms_bytes);
    a.accept_len = take(a.len_bytes);
    a.out_tokens = take(a.outtok_bytes);
    a.out_groups = take(a.outtok_bytes);
    a.out_flags = take(a.len_bytes);
    a.workspace = take(a.ws_bytes);
    a.total = off;
    return a;
}

}  // namespace

extern "C" size_t pcg_verify_host_arena_bytes(int32_t B, int32_t K, int32_t V, int32_t M, pcg_dtype dtype,
                                              uint32_t mode) {
    return layout(B, K, V, M, dtype, mode).total;
}

extern "C" pcg_status pcg_verify_host(const void *target_logits, const void *draft_logits, pcg_dtype dtype, int32_t B,
                                      int32_t K, const int32_t *draft_tokens, const pcg_groups *groups,
                                      const float *uniforms, float temperature, int32_t *out_accept_len,
                                      int32_t *out_tokens, int32_t *out_groups, int32_t *out_flags,
                                      void *device_arena, size_t device_arena_bytes, uint32_t mode,
                                      pcg_stream stream) {
    using namespace pcg;
    if (!groups) {
        set_error("pcg_verify_host: null group handle");
        return PCG_ERR_INVALID_ARG;
    }
    if (!valid_dtype(dtype)) {
        set_error("pcg_verify_host: dtype must be PCG_F32, PCG_BF16 or PCG_F16");
        return PCG_ERR_INVALID_ARG;
    }
    if (B < 0 || K < 1) {
        set_error("pcg_verify_host: need B >= 0 and K >= 1 (B=%d K=%d)", B, K);
        return PCG_ERR_INVALID_ARG;
    }
    if (K > 1024) {
        set_error("pcg_verify_host: K=%d exceeds the supported 1024 drafted positions per sequence", K);
        return PCG_ERR_UNSUPPORTED;
    }
    if (mode != PCG_VERIFY_DEFAULT && mode != PCG_VERIFY_DENSE && mode != PCG_VERIFY_CLUSTER_TERMINAL &&
        mode != PCG_VERIFY_BATCHED_TERMINAL) {
        set_error("pcg_verify_host: unknown or contradictory mode bits 0x%x", mode);
        return PCG_ERR_INVALID_ARG;
    }
    if (!(temperature >= 1e-6f) || !std::isfinite(temperature)) {
        set_error("pcg_verify_host: temperature must be finite and at least 1e-6");
        return PCG_ERR_INVALID_ARG;
    }
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev != groups->device) {
        set_error("pcg_verify_host: the handle lives on device %d but device %d is current", groups->device, dev);
        return PCG_ERR_INVALID_ARG;
    }
    if (mode == PCG_VERIFY_CLUSTER_TERMINAL && !groups->has_sweep) {
        set_error("pcg_verify_host: this handle has no sweep layout, so the cluster terminal is unavailable");
        return PCG_ERR_UNSUPPORTED;
    }
    if (B == 0) return PCG_OK;
    if (!target_logits || !draft_logits || !draft_tokens || !uniforms || !out_accept_len || !out_tokens) {
        set_error("pcg_verify_host: null pointer");
        return PCG_ERR_INVALID_ARG;
    }
    // everything the host can refuse has been refused above: no copy is enqueued for a call that cannot run
    const Arena a = layout(B, K, groups->dev.V, groups->dev.M, dtype, mode);
    if (!device_arena || ((uintptr_t)device_arena & 255u) || device_arena_bytes < a.total) {
        set_error("pcg_verify_host: device arena must be 256-byte aligned and hold %zu bytes (got %zu)", a.total,
                  device_arena_bytes);
        return PCG_ERR_WORKSPACE;
    }
    char *d = (char *)device_arena;
    cudaStream_t cs = (cudaStream_t)stream;
    // From the first enqueued copy on, no return before the stream has drained: the caller may free or overwrite
    // its buffers as soon as this call is back, also after an error.
    auto fail_after_enqueue = [&](pcg_status st) {
        (void)cudaStreamSynchronize(cs);
        return st;
    };
    e = cudaMemcpyAsync(d + a.target, target_logits, a.target_bytes, cudaMemcpyHostToDevice, cs);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d + a.draft, draft_logits, a.draft_bytes, cudaMemcpyHostToDevice, cs);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d + a.tokens, draft_tokens, a.tokens_bytes, cudaMemcpyHostToDevice, cs);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d + a.uniforms, uniforms, a.uniforms_bytes, cudaMemcpyHostToDevice, cs);
    if (e != cudaSuccess) return fail_after_enqueue(cuda_fail(e, "copying inputs to the device"));
    pcg_status st = pcg_verify(d + a.target, d + a.draft, dtype, B, K, (const int32_t *)(d + a.tokens), groups,
                               (const float *)(d + a.uniforms), temperature, (int32_t *)(d + a.accept_len),
                               (int32_t *)(d + a.out_tokens), (int32_t *)(d + a.out_groups),
                               (int32_t *)(d + a.out_flags), d + a.workspace, a.ws_bytes, mode, stream, nullptr);
    if (st != PCG_OK) return fail_after_enqueue(st);
    e = cudaMemcpyAsync(out_accept_len, d + a.accept_len, a.len_bytes, cudaMemcpyDeviceToHost, cs);
    if (e == cudaSuccess) e = cudaMemcpyAsync(out_tokens, d + a.out_tokens, a.outtok_bytes, cudaMemcpyDeviceToHost, cs);
    if (e == cudaSuccess && out_groups)
        e = cudaMemcpyAsync(out_groups, d + a.out_groups, a.outtok_bytes, cudaMemcpyDeviceToHost, cs);
    if (e == cudaSuccess && out_flags)
        e = cudaMemcpyAsync(out_flags, d + a.out_flags, a.len_bytes, cudaMemcpyDeviceToHost, cs);
    if (e != cudaSuccess) return fail_after_enqueue(cuda_fail(e, "copying outputs to the host"));
    e = cudaStreamSynchronize(cs);
    if (e != cudaSuccess) return cuda_fail(e, "waiting for the verification to finish");
    return PCG_OK;
}
