/*
 * pcg.h -- C interface of libpcg: batched group-level verification for
 * speculative decoding with Principled Coarse-Graining (PCG) on NVIDIA B200.
 *
 * Letters used throughout (NOTE: the paper's body uses the opposite letters):
 *   p = TARGET token distribution, q = DRAFT token distribution,
 *   P[g] / Q[g] = target / draft coarse-grained mass of group g.
 *
 * Unless a parameter says HOST, every pointer is DEVICE memory of the device
 * that was current when the group handle was created; that device must also be
 * current when a call is made.  All tensors are dense, row-major, contiguous.
 * Inputs are never written.  No call allocates or frees device memory except
 * pcg_groups_create / pcg_groups_destroy.  Calls that take a stream only
 * enqueue work on it and return without synchronising, except where stated.
 *
 * Every function returns a pcg_status; errors the host can see (null pointers,
 * bad sizes, a handle of another device, too small a workspace) are returned
 * before anything is launched.  Nothing prints, aborts or throws.
 */
#ifndef PCG_H
#define PCG_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PCG_OK = 0,
    PCG_ERR_INVALID_ARG = 1,    /* null pointer, non-positive size, misaligned base, wrong device */
    PCG_ERR_INVALID_GROUPS = 2, /* the membership CSR breaks one of its rules (see pcg_csr) */
    PCG_ERR_UNSUPPORTED = 3,    /* sizes beyond what the kernels are built for (see pcg_groups_create) */
    PCG_ERR_WORKSPACE = 4,      /* workspace missing, misaligned or smaller than the query says */
    PCG_ERR_CUDA = 5            /* a CUDA runtime call failed; pcg_last_error() has the text */
} pcg_status;

typedef enum {
    PCG_F32 = 0,  /* IEEE float32 logits */
    PCG_BF16 = 1, /* bfloat16 logits (upper 16 bits of a float32) */
    PCG_F16 = 2   /* IEEE binary16 logits */
} pcg_dtype;

/* CUDA stream handle (a cudaStream_t / CUstream); NULL is the default stream. */
typedef struct CUstream_st *pcg_stream;
/* CUDA event handle (a cudaEvent_t / CUevent). */
typedef struct CUevent_st *pcg_event;

/* Bits of out_flags[b] written by pcg_verify. */
#define PCG_FLAG_BAD_DRAFT_TOKEN 1 /* a draft token id outside [0,V) was seen and treated as token 0 */
#define PCG_FLAG_ZERO_RESIDUAL 2   /* a rejection whose residual mass summed to <= 0; drew from P instead */
#define PCG_FLAG_NONFINITE 4       /* a row's maximum or normaliser was not finite (NaN/+inf logits, or all -inf) */
#define PCG_FLAG_THINNING_EXHAUSTED 8 /* pcg_verify_thinning: every supplied trial was turned down; the group was
                                         drawn from the enumerated residual instead (same law) */

/* Bits of the `mode` argument of pcg_verify. */
#define PCG_VERIFY_DEFAULT 0u /* per position only the label group's P and Q are formed (what the accept test
                                 needs); all groups are aggregated once per sequence, at its terminal position.
                                 The per-sequence stage runs as CLUSTER_TERMINAL for a handful of sequences
                                 (B * slices <= 2 * SM count) and as BATCHED_TERMINAL beyond that */
#define PCG_VERIFY_DENSE 1u   /* form P and Q of ALL groups at EVERY position (stored in the workspace), then take
                                 the same decisions from the stored vectors */
#define PCG_VERIFY_CLUSTER_TERMINAL 2u /* default per-position stage; per-sequence stage as one thread-block
                                 cluster per sequence (shared-memory aggregation; lowest latency for small batches) */
#define PCG_VERIFY_BATCHED_TERMINAL 4u /* default per-position stage; per-sequence stage as the batched kernels
                                 (transposed residual, sparse product over L2, draw; best throughput for large
                                 batches) */
/* The modes are alternatives, not flags to combine; all four take the same decisions. */

/*
 * Group membership: the Acoustic Similarity Groups as a group->token CSR plus
 * every token's degree N(t) = number of groups containing it (Sec. 2.2, "let
 * S(t) := {k : t in G_k} and N(t) := |S(t)|").
 *
 * Rules (checked by pcg_groups_create, PCG_ERR_INVALID_GROUPS otherwise):
 *   group_ptr[0] == 0, non-decreasing, group_ptr[M] == nnz;
 *   token ids in [0,V), strictly ascending inside a group (no duplicates);
 *   tok_degree[t] equals the number of groups listing t, and is >= 1 for every
 *   token (a token in no group would leak probability mass);
 *   weights, if not NULL: finite, >= 0, and summing to 1 (+-1e-4) over the
 *   groups of each token (the weight equation of Sec. 2.2).
 * Empty groups and duplicate groups are allowed.
 * The three/four arrays may live in HOST or DEVICE memory (they are copied with
 * cudaMemcpyDefault) and may be freed as soon as pcg_groups_create returns.
 */
typedef struct {
    int32_t V;                 /* vocabulary size */
    int32_t M;                 /* number of groups */
    int64_t nnz;               /* number of stored (group, token) pairs */
    const int32_t *group_ptr;  /* [M+1] */
    const int32_t *group_tok;  /* [nnz] */
    const int32_t *tok_degree; /* [V] */
    const float *weights;      /* [nnz] split weights w_{k,t}, or NULL for the paper's default equal split 1/N(t) */
} pcg_csr;

/* Opaque handle: device-resident membership in the layouts the kernels want. */
typedef struct pcg_groups pcg_groups;

typedef struct {
    int32_t V, M;
    int64_t nnz;
    int32_t slices;          /* token slices per row = thread-block cluster size of the aggregation kernels */
    int32_t slice_len;       /* tokens per slice */
    int32_t max_group_size;  /* largest |G_g| */
    int32_t max_degree;      /* largest N(t) */
    int32_t device;          /* CUDA device ordinal the handle lives on */
    int32_t has_weights;     /* 1 if general weights were given */
    int64_t device_bytes;    /* device memory held by the handle */
} pcg_groups_info_t;

const char *pcg_status_string(pcg_status s);

/* Text of the last error raised on the calling thread ("" if none). The pointer stays valid until the next call. */
const char *pcg_last_error(void);

/*
 * Build the handle (the groups are "precomputed once and cached", Sec. 2.2
 * "Complexity and memory").  One-time set-up, not part of the hot path:
 * validates the CSR on the host, builds the reverse membership S(t) (ascending
 * group id -- the "optional reverse indices" of the same paragraph), the 1/N(t)
 * table and a token-sliced copy of the CSR with 16-bit in-slice token offsets,
 * uploads them and synchronises the device.  The handle also holds the scratch of pcg_group_probs
 * (4 * (V + M) * min(256, ...) bytes: 80 MB at V = 65536, M = 16384; pcg_group_probs_ws does not use it).
 *
 *   slices_hint: 0 = choose automatically; 1, 2, 4 or 8 = force that many token
 *                slices (= cluster size).  Rounded up if a slice would not fit
 *                in shared memory.
 * The token-sliced copy needs M <= 65534 (16-bit group ids) and, per thread block, slice_len*4 + M*4 +
 * (M/slices)*4 bytes plus 2 KB within 227 KB of shared memory with slices <= 8.  Where that is impossible the
 * handle is built WITHOUT it (pcg_groups_info reports slices = 0): everything runs on the batched kernels,
 * PCG_VERIFY_CLUSTER_TERMINAL and pcg_verify_static then return PCG_ERR_UNSUPPORTED, and a slices_hint other than 0
 * is refused.
 * Errors: INVALID_ARG (null, V/M < 1), INVALID_GROUPS, UNSUPPORTED, CUDA.
 */
pcg_status pcg_groups_create(const pcg_csr *csr, int slices_hint, pcg_groups **out);

/* Free the handle and its device memory. NULL is allowed. The caller must have synchronised all work using it. */
void pcg_groups_destroy(pcg_groups *groups);

pcg_status pcg_groups_info(const pcg_groups *groups, pcg_groups_info_t *out);

/*
 * Constant added to the acceptance ratio of every later pcg_verify call with this handle: accept iff
 * u < min(1, P/Q) + bias.  0 (the default) is PCG; a positive value gives the lossy relaxation the paper compares
 * against (Sec. 3.2: speculative decoding with a constant bias of 0.3 on the acceptance probability).  The
 * residual and the token draws are unchanged.  Errors: INVALID_ARG (null, bias < 0 or not finite).
 */
pcg_status pcg_groups_set_accept_bias(pcg_groups *groups, float bias);

/*
 * Coarse-grained group distribution of every row (the coarse-grained
 * distribution equations of Sec. 2.2):
 *     out[r, g] = sum_{t in G_g} softmax(logits[r, :] / temperature)[t] * w_{g,t},
 * w_{g,t} = 1/N(t) unless the handle carries weights.  Each row of out sums to
 * 1 up to rounding; no renormalisation is applied.
 *
 *   logits  [rows, V] of `dtype`; base 16-byte aligned for the vector path
 *           (other alignments, or V*elemsize not a multiple of 16, use a slower scalar path)
 *   out     [rows, M] float32, fully overwritten
 * From 64 rows on the rows go, up to 256 at a time, through scratch memory (a transposed copy of the rows'
 * probabilities).  pcg_group_probs uses scratch that belongs to the handle: two such calls with the SAME handle
 * must not overlap on the device (different streams).  pcg_group_probs_ws is the same call with the scratch
 * supplied by the caller (pcg_group_probs_workspace_bytes(V, M) bytes, 256-byte aligned, contents irrelevant): calls
 * with separate workspaces may overlap freely, the handle is only read.
 * rows == 0 is a no-op.  Errors: INVALID_ARG (null, rows < 0, temperature <= 0 or not finite, bad dtype,
 * wrong device), WORKSPACE (pcg_group_probs_ws: workspace missing, misaligned or too small), CUDA (launch failure).
 */
pcg_status pcg_group_probs(const void *logits, pcg_dtype dtype, int64_t rows, float temperature,
                           const pcg_groups *groups, float *out, pcg_stream stream);
size_t pcg_group_probs_workspace_bytes(int32_t V, int32_t M);
pcg_status pcg_group_probs_ws(const void *logits, pcg_dtype dtype, int64_t rows, float temperature,
                              const pcg_groups *groups, float *out, void *workspace, size_t workspace_bytes,
                              pcg_stream stream);

/* Bytes of workspace pcg_verify needs for these sizes and mode (256-byte aligned base required). Never 0. */
size_t pcg_verify_workspace_bytes(int32_t B, int32_t K, int32_t V, int32_t M, pcg_dtype dtype, uint32_t mode);

/*
 * Batched PCG verification: Algorithm 1 from the label draw to the returned
 * token list, for B sequences of K drafted positions, with all randomness
 * supplied by the caller.
 *
 * For sequence b and drafted position i < K (x = draft_tokens[b,i]):
 *   label   g = the j-th smallest group id containing x, j = min(floor(u[b,i,0] * N(x)), N(x)-1)
 *           (with weights: inverse CDF of w_{.,x} over S(x) in ascending group id)   -- group-label coupling
 *   accept  iff P[g] >= Q[g] or u[b,i,1] * Q[g] < P[g]                               -- min(1, P/Q) acceptance
 * n_b = first rejected position (K if none).  Terminal draw at position n_b:
 *   R[g] = max(0, P[g] - Q[g]) if n_b < K (residual), R[g] = P[g] of target row K otherwise (bonus token);
 *   g* = first g whose inclusive prefix of R exceeds u[b,K,0] * sum(R) (last g with R > 0 if rounding leaves none);
 *   z  = first token t of G_g* (CSR order) whose inclusive prefix of p(t) w_{g*,t} exceeds u[b,K,1] * its sum.
 * Emitted: out_tokens[b, i<n_b] = draft token (kept on acceptance), out_tokens[b, n_b] = z, later slots -1;
 *          out_accept_len[b] = n_b; out_groups likewise (labels, then g*, then -1).
 *
 *   target_logits [B, K+1, V], draft_logits [B, K, V] of `dtype`, same alignment rule as pcg_group_probs
 *   draft_tokens  [B, K] int32          uniforms [B, K+1, 2] float32 in [0,1)
 *   out_accept_len [B] int32            out_tokens [B, K+1] int32
 *   out_groups [B, K+1] int32 or NULL   out_flags [B] int32 or NULL (PCG_FLAG_* bits)
 *   workspace: >= pcg_verify_workspace_bytes(...) bytes, 256-byte aligned, contents irrelevant on entry;
 *              calls that share a workspace must not overlap on the device
 *   stage_events: NULL, or 3 events recorded on `stream` before the position kernel, between it and the
 *              terminal kernel, and after the terminal kernel (for timing the stages)
 * Results are bit-identical from run to run.  1 <= K <= 1024, B >= 0 (B == 0 is a no-op).
 * Masses below the float32 normal range flush to zero.
 * Errors: INVALID_ARG, UNSUPPORTED (K > 1024), WORKSPACE, CUDA.
 */
pcg_status pcg_verify(const void *target_logits, const void *draft_logits, pcg_dtype dtype, int32_t B, int32_t K,
                      const int32_t *draft_tokens, const pcg_groups *groups, const float *uniforms, float temperature,
                      int32_t *out_accept_len, int32_t *out_tokens, int32_t *out_groups, int32_t *out_flags,
                      void *workspace, size_t workspace_bytes, uint32_t mode, pcg_stream stream,
                      const pcg_event *stage_events);

/* Bytes of device staging memory pcg_verify_host needs (inputs, outputs and the verify workspace). */
size_t pcg_verify_host_arena_bytes(int32_t B, int32_t K, int32_t V, int32_t M, pcg_dtype dtype, uint32_t mode);

/*
 * pcg_verify for callers whose tensors live in HOST memory (pinned memory makes
 * the copies asynchronous and fast; pageable memory works but is slower).
 * Copies the inputs into `device_arena`, runs pcg_verify there, copies the
 * outputs back and SYNCHRONISES `stream` before returning.
 *   target_logits, draft_logits, draft_tokens, uniforms, out_*: HOST pointers, shapes as in pcg_verify
 *   device_arena: DEVICE memory, >= pcg_verify_host_arena_bytes(...), 256-byte aligned, caller-owned
 * Errors: as pcg_verify.
 */
pcg_status pcg_verify_host(const void *target_logits, const void *draft_logits, pcg_dtype dtype, int32_t B, int32_t K,
                           const int32_t *draft_tokens, const pcg_groups *groups, const float *uniforms,
                           float temperature, int32_t *out_accept_len, int32_t *out_tokens, int32_t *out_groups,
                           int32_t *out_flags, void *device_arena, size_t device_arena_bytes, uint32_t mode,
                           pcg_stream stream);

/*
 * Group construction on the GPU (the group-construction equation of Sec. 2.1): the neighbourhood of token t is
 *     G(t) = { t' : cos(Emb(t), Emb(t')) > theta },
 * and the DISTINCT neighbourhoods form the groups.  One-time set-up ("precomputed once and cached", Sec. 2.2
 * "Complexity and memory"), not part of the verification hot path.
 *
 *   emb    [V, d] DEVICE memory, row-major, PCG_BF16 or PCG_F32 (a float32 table is rounded to bfloat16,
 *          nearest even, first: the similarity is defined on bfloat16 values, with products and sums in float32
 *          and cos = dot * (1/|a|) * (1/|b|))
 *   theta  threshold (strict >).  t is always a member of G(t); a zero embedding is similar to nothing else.
 *   flags  0: the similarity tiles run on the 5th-generation tensor cores (tcgen05.mma, accumulators in tensor
 *          memory); PCG_ASG_MMA_SYNC: the same tiles with warp-level mma.sync (kept as a cross-check)
 * Groups are numbered by the smallest token whose neighbourhood equals the set; tokens inside a group ascend;
 * tok_degree counts the distinct groups containing a token.
 * The call allocates device memory (V*V/8 bytes of scratch, freed before it returns, plus the result),
 * synchronises the device, and returns an object that owns the result until pcg_asg_destroy.
 * pcg_asg_csr fills a pcg_csr whose arrays are DEVICE pointers owned by the object (valid until destroy); it can
 * be handed to pcg_groups_create as is.
 * Errors: INVALID_ARG (null, V < 1, d < 1, bad dtype, theta not finite, unknown flags), UNSUPPORTED (V > 2^20),
 * CUDA (also when the tensor-core kernel gave up a bounded wait; pcg_last_error says so).
 */
typedef struct pcg_asg pcg_asg;
typedef struct {
    int32_t V, M;
    int64_t nnz;
    int32_t max_group_size;
    int32_t max_degree;
    float similarity_ms; /* device time of the similarity (tensor-core) kernel */
    float total_ms;      /* device time of the whole construction */
    int32_t tensor_path; /* 1 = tcgen05, 0 = mma.sync */
} pcg_asg_info_t;
#define PCG_ASG_MMA_SYNC 1u
pcg_status pcg_asg_create(const void *emb, pcg_dtype dtype, int32_t V, int32_t d, float theta, uint32_t flags,
                          pcg_asg **out);
pcg_status pcg_asg_info(const pcg_asg *asg, pcg_asg_info_t *out);
pcg_status pcg_asg_csr(const pcg_asg *asg, pcg_csr *out);
void pcg_asg_destroy(pcg_asg *asg);

/*
 * pcg_verify for callers that have no workspace to give.  (The paper has no counterpart to this entry point;
 * it exists for the library's users only.)
 *
 * Who needs it: code that runs after its host application has handed out all device memory and forbids
 * further allocation -- an inference server whose memory pool was carved up at start-up, a plug-in running
 * inside someone else's process, a latency-critical loop that must never meet cudaMalloc (which may stall the
 * whole device, or fail once the pool owns all memory).  Such a caller cannot size and allocate the workspace
 * pcg_verify asks for, so this variant keeps its scratch in an array that is part of the library image: 1 MiB
 * of device memory on every GPU that loads libpcg.so, held until the process exits.  The call allocates and
 * frees nothing, on the host side of CUDA or through any library.
 *
 * Same arguments, results and errors as pcg_verify in PCG_VERIFY_CLUSTER_TERMINAL mode, without workspace,
 * mode and stage events.  Limits: the per-position bookkeeping of the call must fit the array -- 28 bytes per
 * drafted position plus 24 per sequence (each array rounded up to 256 bytes), i.e. roughly B*K <= 35,000; larger calls return
 * PCG_ERR_UNSUPPORTED with a message that says so, before anything is launched.
 *
 * The first call on each device looks up the array's device address (with that device current) and remembers
 * it; make that first call outside any stream capture.  All calls on one device share the one array, which
 * keeps whatever the previous call left in it (nothing in it needs clearing: every field is written before it
 * is read within a call).  Two calls whose kernels can overlap on the same GPU -- different streams, or different
 * host threads -- race on it: serialise them, or use pcg_verify with separate workspaces.
 */
pcg_status pcg_verify_static(const void *target_logits, const void *draft_logits, pcg_dtype dtype, int32_t B, int32_t K,
                             const int32_t *draft_tokens, const pcg_groups *groups, const float *uniforms,
                             float temperature, int32_t *out_accept_len, int32_t *out_tokens, int32_t *out_groups,
                             int32_t *out_flags, pcg_stream stream);

/*
 * pcg_verify with the paper's own sampler for the terminal group: the thinning sampler of Sec. 2.2.
 *
 * Everything up to the first rejection is pcg_verify's per-position stage (label, acceptance, first-reject scan).
 * The group at the rejected position is then drawn WITHOUT enumerating the groups.  Trial r = 0, 1, ... draws a
 * token y from the target row by inverse CDF with thin_uniforms[b, r, 0] (the paper fixes the law y ~ target; how a
 * uniform is mapped to y is this interface's rule:
 *     CANDIDATE ORDER: the inverse CDF walks the tokens in ascending order of the pair ((t div W) mod 128, t),
 *     where W = 16 / (bytes per logit), i.e. 4 for PCG_F32 and 8 for the 16-bit types;
 * y is the first token of that order whose inclusive running sum of p exceeds u times the total), a label
 * k ~ w_{.,y} over
 * the groups containing y with thin_uniforms[b, r, 1] (so k follows the target's coarse distribution), and keeps
 * k if thin_uniforms[b, r, 2] < [1 - Q(k)/P(k)]_+ (draft mass over target mass of group k alone); otherwise the
 * next trial draws a new candidate.  The kept group's law is the normalised residual (P - Q)_+ exactly; the
 * expected number of trials is 1 / TV(P, Q).  After a sequence whose K positions were all accepted there is no
 * draft mass: the first candidate is kept (the bonus group, from the target's coarse distribution).  The token
 * inside the kept group is drawn from the target-conditional p(t) w / P(k) with uniforms[b, K, 1], as in
 * pcg_verify.  The paper's loop is unbounded; this call runs at most n_trials trials per sequence and, if all
 * are turned down, draws the group from the enumerated residual with uniforms[b, K, 0] (what pcg_verify does;
 * same law) and sets PCG_FLAG_THINNING_EXHAUSTED for that sequence.  That fallback costs more than a trial, and how
 * much depends on n_trials.  From 24 supplied trials on (running out is then rare) it is done by the sequence's own
 * thread block, which walks all nnz memberships alone: 0.47 ms for one such sequence at V = 65536, M = 16384,
 * nnz = 393216 on a B200, more than the rest of a 256-sequence call.  With fewer trials the call launches one more
 * kernel (about 3 microseconds when it finds nothing to do) in which ALL thread blocks share the enumeration of the
 * sequences that ran out: about 15 microseconds for one, about 10 for each further one.  Trials themselves are cheap:
 * they run side by side (8 in the first round, 16 in each later one), and a further round (about 4 microseconds) is
 * entered only by sequences whose earlier candidates were all turned down.  So supply trials
 * generously: a rejected sequence runs out of n_trials with probability (1 - TV(P,Q))^n_trials.  Results are a deterministic function of
 * the inputs; they equal pcg_verify's in distribution, not draw by draw (the two consume different uniforms).
 *
 *   thin_uniforms [B, n_trials, 3] float in [0,1), device, read-only; 1 <= n_trials <= 65536
 *   out_trials    [B] int32 or NULL: candidates drawn (1 after an all-accepted sequence; n_trials when exhausted)
 *   workspace     device, 256-byte aligned, at least pcg_verify_thinning_workspace_bytes(...) bytes (2076 bytes per
 *                 drafted position plus 2*B*M*4 for sequences whose trials run out); contents need no initialisation
 *   the remaining arguments, ownership, asynchrony (no allocation, no synchronisation, the caller's stream only)
 *   and errors are pcg_verify's.  Rows that do not start on 16-byte boundaries or are not whole 16-byte words
 *   long (V * bytes per logit not a multiple of 16) give the same results, a little slower (their slot masses
 *   are summed by the thinning kernel itself).
 */
size_t pcg_verify_thinning_workspace_bytes(int32_t B, int32_t K, int32_t V, int32_t M, pcg_dtype dtype);
pcg_status pcg_verify_thinning(const void *target_logits, const void *draft_logits, pcg_dtype dtype, int32_t B, int32_t K,
                               const int32_t *draft_tokens, const pcg_groups *groups, const float *uniforms,
                               const float *thin_uniforms, int32_t n_trials, float temperature,
                               int32_t *out_accept_len, int32_t *out_tokens, int32_t *out_groups, int32_t *out_flags,
                               int32_t *out_trials, void *workspace, size_t workspace_bytes, pcg_stream stream,
                               const pcg_event *stage_events);

#ifdef __cplusplus
}
#endif
#endif /* PCG_H */
