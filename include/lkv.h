/*
 * lkv.h -- C ABI of the recurrent-layer half of hybrid position-independent
 * caching ("LinearKV"), hand-written for NVIDIA B200 (sm_100a).
 *
 * A hybrid LLM keeps, per recurrent layer and head, a fixed-size state
 * S in R^{d_k x d_v} that follows the affine recurrence S_i = T_i S_{i-1} + u_i
 * (Eq. 1).  Serving a request from K independently cached chunks needs two
 * things from each recurrent layer, and this library provides exactly those:
 *
 *   1. lkv_init_state*      S_init = f(S_1 .. S_K)                   (Eq. 4)
 *        f = one cached state (Section 3.2, "Single-block initialization";
 *            any block index per Appendix A), or
 *        f = exact composition sum_j (prod_{m>j} T_{C_m}) S_j        (Eq. 6)
 *            with scalar transitions for Mamba-2 and dense d_k x d_k
 *            transitions for Gated DeltaNet (Eq. 5, Eq. 2, Eq. 3);
 *   2. lkv_gdn_fwd / lkv_ssd_fwd   advance the recurrence from S_init through
 *        a run of tokens in context order, returning the per-token outputs
 *        and the final state (Algorithm 1, line 3; Eq. 1-3), computed in the
 *        chunkwise-parallel form.
 *
 * General rules
 *   - Every data pointer is a DEVICE pointer unless its comment says HOST.
 *     Small index arrays (chunk ids, cu_k, sel_index, cu_seqlens) are HOST
 *     int32 arrays: they are range-checked on the host before anything is
 *     launched and copied to the device by the call itself (into the
 *     caller's workspace).  They may be reused as soon as the call returns.
 *     A list that fits the kernel parameters (n_req + 1 + selection indices +
 *     chunk ids <= 4000 ints for the initialisers, 2 n_seq + 1 <= 1000 for the
 *     scans, which send the launch order along: longest sequence first) travels inside the launch and the call may be captured into a
 *     CUDA graph; a longer list needs a host-to-device copy of an array that
 *     dies with the call, so such a call returns LKV_ERR_UNSUPPORTED while
 *     `stream` is capturing.
 *   - The caller owns every buffer.  The library allocates nothing, frees
 *     nothing and keeps no pointer after a call returns; scratch lives in a
 *     caller-provided workspace whose size lkv_workspace_bytes() reports.
 *     A workspace must not be shared by calls that can overlap on the GPU.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*,
 *     NULL = the legacy default stream).  They do not synchronise.
 *   - Return value: 0 (LKV_OK) or a negative LKV_ERR_* code.  All argument
 *     errors are found on the host before any launch; nothing is written in
 *     that case.  There is no CPU fallback: an unsupported shape returns
 *     LKV_ERR_UNSUPPORTED.
 *   - Device-side waits (TMA / tensor-core completion barriers) are bounded.
 *     A kernel whose wait runs out sets the status word (the first 4 bytes of
 *     the workspace), drains without writing any further result, and returns;
 *     lkv_device_status() reads the word.  The word is sticky: the library
 *     only ever sets it.  The caller zeroes the first 256 bytes of a
 *     workspace once before its first use, and again after a reported
 *     time-out; results of a call whose workspace reports a time-out are
 *     undefined (partly written).
 *   - Data pointers must be 16-byte aligned (LKV_ERR_ALIGN otherwise).
 *   - Outputs must not overlap inputs or each other (LKV_ERR_OVERLAP, checked
 *     on the host from the sizes the descriptor implies), except that S_T
 *     may be exactly S0 in the scan calls.
 *   - States are row-major [.., d_k, d_v] with d_v contiguous, always fp32 on
 *     output.  All results are deterministic: the same inputs give the same
 *     bits on every run.
 */
#ifndef LKV_H_
#define LKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LKV_VERSION 100 /* 0.1.0 */

/* status codes */
#define LKV_OK 0
#define LKV_ERR_NULL (-1)           /* a required pointer is NULL */
#define LKV_ERR_DIM (-2)            /* a dimension is negative, zero where it may not be, or inconsistent */
#define LKV_ERR_MODE (-3)           /* unknown mode / family / dtype / compute value */
#define LKV_ERR_INDEX (-4)          /* chunk id, selection index or cu_* entry out of range / not monotone */
#define LKV_ERR_ALIGN (-5)          /* a data pointer is not 16-byte aligned */
#define LKV_ERR_UNSUPPORTED (-6)    /* valid request, but no kernel for this shape / dtype */
#define LKV_ERR_WORKSPACE (-7)      /* workspace missing or too small */
#define LKV_ERR_CUDA (-8)           /* a CUDA runtime call failed (launch, copy, attribute) */
#define LKV_ERR_DEVICE_TIMEOUT (-9) /* a bounded device-side wait ran out (reported by lkv_device_status) */
#define LKV_ERR_OVERLAP (-10)       /* an output buffer overlaps an input buffer or another output */

/* recurrence family (Eq. 2 vs Eq. 3) */
#define LKV_FAMILY_MAMBA2 0
#define LKV_FAMILY_GDN 1

/* element types */
#define LKV_DTYPE_F32 0
#define LKV_DTYPE_BF16 1

/* initialiser f of Eq. 4 */
#define LKV_INIT_LAST 0  /* S_init = S_K, the last matched chunk (the paper's default) */
#define LKV_INIT_INDEX 1 /* S_init = S_b for a caller-chosen position b (Appendix A) */
#define LKV_INIT_EXACT 2 /* S_init = exact composition, Eq. 6 */

/* arithmetic used for the dense contractions */
#define LKV_COMPUTE_AUTO 0   /* tensor cores where a kernel exists for the shape, else fp32.  Note: for GDN exact
                                composition at d_k = d_v = 128 this means tf32 products (operands rounded to nearest,
                                11-bit significands, fp32 accumulation; about 1e-3 relative on the carried part):
                                ask for LKV_COMPUTE_FP32 where fp32 products are wanted */
#define LKV_COMPUTE_FP32 1   /* fp32 FMA on CUDA cores everywhere (tight-tolerance / small shapes) */
#define LKV_COMPUTE_TENSOR 2 /* tensor cores (bf16 operands in the scans, tf32 in GDN composition),
                                fp32 accumulate; LKV_ERR_UNSUPPORTED if no such kernel fits */

/* `which` of lkv_workspace_bytes */
#define LKV_WS_INIT 0
#define LKV_WS_GDN 1
#define LKV_WS_SSD 2

/*
 * Descriptor of lkv_init_state / lkv_init_state_batched.
 *
 * The cached artefacts live in POOLS indexed by chunk id, so that one cached
 * chunk can appear at different positions of different requests:
 *   states       [n_chunks, H, d_k, d_v]   state_dtype (fp32 or bf16)
 *   transitions  MAMBA2: float [n_chunks, H]            log of the chunk's scalar decay,
 *                                                      lambda = A_h * sum_t dt_t
 *                GDN:    float [n_chunks, H, d_k, d_k]  row-major accumulated transition
 *                                                      T_C = T_{t_L} ... T_{t_1} (Eq. 5)
 * For Mamba-2, d_k is d_state (N) and d_v is headdim (P).
 */
typedef struct lkv_init_desc {
    int32_t family;           /* LKV_FAMILY_* */
    int32_t H;                /* heads that own a state (GDN: value heads) */
    int32_t d_k;
    int32_t d_v;
    int32_t n_chunks;         /* pool size */
    int32_t state_dtype;      /* dtype of the `states` pool; S0 is always fp32 */
    int32_t sel_index;        /* lkv_init_state, mode INDEX: position b in [0, K) */
    int32_t compute;          /* LKV_COMPUTE_* (only GDN exact composition looks at it) */
    const int32_t *chunk_ids; /* lkv_init_state: HOST int32[K] pool ids in context order; NULL = 0..K-1 */
    void *workspace;          /* device, >= lkv_workspace_bytes(LKV_WS_INIT, desc, n_req, total_K) */
    size_t workspace_bytes;
} lkv_init_desc;

/*
 * Descriptor of lkv_gdn_fwd.  Token tensors are packed over sequences:
 *   q, k   [T_total, H_k, d_k]   io_dtype        v  [T_total, H_v, d_v]  io_dtype
 *   g      float [T_total, H_v]  log-decay, alpha = exp(g) <= 1 expected
 *   beta   float [T_total, H_v]
 *   S0     float [n_seq, H_v, d_k, d_v]          o  [T_total, H_v, d_v]  io_dtype
 *   S_T    [n_seq, H_v, d_k, d_v] state_dtype (fp32, or bf16 as a cache pool stores states)
 * Value head h reads q/k head h / (H_v / H_k).
 */
typedef struct lkv_gdn_desc {
    int32_t T_total;
    int32_t n_seq;
    const int32_t *cu_seqlens; /* HOST int32[n_seq + 1], cu[0] = 0, cu[n_seq] = T_total; NULL = one sequence */
    int32_t H_k;
    int32_t H_v;               /* multiple of H_k */
    int32_t d_k;
    int32_t d_v;
    int32_t io_dtype;          /* dtype of q, k, v and o */
    int32_t compute;           /* LKV_COMPUTE_* */
    float scale;               /* read-out scale; 0 selects d_k^(-1/2) */
    int32_t state_dtype;       /* dtype of S_T: LKV_DTYPE_F32 (0) or LKV_DTYPE_BF16; S0 is always fp32 */
    void *workspace;
    size_t workspace_bytes;
} lkv_gdn_desc;

/*
 * Descriptor of lkv_ssd_fwd.
 *   x  [T_total, H, P] io_dtype      dt float [T_total, H] (already activated, > 0)
 *   A  float [H] (< 0)               B, C [T_total, G, N] io_dtype
 *   S0 float [n_seq, H, N, P]        y  [T_total, H, P] io_dtype
 *   S_T [n_seq, H, N, P] state_dtype (fp32, or bf16 as a cache pool stores states)
 * Head h reads group h / (H / G).
 */
typedef struct lkv_ssd_desc {
    int32_t T_total;
    int32_t n_seq;
    const int32_t *cu_seqlens; /* HOST, as in lkv_gdn_desc */
    int32_t H;
    int32_t P;                 /* headdim */
    int32_t N;                 /* d_state */
    int32_t G;                 /* groups, divides H */
    int32_t io_dtype;
    int32_t compute;
    int32_t state_dtype;       /* dtype of S_T: LKV_DTYPE_F32 (0) or LKV_DTYPE_BF16; S0 is always fp32 */
    void *workspace;
    size_t workspace_bytes;
} lkv_ssd_desc;

/*
 * State initialisation for ONE request (Eq. 4; Algorithm 1, line 1).
 *
 *   states, transitions  pools as described at lkv_init_desc (device)
 *   K                    number of matched chunks, >= 0; their pool ids are d->chunk_ids
 *   mode                 LKV_INIT_LAST | LKV_INIT_INDEX | LKV_INIT_EXACT
 *   S0                   out, float [H, d_k, d_v] (device)
 *
 * LAST / INDEX copy one stored state (widened exactly if the pool is bf16):
 * with an fp32 pool S0 is bit-identical to the stored state.  `transitions`
 * is not read and may be NULL.
 * EXACT evaluates Eq. 6 as the chain S <- S_{c_1}; S <- T_{c_j} S + S_{c_j}
 * for j = 2..K (Eq. 5 applied in context order); the transition of the first
 * chunk is never read.  K == 1 returns S_{c_1} untouched in every mode;
 * K == 0 returns the zero state.
 * Errors: NULL states/S0/desc (or transitions in EXACT with K >= 2), bad
 * mode/family/dtype, K < 0, id outside [0, n_chunks), sel_index outside
 * [0, K), misaligned pointers, unsupported dims, workspace too small.
 */
int lkv_init_state(const void *states, const void *transitions, int K, int mode, void *S0,
                   const lkv_init_desc *d, void *stream);

/*
 * The same for n_req requests in one launch (batched / ragged serving).
 *
 *   chunk_ids  HOST int32[cu_k[n_req]]  pool ids of all requests, concatenated, each in context order
 *   cu_k       HOST int32[n_req + 1]    request r owns chunk_ids[cu_k[r] .. cu_k[r+1])
 *   sel_index  HOST int32[n_req]        mode INDEX: position within each request; ignored otherwise (may be NULL)
 *   S0         out, float [n_req, H, d_k, d_v]
 * d->chunk_ids and d->sel_index are ignored.
 */
int lkv_init_state_batched(const void *states, const void *transitions, const int32_t *chunk_ids,
                           const int32_t *cu_k, int n_req, int mode, const int32_t *sel_index, void *S0,
                           const lkv_init_desc *d, void *stream);

/*
 * lkv_init_state_batched without any caller-provided scratch.  (The paper has no
 * counterpart: this entry point exists for integration reasons only.)
 *
 * Who needs it: code that runs where device memory cannot be allocated or handed
 * over -- a serving engine that has already given its whole memory budget to its own
 * pool and forbids cudaMalloc on the request path, a plugin called from inside
 * someone else's allocator-owned stream callback, a process that must not touch the
 * allocator while another component is capturing work.  Such a caller still owns the
 * inputs and the output, but has nowhere to get a workspace from.
 *
 * What differs from lkv_init_state_batched: d->workspace and d->workspace_bytes are
 * ignored.  The scratch the batched kernels use (status word + the request/chunk index
 * list) lives in a fixed array inside the library image, LKV_STATIC_SCRATCH_BYTES
 * bytes of device memory on every GPU that loads the library, held until the process
 * exits.  The call allocates nothing and frees nothing, directly or through a library.
 *
 * Limits and rules:
 *   - 2 * n_req + 1 + (number of chunk ids) must not exceed LKV_STATIC_MAX_INDEX;
 *     a larger request returns LKV_ERR_WORKSPACE and launches nothing.
 *   - The first call on each device looks up the array's device address (with that
 *     device current).  Make that first call outside any stream capture.
 *   - All calls on one device share the one array; it keeps whatever the previous
 *     call left in it, and every call rewrites the parts it reads before its kernel
 *     runs.  Two calls that can overlap on the GPU (different streams, no ordering
 *     between them) race on it: order them, or use lkv_init_state_batched with
 *     separate workspaces.
 *   - The status word of a bounded device-side wait lives in the same array (it
 *     starts at zero when the library is loaded).  The caller has no pointer to it:
 *     lkv_device_status_static() reads it, and clears it when it was set.
 *   - An argument error is found before anything is put on the stream.
 *   - Everything else (arguments, modes, errors, results) is as for
 *     lkv_init_state_batched; results are identical bit for bit.
 */
#define LKV_STATIC_MAX_INDEX 16384
#define LKV_STATIC_SCRATCH_BYTES (256 + 4 * LKV_STATIC_MAX_INDEX)
int lkv_init_state_batched_static(const void *states, const void *transitions, const int32_t *chunk_ids,
                                  const int32_t *cu_k, int n_req, int mode, const int32_t *sel_index,
                                  void *S0, const lkv_init_desc *d, void *stream);
/*
 * Status word of the scratch of lkv_init_state_batched_static on the current device: synchronises
 * `stream`, returns LKV_OK or LKV_ERR_DEVICE_TIMEOUT, and resets the word after reporting a time-out
 * (LKV_ERR_CUDA if a runtime call fails).  Allocates nothing.  (No counterpart in the paper.)
 */
int lkv_device_status_static(void *stream);

/*
 * Gated DeltaNet scan from an initial state (Eq. 1 with Eq. 3; Algorithm 1, line 3).
 * For each sequence and value head, in token order:
 *     S_t = exp(g_t) (I - beta_t k_t k_t^T) S_{t-1} + beta_t k_t v_t^T
 *     o_t = scale * S_t^T q_t
 * evaluated chunkwise: inside a block of tokens the triangular system that
 * couples the tokens (WY / UT transform) is solved at once, and the state is
 * carried from block to block.  S0 == NULL starts from the empty state;
 * S_T == NULL skips the final-state write; S_T may alias S0; o == NULL skips
 * the outputs (final states only; S_T is then required).  Sequences of
 * any length >= 0 are accepted (no padding is required).
 */
int lkv_gdn_fwd(const void *q, const void *k, const void *v, const float *g, const float *beta,
                const float *S0, void *o, void *S_T, const lkv_gdn_desc *d, void *stream);

/*
 * lkv_gdn_fwd for ONE long sequence, cut into n_segments segments that are scanned in parallel (a sequence-parallel
 * prefill; Eq. 5 and Eq. 6 applied inside one request): pass 1 computes, in one launch, the state each of the first
 * n_segments - 1 segments reaches from an empty start (the first one from S0) and the accumulated transitions of
 * segments 1 .. n_segments - 2; pass 2 composes the state every segment starts from (exact composition); pass 3 scans
 * all segments at once from those states.  About twice the arithmetic of lkv_gdn_fwd, but n_segments times the
 * CTAs: for a single sequence on an otherwise idle GPU it shortens the chain of dependent blocks.
 * Same arguments and results as lkv_gdn_fwd (results equal up to the rounding of the composition, which uses the
 * arithmetic of d->compute: tf32 products under AUTO / TENSOR at d = 128); requires d->n_seq == 1, d_k == d_v,
 * state_dtype fp32.  scratch: device, 16-byte aligned, >= lkv_gdn_segmented_scratch_bytes(d, n_segments) bytes, owned by
 * the caller.  n_segments == 1 is lkv_gdn_fwd itself; n_segments == 0 lets the library choose (as many segments as keep
 * both scanning passes within one round of CTAs on the current GPU, none shorter than 512 tokens; the scratch-size call
 * makes the same choice).  Five stream operations besides the three kernel launches
 * (memsets / device copies of single states).  (The paper has no counterpart: its prefill is the plain scan.)
 */
int lkv_gdn_fwd_segmented(const void *q, const void *k, const void *v, const float *g, const float *beta,
                          const float *S0, void *o, void *S_T, const lkv_gdn_desc *d, int n_segments,
                          void *scratch, size_t scratch_bytes, void *stream);
size_t lkv_gdn_segmented_scratch_bytes(const lkv_gdn_desc *d, int n_segments);

/*
 * Host-resident cache -> device staging pool (Section 4.1, "Environment": the cached artefacts live in host memory and
 * are loaded at serving time).  The chunks that a batch of requests names are copied, each once, from pools in HOST
 * memory (pinned for asynchronous copies) into compact pools in device memory, and the requests' chunk ids are rewritten
 * to the slots of the staging pools, ready for lkv_init_state_batched with d->n_chunks = *n_staged.
 *
 *   host_states, host_transitions  HOST pools laid out as lkv_init_desc describes (n_chunks = d->n_chunks entries);
 *                                  host_transitions may be NULL (single-state modes), then dev_transitions must be too
 *   chunk_ids                      HOST int32[n_ids], ids into the host pools, in any order, repeats allowed
 *   dev_states, dev_transitions    device staging pools with room for `capacity` chunks
 *   staged_ids                     HOST out int32[n_ids]: slot of chunk_ids[i]; slots are given in order of first appearance
 *   n_staged                       HOST out: number of distinct chunks copied
 * One cudaMemcpyAsync per chunk and pool on `stream`; nothing is copied when an argument is wrong or the distinct chunks
 * exceed `capacity` (LKV_ERR_WORKSPACE).  The host pools must stay valid until the copies have run.
 */
int lkv_stage_chunks(const void *host_states, const void *host_transitions, const int32_t *chunk_ids, int n_ids,
                     void *dev_states, void *dev_transitions, int capacity, int32_t *staged_ids, int32_t *n_staged,
                     const lkv_init_desc *d, void *stream);

/*
 * Mamba-2 (SSD) scan from an initial state (Eq. 1 with Eq. 2; Algorithm 1, line 3).
 * For each sequence and head, in token order:
 *     S_t = exp(dt_t A_h) S_{t-1} + dt_t B_t x_t^T,      y_t = S_t^T C_t
 * evaluated chunkwise (intra-block masked contraction + inter-block state carry).
 * NULL conventions as in lkv_gdn_fwd.
 */
int lkv_ssd_fwd(const void *x, const float *dt, const float *A, const void *B, const void *C,
                const float *S0, void *y, void *S_T, const lkv_ssd_desc *d, void *stream);

/*
 * Producers of the cached artefacts that exact composition consumes (Eq. 5: a chunk C maps an incoming
 * state as S_out = T_C S_in + S_local).  S_local of a chunk is the final state of a scan of the chunk from
 * the empty state: call lkv_gdn_fwd / lkv_ssd_fwd with S0 == NULL and the chunks as sequences (o / y may
 * be NULL there when only final states are wanted).  The two calls below give the other half, T_C.
 *
 * lkv_gdn_chunk_transition: for every sequence (= cache chunk) c of `cu_seqlens` and every value head h,
 *     T_c = prod_t exp(g_t) (I - beta_t k_t k_t^T)      (Eq. 3; later tokens on the left)
 * written to transitions[c][h] as a row-major d_k x d_k fp32 matrix (device, n_seq x H_v x d_k x d_k), the
 * layout lkv_init_state reads.  It is the scan run from S = I with v = 0, so `d` is the descriptor of
 * lkv_gdn_fwd on the same tokens (d_v must equal d_k; scale is ignored); k, g, beta as in lkv_gdn_fwd.
 * An empty chunk gives the identity.  Precision is that of the scan path `d->compute` selects.
 *
 * lkv_mamba_chunk_logdecay: for every sequence c and head h, lambda[c][h] = A_h * sum_t dt_t (fp32, device,
 * n_seq x H): exp(lambda) is the scalar T_c of Eq. 2 / Eq. 5, kept as a logarithm because it underflows
 * fp32 for long chunks.  `d` is the descriptor of lkv_ssd_fwd on the same tokens (P, N, G unused).
 *
 * Errors as for the scans (LKV_ERR_DIM if d_v != d_k).  Both need the scan workspace.
 */
int lkv_gdn_chunk_transition(const void *k, const float *g, const float *beta, float *transitions,
                             const lkv_gdn_desc *d, void *stream);
int lkv_mamba_chunk_logdecay(const float *dt, const float *A, float *logdecay, const lkv_ssd_desc *d, void *stream);

/*
 * Both cached artefacts of every GDN chunk in ONE launch: states[c] = the state chunk c reaches from an empty start
 * (S_local) and transitions[c] = its accumulated transition T_C (Eq. 5), fp32 [n_seq, H_v, d, d] each, the chunks being
 * the sequences of d->cu_seqlens.  Every chunk is scanned twice inside the launch (once with its values from S = 0, once
 * with v = 0 from S = I); what one launch buys over lkv_gdn_fwd + lkv_gdn_chunk_transition is that the two scans of a
 * chunk run side by side, which matters when a few chunks do not fill the GPU.  Results are bit-identical to those two
 * calls.  k, v, g, beta and errors as for lkv_gdn_fwd (d_k == d_v required; state_dtype must be fp32); the workspace must
 * be sized for 2 * n_seq sequences (lkv_workspace_bytes(LKV_WS_GDN, d, 2 * n_seq, 0)).
 */
int lkv_gdn_chunk_artifacts(const void *k, const void *v, const float *g, const float *beta, float *states,
                            float *transitions, const lkv_gdn_desc *d, void *stream);

/*
 * GDN exact composition for ONE request WITHOUT materialised transitions (the "online fold": Eq. 6 evaluated as the
 * chain of Eq. 5 with every T_C applied token by token from the chunk's cached key / gate stream):
 *     S <- S_{c_1};   S <- (scan of chunk c_j's tokens with v = 0 from S) + S_{c_j},   j = 2..K.
 * It trades the d_k x d_k fp32 transition per (chunk, head) for the chunk's k / g / beta stream and one scan per chunk.
 *
 *   states     fp32 pool [n_chunks, H, d_k, d_v] (d->state_dtype must be LKV_DTYPE_F32)
 *   k          [total_tokens, H_k, d_k] io_dtype, the cached chunks' keys back to back in pool order
 *   g, beta    float [total_tokens, H] as for lkv_gdn_fwd (H = d->H value heads)
 *   cu_tokens  HOST int32[n_chunks + 1]: chunk c owns tokens cu_tokens[c] .. cu_tokens[c + 1]
 *   K, d->chunk_ids, S0, d->workspace, d->compute as for lkv_init_state; d->family must be LKV_FAMILY_GDN, d_k == d_v.
 * Launches 1 + (K - 1) kernels on `stream`.  The result equals lkv_init_state(..., LKV_INIT_EXACT) on transitions
 * built by lkv_gdn_chunk_transition from the same streams, up to rounding.  Errors as for lkv_init_state and the scans.
 */
int lkv_init_state_fold(const void *states, const void *k, const float *g, const float *beta,
                        const int32_t *cu_tokens, int K, void *S0, const lkv_init_desc *d, int H_k, int io_dtype,
                        void *stream);

/*
 * Diagnostic of Section 3.2 ("Diagnosis via relative error"): how far a constructed initial state is from the
 * true full-prefix state, rel_err[i] = ||S_init_i - S_ref_i||_F / ||S_ref_i||_F for i < n_states, where state i
 * is the i-th run of state_elems consecutive fp32 values of S_init / S_ref (device; a run may be one head's
 * state, one request's, or a whole layer's).  rel_err: n_states fp32 (device).  state_elems must be a positive
 * multiple of 4 and both arrays 16-byte aligned.  The workspace (device, 16-byte aligned) holds the partial sums:
 * at least lkv_state_rel_error_workspace_bytes(n_states, state_elems) bytes.  Sums are fp32 accumulated in a
 * fixed order (deterministic).  A zero reference gives inf (nan if the constructed state is zero too).
 */
int lkv_state_rel_error(const float *S_init, const float *S_ref, float *rel_err, int n_states, size_t state_elems,
                        void *workspace, size_t workspace_bytes, void *stream);
size_t lkv_state_rel_error_workspace_bytes(int n_states, size_t state_elems);

/*
 * Workspace size in bytes for a call described by `desc` (lkv_init_desc, lkv_gdn_desc or
 * lkv_ssd_desc according to `which`).  n_units is the number of requests (init) or
 * sequences (scans) and n_index the total number of chunk ids over all requests
 * (init; 0 for the scans).  Returns 0 for a NULL or invalid descriptor.
 */
size_t lkv_workspace_bytes(int which, const void *desc, int n_units, int n_index);

/*
 * Reads the device status word of a workspace: synchronises `stream`, copies 4 bytes to
 * the host, and returns LKV_OK or LKV_ERR_DEVICE_TIMEOUT (LKV_ERR_CUDA if the copy fails).
 * The only call here that blocks the host.
 */
int lkv_device_status(const void *workspace, void *stream);

/*
 * Self-test of the bounded device-side waits (no counterpart in the paper): launches one small kernel that
 * waits, with the wait every tensor-core kernel of the library uses, on a barrier nobody will ever arrive on,
 * giving up after `poll_limit` polls (1 .. 2^20).  The kernel then sets the status word of `workspace`
 * (device, 16-byte aligned, at least 256 bytes, zeroed by the caller) and ends; it neither traps nor spins on.
 * Afterwards lkv_device_status(workspace) must report LKV_ERR_DEVICE_TIMEOUT, and word 1 of the workspace
 * must still be zero (it is set if a wait claimed to have succeeded).
 */
int lkv_selftest_bounded_wait(int poll_limit, void *workspace, void *stream);

/* Human-readable name of a status code (static storage, never NULL). */
const char *lkv_status_string(int status);

/* LKV_VERSION of the loaded library. */
int lkv_version(void);

#ifdef __cplusplus
}
#endif
#endif /* LKV_H_ */
