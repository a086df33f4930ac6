/*
 * smat.h — C boundary of the B200 chunkwise hard-routing SMat-Attention prefill.
 *
 * The library computes, for every (batch, head) independently,
 *
 *        O = (M^(d) ⊙ Q Kᵀ) V                                  [Sec. 2, augmented output with
 *                                                                identity feature maps, no division]
 *
 * under the structured causal mask family M^(d) of Sec. 3 (block form, Eq. "blockform";
 * point–hyperplane incidences over F_q^{d-1}, Eq. "Bcount", Eq. "Gdef"; positional
 * assignment of profiles and types), without ever materialising M^(d): Algorithm 1
 * (pool → tabulate → typed read ‖ chunk summaries → scan → per-chunk output) with the
 * implicit incidence tabulation of Algorithm 2, and the matching backward pass of the
 * chunking proof (Eq. "lr-adjoint", Eq. "local-adjoint", suffix scan).
 *
 * Conventions shared by all entry points
 *   - Plain C linkage; no exceptions; the library keeps no global mutable state, with one exception that is
 *     stated where it applies: the fixed device array (and its cached address) behind smat_forward_causal_static.
 *   - Q, K are [batch, heads, T, d_k]; V, O, dO are [batch, heads, T, d_v]; dQ, dK like Q,
 *     dV like V.  All are DEVICE pointers to contiguous row-major arrays (feature dimension
 *     fastest) of the plan's dtype, 16-byte aligned.  Accumulation is fp32.
 *   - The workspace is a DEVICE buffer owned by the caller, at least smat_workspace_bytes()
 *     long and 256-byte aligned.  The library allocates no device memory, keeps no pointer
 *     after a call returns, launches only on the stream it is given (a cudaStream_t passed
 *     as void*; NULL is the default stream) and never synchronises it, except where stated.
 *   - Every function returns a status code; argument errors are detected before any launch.
 *   - Tokens are 0-based; token t < n is "distant", t >= n is "recent"; the paper's 1-based
 *     recent index is i = t - n + 1.
 */
#ifndef SMAT_H_
#define SMAT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct smat_plan smat_plan; /* opaque, host memory, immutable after creation */

typedef enum {
  SMAT_OK = 0,
  SMAT_ERR_NULL = 1,           /* a required pointer is NULL */
  SMAT_ERR_SHAPE = 2,          /* unsupported batch/heads/T/d_k/d_v/chunk combination */
  SMAT_ERR_DTYPE = 3,          /* unknown dtype */
  SMAT_ERR_GEOMETRY = 4,       /* d out of range, q not prime, q^(d-1) too large, T < 2*chunk with d >= 2 */
  SMAT_ERR_WORKSPACE = 5,      /* workspace too small */
  SMAT_ERR_ALIGN = 6,          /* a pointer is not aligned as required */
  SMAT_ERR_ARCH = 7,           /* the current device is not compute capability 10.x */
  SMAT_ERR_LAUNCH = 8,         /* a CUDA launch or runtime call failed */
  SMAT_ERR_DEVICE_TIMEOUT = 9, /* a bounded device-side wait expired (read by smat_check_status) */
  SMAT_ERR_UNSUPPORTED = 10    /* the request is valid but this build has no path for it */
} smat_status;

typedef enum { SMAT_F32 = 0, SMAT_BF16 = 1 } smat_dtype;

/* plan flags */
#define SMAT_FLAG_SIMT_ONLY 1u      /* never use the tensor-core kernels (bf16 plans run the fp32-ALU path) */
#define SMAT_FLAG_ALG2_TABULATION 2u /* tabulate with the direct double loop of Algorithm 2 instead of the staged sums */
#define SMAT_FLAG_KEEP_FORWARD_TABLES 8u /* smat_backward does not rebuild the profile and type tables F, U: the caller
                                            promises that `workspace` still holds what smat_forward wrote for the same
                                            K, V with this plan (no other call on that workspace in between).  With
                                            SMAT_FLAG_GATED: smat_backward_gated right after smat_forward_gated of the
                                            same inputs and gates (tensor-core shapes) reuses its tables likewise; after
                                            any other call it rebuilds them */
#define SMAT_FLAG_PER_TILE_STATES 4u /* tensor-core causal branch: store one incoming state per 128-token tile (scan, then
                                        independent tiles) instead of one per segment of tiles (two-level form) */

#define SMAT_FLAG_ALU_TABULATION 16u /* d = 3, 4 on the tensor-core path: keep the profile table in fp32 and tabulate
                                        with staged sums on the fp32 ALUs instead of the Radon stages on the tensor cores
                                        (which keep F, U and the stage intermediate in bf16) */

#define SMAT_FLAG_D3_SHARED_SUMS 32u /* d = 3 with a prime beyond the tensor-core tabulation: form every q-term sum
                                        straight from the shared-memory slab (one output row per thread) instead of
                                        the register-resident form (K slopes x q offsets per thread) */

#define SMAT_FLAG_SEPARATE_TILE_ADJOINTS 256u /* tensor-core backward: dQ, dK, dV of a tile by three launches of the general
                                                 tile-product kernel instead of the one fused kernel (for comparison) */
#define SMAT_FLAG_GATED 64u          /* the plan serves smat_forward_gated / smat_backward_gated: its workspace holds λ and the
                                        rescaled copies of Q, K, V, dO.  Both passes run on the tensor cores where the
                                        shape allows (with SMAT_FLAG_SIMT_ONLY: never), else on the fp32-ALU kernels */

#define SMAT_FLAG_NORMALIZED 128u    /* the plan serves smat_forward_normalized / smat_backward_normalized: its workspace
                                        also holds the augmented values, the unnormalised rows and their upstream */

/* Sizes of the construction (Sec. 3, "construction of G" and "Scaling with sequence length"). */
typedef struct {
  int64_t T, c, n, m;  /* sequence length, chunk width, distant = c*floor(T/2c), recent = T - n */
  int32_t d, q;        /* VC dimension; prime field size (0 when d = 1) */
  int64_t P;           /* profile cells q^(d-1)            (1 when d = 1) */
  int64_t A;           /* normalised directions (q^(d-1)-1)/(q-1) (1 when d = 1) */
  int64_t B;           /* types = hyperplanes = q*A = cached subset states (1 when d = 1) */
  int64_t nnzC;        /* nonzeros of the incidence matrix = B*q^(d-2) */
  int32_t vc_conditions_met; /* P <= n and 2B <= m, the conditions of the positional construction */
} smat_geometry;

/*
 * Create a plan for one problem shape.
 *   batch, heads >= 1; T >= 1 and a multiple of `chunk`; d_k, d_v in {64, 128};
 *   chunk in {16, 32, 64, 128}; d in [1, 8] is the VC dimension of the mask (d = 1: causal mask).
 *   q_override = 0 takes the default field size, the smallest prime q with q^d >= n
 *   (Sec. 3 asks for q = Θ(n^{1/d}); this constant reproduces the cache sizes the paper prints);
 *   any other value must be a prime and is used as given (small test cases).
 * On success *out owns host memory until smat_plan_destroy.  No device work is done and no device is queried: the
 * kernels a plan uses follow from the shape and the flags alone.  Calls that launch return SMAT_ERR_ARCH when the
 * current device is not compute capability 10.x (the library holds sm_100a code only).
 */
smat_status smat_plan_create(smat_plan** out, int batch, int heads, int64_t T, int d_k, int d_v, int d, int chunk,
                             int q_override, smat_dtype dtype, unsigned flags);
void smat_plan_destroy(smat_plan* plan);

smat_status smat_get_geometry(const smat_plan* plan, smat_geometry* out);

/* 1 when this plan runs its causal branch on the tcgen05 tensor-core kernels (bf16, d_k = d_v = 128, block
 * boundary and recent length multiples of 128, SMAT_FLAG_SIMT_ONLY not set), 0 when it runs on the fp32 ALUs.
 * A property of the shape, not of the device. */
int smat_uses_tensor_cores(const smat_plan* plan);

/* 1 when smat_forward_gated / smat_backward_gated of this plan (SMAT_FLAG_GATED) run on the tensor-core kernels: the
 * same shape rule as above (the backward also needs the plan to keep its tables in bf16, which the tabulation flags
 * can prevent).  Every other shape runs on the fp32 ALUs.  The gated passes go through a plan of their own inside the
 * gated plan; smat_uses_tensor_cores of a gated plan itself is 0. */
int smat_gated_forward_uses_tensor_cores(const smat_plan* plan);
int smat_gated_backward_uses_tensor_cores(const smat_plan* plan);

/* Bytes per element of the type table U as smat_forward keeps it: 4 (fp32), or 2 when the plan runs the typed read on
 * the tensor cores (bf16 inputs; d >= 3, or d = 2 with at least 12 tokens per profile): there U is only ever a bf16
 * MMA operand, so it is rounded once when it is stored and the table's HBM traffic halves (for d = 2 the profile
 * table is the type table and is kept in bf16 too). */
int smat_type_table_element_bytes(const smat_plan* plan);

/* Bytes per element of the profile table F as smat_forward keeps it: 2 for d = 2 on the tensor-core path and for
 * d = 3, 4 when the tabulation (Algorithm 2) runs as Radon stages on the tensor cores — F, the stage intermediate and
 * U are then bf16 MMA operands, sums are taken in fp32 — else 4.  On those plans smat_backward keeps the adjoint
 * tables (the per-type sums of q dOᵀ and their transposed tabulation) in bf16 as well. */
int smat_profile_table_element_bytes(const smat_plan* plan);

/* Bytes of workspace smat_forward (for_backward = 0) or smat_backward (for_backward = 1) needs. 0 if plan is NULL.
 * Every region is sized for the element type the plan stores in it (bf16 tables on tensor-core plans), and the
 * score-tile buffers of the fp32-ALU path are reserved only for plans that run on it. */
size_t smat_workspace_bytes(const smat_plan* plan, int for_backward);

/*
 * Forward pass, Algorithm 1 steps 2-7 (step 1 is implicit: φ = q_i, ψ = k_j, Z_j = k_j v_jᵀ).
 * Reads Q, K, V; writes O (plan dtype).  The profile table F and the type table U ("cached subset
 * states") are left in the workspace in the element type the plan keeps them in (fp32, or bf16: see
 * smat_profile_table_element_bytes / smat_type_table_element_bytes), the incoming states S_in as fp32 per
 * chunk (fp32-ALU plans) or as bf16 per 128-token tile (tensor-core plans with SMAT_FLAG_PER_TILE_STATES);
 * smat_debug_tables reads them back widened to fp32.  Asynchronous on `cuda_stream`.
 */
smat_status smat_forward(const smat_plan* plan, const void* Q, const void* K, const void* V, void* O, void* workspace,
                         size_t workspace_bytes, void* cuda_stream);

/*
 * Backward pass (chunking proof, "Backward Pass"): given dO = ∂L/∂O writes dQ, dK, dV (plan dtype).
 * It rebuilds the forward tables it needs (S_in, F, U) inside the workspace, so it does not
 * depend on an earlier smat_forward call — unless the plan was created with SMAT_FLAG_KEEP_FORWARD_TABLES
 * (tensor-core plans only), in which case F and U are taken from the workspace as the preceding smat_forward
 * left them.  Asynchronous on `cuda_stream`.
 */
smat_status smat_backward(const smat_plan* plan, const void* Q, const void* K, const void* V, const void* dO, void* dQ,
                          void* dK, void* dV, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The same two passes under USER-SUPPLIED ROUTING (Sec. 3, "construction of G", the content-based assignment: any map
 * of distant tokens to profile cells and of recent tokens to types gives G_ij = C[type(i), prof(j)], Eq. "Gdef" with
 * the incidence matrix of Eq. "C"; the positional assignment is the special case smat_routing_indices returns).
 *   prof [batch*heads, n]  DEVICE int32: the packed cell index in [0, P) of distant token t of every (batch, head)
 *                          (little-endian base-q digits, as smat_routing_indices packs them)
 *   type [batch*heads, m]  DEVICE int32: the type h = dir*q + b in [0, B) of recent token n + i
 * Both are read once per call: a stable counting sort turns them into per-cell and per-type token lists in the
 * workspace, and pooling (step 2), the typed read (step 4) and their adjoints walk those lists — a data-dependent
 * gather — instead of the positional strides; tabulation and the causal branch are unchanged.  An entry outside its
 * range puts the token in no group (it writes to, or reads from, no cached state).  Group sizes may be arbitrarily
 * skewed, including empty groups.  d = 1 ignores both arrays (one cell, one type).  Everything else — workspace
 * size, dtypes, errors — is as for smat_forward / smat_backward; SMAT_ERR_UNSUPPORTED if P or B exceeds 27000.
 */
smat_status smat_forward_routed(const smat_plan* plan, const void* Q, const void* K, const void* V, void* O,
                                const int32_t* prof, const int32_t* type, void* workspace, size_t workspace_bytes,
                                void* cuda_stream);
smat_status smat_backward_routed(const smat_plan* plan, const void* Q, const void* K, const void* V, const void* dO,
                                 void* dQ, void* dK, void* dV, const int32_t* prof, const int32_t* type,
                                 void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * NORMALISED OUTPUT (Sec. 2, Eq. "augmented-kv-state", Eq. "augmented-attention-output"; "backward of the final
 * division" in the chunking proof).  The value is augmented with a ones column, v̄_j = [v_j; 1], the linear pass runs
 * once on it, and one division at the end gives o_i = ȳ_{1:p-1} / ȳ_p.  Here the augmented width is the plan's
 * d_v = p: V carries p - 1 value columns and its LAST column is the normaliser column — the library replaces whatever
 * the caller left there by one.  O [batch, heads, T, p] receives the normalised values in columns 0 .. p-2 and the
 * normaliser ȳ_p itself in column p-1.  The caller supplies the (non-negative) features φ = Q, ψ = K; the normalisers
 * must be positive, as Theorem 2 assumes.
 * smat_backward_normalized takes the O that the forward returned (it holds the normaliser) and dO of the same shape
 * (its last column is the upstream of the normaliser output; pass zeros if unused); dV's last column is returned as
 * zero.  The plan must carry SMAT_FLAG_NORMALIZED.  Otherwise as smat_forward / smat_backward.
 */
smat_status smat_forward_normalized(const smat_plan* plan, const void* Q, const void* K, const void* V, void* O,
                                    void* workspace, size_t workspace_bytes, void* cuda_stream);
smat_status smat_backward_normalized(const smat_plan* plan, const void* Q, const void* K, const void* V, const void* O,
                                     const void* dO, void* dQ, void* dK, void* dV, void* workspace,
                                     size_t workspace_bytes, void* cuda_stream);

/*
 * SCALAR-GATED SMat (Sec. 3.2, Eq. "gated"; Lemma "Gated SMat"): the binary mask is replaced by
 *        M~_ij = M_ij exp(λ_i - λ_j),   λ_i = Σ_{k <= i} log a_k,   j <= i,
 * for per-token decay gates a_k in (0, 1].  log_a is a DEVICE fp32 array [batch*heads, T] of log-gates (<= 0).
 * The chunkwise form of the lemma is used: λ by one prefix sum; within-chunk tiles times exp(λ_i - λ_j); chunk
 * summaries of keys scaled to the chunk's last index; the carried state decayed by every chunk it passes and read with
 * exp(λ_i - λ_{e(b-1)}); in the long-range branch the factor splits at the block boundary into a key-side scalar folded
 * into k_j before pooling and a query-side scalar on the typed read, so tables and tabulation are the ungated ones of
 * rescaled inputs.  Every factor is the exponential of a non-positive difference: nothing overflows however strong
 * the decay.  smat_backward_gated also returns dlog_a [batch*heads, T] (DEVICE fp32), the gradient with respect to the
 * log-gates.  The plan must carry SMAT_FLAG_GATED (else SMAT_ERR_UNSUPPORTED).  The passes run on the tensor
 * cores where smat_gated_forward_uses_tensor_cores / smat_gated_backward_uses_tensor_cores say so, else on the fp32-ALU
 * kernels.
 * Otherwise as smat_forward / smat_backward.
 */
smat_status smat_forward_gated(const smat_plan* plan, const void* Q, const void* K, const void* V, const float* log_a,
                               void* O, void* workspace, size_t workspace_bytes, void* cuda_stream);
smat_status smat_backward_gated(const smat_plan* plan, const void* Q, const void* K, const void* V, const float* log_a,
                                const void* dO, void* dQ, void* dK, void* dV, float* dlog_a, void* workspace,
                                size_t workspace_bytes, void* cuda_stream);

/*
 * Routing as the library's index code sees it (HOST output buffers, caller-allocated):
 *   prof    [n * (d-1)]  base-q digits of (t mod P), least significant first      (Sec. 3, positional assignment)
 *   type    [m]          (t - n + 1) mod B for t = n .. T-1
 *   type_ab [B * d]      for every type h = dir*q + b: the direction a (d-1 entries), then b
 * Any of the three may be NULL to skip it.  For d = 1 prof is empty, type is all zeros and
 * type_ab holds the single entry 0.
 */
smat_status smat_routing_indices(const smat_plan* plan, int32_t* prof, int32_t* type, int32_t* type_ab);

/*
 * The mask M^(d) as the DEVICE index code evaluates it: mask is a DEVICE buffer of T*T bytes
 * (row-major, 0/1).  Only for T <= 8192.  Asynchronous on `cuda_stream`.
 */
smat_status smat_debug_mask(const smat_plan* plan, uint8_t* mask, void* cuda_stream);

/*
 * Copies, widened to fp32, of the tables a finished forward (or backward) left in `workspace`, into DEVICE
 * buffers (any may be NULL):
 *   F   [batch*heads, P, d_k, d_v]     profile table        (Eq. "schedule")
 *   U   [batch*heads, B, d_k, d_v]     type table           (Eq. "schedule", Algorithm 2)
 *   Sin [batch*heads, T/w, d_k, d_v]   incoming states of the causal branch (Sec. 3.1), one per chunk (w = chunk) on
 *                                      fp32-ALU plans, one per 128-token tile (w = 128) on tensor-core plans
 * For d = 1 there is no separate F/U: the single state U_0 = F_0 is carried by the scan, and
 * F and U receive that state (the incoming state of the first recent chunk or tile).
 * Tensor-core plans have per-tile states only after a forward of a plan created with SMAT_FLAG_PER_TILE_STATES, or
 * after smat_backward; the two-level form keeps one state per segment of tiles, which is no per-chunk table: there
 * Sin (and, for d = 1, F and U) must be NULL, otherwise SMAT_ERR_UNSUPPORTED is returned.
 * Asynchronous on `cuda_stream`.
 */
smat_status smat_debug_tables(const smat_plan* plan, const void* workspace, float* F, float* U, float* Sin,
                              void* cuda_stream);

/*
 * Synchronises `cuda_stream` and reads the device status word kept at the start of the
 * workspace.  Returns SMAT_OK, SMAT_ERR_DEVICE_TIMEOUT if a bounded wait inside a kernel
 * expired (the kernel then returned early and the outputs are invalid), or SMAT_ERR_LAUNCH
 * if the stream reports a CUDA error.
 */
smat_status smat_check_status(const smat_plan* plan, const void* workspace, void* cuda_stream);

/*
 * Per-kernel timing for measurement (the paper has no counterpart; this serves the roofline report).
 * While enabled, smat_forward / smat_backward record a CUDA event on the launching stream before
 * and after every kernel they launch.  The events belong to the plan and to the device that was
 * current when profiling was enabled; disable before destroying the context.
 * smat_profile_read waits for the last recorded event, then fills up to max_stages kernel names
 * (static strings) and durations in milliseconds, in launch order, and returns how many it filled.
 */
smat_status smat_profile_enable(smat_plan* plan, int enable);
int smat_profile_read(const smat_plan* plan, const char** names, float* ms, int max_stages);

/*
 * Causal forward without any workspace from the caller (the paper has no counterpart: this exists for
 * integration, not for the method).  Computes O = (L_T ⊙ QKᵀ)V — the d = 1 member of the family — for
 * bf16 Q, K, V, O of shape [batch, heads, T, 128] (DEVICE pointers, 16-byte aligned, T a multiple of 128).
 *
 * Who needs it: callers that cannot allocate device memory themselves — a plug-in inside an application
 * that owns the whole device heap, or a serving loop that bans cudaMalloc on its request path because an
 * allocation can synchronise the device.  The incoming chunk states this path needs live in a fixed array
 * inside the library image (SMAT_STATIC_MAX_TILES bf16 states of 32 KB plus a status word, 32 MiB in all,
 * resident on every device that loads the library until the process exits).  The call allocates nothing,
 * neither with cudaMalloc nor through any library.
 *
 * Limit: batch * heads * (T / 128) <= SMAT_STATIC_MAX_TILES, otherwise SMAT_ERR_WORKSPACE (use smat_forward
 * with a workspace of your own).  Other errors as for smat_forward; SMAT_ERR_ARCH if the tensor-core path is
 * unavailable.
 *
 * The first call on each device looks up the device address of that array (with the device current); make
 * that first call outside any stream capture.  All calls on a device share the one array, which keeps the
 * previous call's contents (the library clears the part that must start at zero): two calls that overlap on
 * the GPU — different streams, or different host threads — race on it, so serialise them.
 * Asynchronous on `cuda_stream`.
 */
#define SMAT_STATIC_MAX_TILES 1024
smat_status smat_forward_causal_static(const void* Q, const void* K, const void* V, void* O, int batch, int heads,
                                       int64_t T, void* cuda_stream);

/*
 * Status of the last smat_forward_causal_static on the current device (the paper has no counterpart).  That call has
 * no workspace whose status word smat_check_status could read, so this reads the word kept in the static array:
 * synchronises `cuda_stream`, returns SMAT_OK, SMAT_ERR_DEVICE_TIMEOUT if a bounded wait inside its kernels ran out
 * (O is then invalid), or SMAT_ERR_LAUNCH if the stream reports a CUDA error.  Allocates nothing.
 */
smat_status smat_static_check_status(void* cuda_stream);

/*
 * Failure-path probe (the paper has no counterpart).  Launches a one-warp kernel in which one thread waits, with the
 * same bounded wait every kernel of the library uses, on a barrier that nobody arrives on; after `limit_cycles` SM
 * clock cycles (1 .. 2e9) the wait gives up, sets the status word at the start of `workspace` (DEVICE, 256-byte
 * aligned, at least 256 bytes) and the kernel returns normally.  smat_check_status on that workspace then reports
 * SMAT_ERR_DEVICE_TIMEOUT; the next smat_forward / smat_backward clears the word again.  Nothing faults or hangs.
 */
smat_status smat_debug_timeout_probe(void* workspace, int64_t limit_cycles, void* cuda_stream);

/*
 * Measured fp32 add rate of the plain ALUs of the current device (the paper has no counterpart; this is the ceiling
 * the state additions of Algorithm 2 are charged against in the roofline report).  Runs independent register add
 * chains on every SM, scalar adds (packed = 0) or two-lane adds (packed = 1), times them with CUDA events on
 * `cuda_stream`, synchronises, and writes additions per second to *adds_per_second (HOST).  `scratch` is a DEVICE
 * buffer of at least 4 bytes.
 */
smat_status smat_measure_fadd_rate(void* scratch, int packed, double* adds_per_second, void* cuda_stream);

/* ---- Cached decoding of the recent block (Sec. "Memory-efficient decoding", Theorem "Streaming decoding") ----
 * The plan fixes T and with it the boundary n.  After the distant block (tokens 0 .. n-1) the decoder keeps B type
 * states U_h and one running state S per (batch, head); each recent token t = n, n+1, ... then costs O(d_k d_v):
 *     S_t = S_{t-1} + k_t v_t^T   (S_{n-1} = 0),      o_t = q_t^T (U_type(t) + S_t),     type(t) = (t - n + 1) mod B.
 * o_t equals row t of smat_forward's O (no normaliser, like the rest of the library).
 *
 * cache: device memory owned by the caller, 256-byte aligned, smat_decode_cache_bytes(plan) bytes:
 *        the type table [B*H][B][d_k][d_v] in the element type smat_type_table_element_bytes reports (fp32 for d = 1),
 *        then S [B*H][d_k][d_v] in fp32.
 * smat_decode_begin : K [B,H,T,d_k], V [B,H,T,d_v] device pointers of which rows 0 .. n-1 of every head are read;
 *        pools and tabulates them (steps 2-3 of Algorithm 1, through `workspace` as smat_forward would), stores the
 *        type table in the cache and zeroes S.  workspace: as for smat_forward (for_backward = 0).
 * smat_decode_step  : q, k [B,H,d_k], v [B,H,d_v] device rows of token t for every (batch, head) in the plan's dtype,
 *        o [B,H,d_v] device output in the same dtype.  Steps must be issued for t = n, n+1, ... in order, on one
 *        stream (S is updated in place).  n <= t < T, else SMAT_ERR_SHAPE.
 * Both launch on the given stream and return without synchronising; errors as for smat_forward. */
size_t smat_decode_cache_bytes(const smat_plan* plan);
smat_status smat_decode_begin(const smat_plan* plan, const void* K, const void* V, void* cache, size_t cache_bytes,
                              void* workspace, size_t workspace_bytes, void* cuda_stream);
smat_status smat_decode_step(const smat_plan* plan, const void* q, const void* k, const void* v, int64_t t, void* o,
                             void* cache, size_t cache_bytes, void* cuda_stream);

/* The same for the scalar-gated variant (Sec. 3.2, the streaming form of Lemma "Gated SMat"); the plan must carry
 * SMAT_FLAG_GATED (the ungated pair of calls then returns SMAT_ERR_UNSUPPORTED, and these on an ungated plan):
 *     S_t = a_t S_{t-1} + k_t v_t^T,   g_t = a_t g_{t-1}  (g_{n-1} = 1),   o_t = q_t^T (g_t U_type(t) + S_t),
 * where the cached type table is built from the keys rescaled to the block boundary, exp(λ_{n-1} - λ_j) k_j.
 * o_t equals row t of smat_forward_gated's O.  The cache holds, after the type table (bf16 where the plan's gated
 * forward runs on the tensor cores, else fp32) and S, one fp32 word per (batch, head): log g.
 * smat_decode_begin_gated : log_a DEVICE fp32 [B*H, T] as for smat_forward_gated (entries 0 .. n-1 of every head are used).
 * smat_decode_step_gated  : log_a_t DEVICE fp32 [B*H], the log-gates of token t. */
smat_status smat_decode_begin_gated(const smat_plan* plan, const void* K, const void* V, const float* log_a, void* cache,
                                    size_t cache_bytes, void* workspace, size_t workspace_bytes, void* cuda_stream);
smat_status smat_decode_step_gated(const smat_plan* plan, const void* q, const void* k, const void* v, const float* log_a_t,
                                   int64_t t, void* o, void* cache, size_t cache_bytes, void* cuda_stream);

/* Host-only self-check (the paper has no counterpart): 1 when, for field size q, the shared-memory map of every launch
 * shape of the tensor-core tabulation kernel (ring slots, extra-class rows, output-row table, barrier words) is
 * disjoint and inside the allocation, and no load box or staged tile can leave its slot; 0 otherwise.  The launcher
 * makes the same check before every launch. */
int smat_debug_tabulation_layout_ok(int q);

/* Number of kernels the last smat_forward / smat_backward on this plan launched (host counter). */
int smat_last_launch_count(const smat_plan* plan);

const char* smat_status_string(smat_status s);

#ifdef __cplusplus
}
#endif
#endif /* SMAT_H_ */
