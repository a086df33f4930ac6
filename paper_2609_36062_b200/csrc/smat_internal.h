// Internal declarations shared by the translation units of libsmat (not part of the C boundary).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "smat_geometry.h"

// ---- token groups -----------------------------------------------------------------------------
// A "group" is a set of tokens t0, t0+ts, t0+2ts, ... that one state belongs to:
//   CHUNK   g = chunk index        tokens g*c .. g*c+c-1                          (Sec. 3.1, causal branch)
//   PROFILE g = packed profile x   distant tokens t ≡ x (mod P), t < n            (Eq. "schedule", F_x)
//   TYPE    g = type h             recent tokens with (t-n+1) ≡ h (mod B), t < T  (Eq. "schedule", U_h)
enum SmatGroupMode { SMAT_GM_NONE = 0, SMAT_GM_CHUNK = 1, SMAT_GM_PROFILE = 2, SMAT_GM_TYPE = 3 };

struct SmatGroupSpec {
  int mode;
  int64_t n, T, c, period;  // period = P (PROFILE) or B (TYPE)
  // User-supplied routing (content-based assignment, Sec. 3): when `list` is non-null the tokens of PROFILE / TYPE
  // group g of head bh are list[bh * list_stride + offs[bh * offs_stride + g] ...  offs[... + g + 1]) (token positions
  // in [0, T), ascending inside a group) instead of the positional strides.
  const int32_t* list;
  const int32_t* offs;
  int64_t list_stride, offs_stride;
};

// The tokens of one group: position of the k-th one is at(k).
struct SmatTokens {
  int64_t t0, ts, cnt;
  const int32_t* lst;
  SMAT_HD int64_t at(int64_t k) const { return lst ? (int64_t)lst[k] : t0 + k * ts; }
};

SMAT_HD SmatTokens smat_group_tokens(const SmatGroupSpec& s, int64_t bh, int64_t g) {
  SmatTokens r;
  r.lst = nullptr; r.t0 = 0; r.ts = 1; r.cnt = 0;
  if (s.mode != SMAT_GM_CHUNK && s.list) {
    const int32_t* o = s.offs + bh * s.offs_stride + g;
    r.lst = s.list + bh * s.list_stride + o[0];
    r.cnt = o[1] - o[0];
    return r;
  }
  switch (s.mode) {
    case SMAT_GM_CHUNK:
      r.t0 = g * s.c; r.ts = 1; r.cnt = s.c;
      break;
    case SMAT_GM_PROFILE:
      r.t0 = g; r.ts = s.period; r.cnt = g < s.n ? (s.n - g + s.period - 1) / s.period : 0;
      break;
    case SMAT_GM_TYPE: {
      int64_t i0 = g ? g : s.period;  // paper's 1-based recent index of the first token of this type
      int64_t m = s.T - s.n;
      r.t0 = s.n + i0 - 1; r.ts = s.period; r.cnt = i0 <= m ? (m - i0) / s.period + 1 : 0;
      break;
    }
    default:
      break;
  }
  return r;
}

// ---- generic batched small GEMM on the fp32 ALUs ---------------------------------------------------
// C(m,n) = [Cin(m,n) +] Σ_k A(m,k) B(k,n), optionally zeroed above the diagonal (n > m).
// An operand element lives at  ptr + bh*s_bh + g*s_g + X0*s0 + X1*s1  where Xi is the logical
// index itself or, when the operand's tok flag for that index is set, the token it maps to.
struct SmatOperand {
  const void* ptr;
  int bf16;  // 0: float, 1: __nv_bfloat16
  int64_t s_bh, s_g, s0, s1;
  int tok0, tok1;  // 1: that logical index of this operand is a token position of the group
};

struct SmatGemmArgs {
  SmatOperand A, B, C, Cin;  // Cin.ptr == nullptr: no addend.  Cin is always float.
  int M, N, K;               // extents of the dimensions that are not token dimensions
  int tokM, tokN, tokK;      // 1: that dimension runs over the group's tokens (extent = token count)
  int tril;
  int tilesN;                // number of 64-wide column tiles launched
  SmatGroupSpec grp;
  const float* lam;          // gated variant: prefix sums of the log-gates [bh][T]; a tril tile over the tokens of a chunk
                             // is multiplied entrywise by exp(λ_m - λ_n) (null: no decay)
};

cudaError_t smat_launch_gemm(const SmatGemmArgs& a, int max_M, int max_N, int64_t groups, int bh, cudaStream_t st);

// Exclusive scan of per-chunk states in place, over up to two independent chunk ranges; reverse = suffix scan.
cudaError_t smat_launch_scan(float* S, int64_t state_elems, int64_t NC, int bh, int64_t lo0, int64_t hi0, int64_t lo1,
                             int64_t hi1, int reverse, cudaStream_t st);

// Algorithm 2 (direct form) and its transpose, one slab of state entries per CTA held in shared memory.
// transpose = 0: out[h] = Σ_{x ∈ H_h} in[x]  (in: P states, out: B states)
// transpose = 1: out[x] = Σ_{h ∋ x} in[h]   (in: B states, out: P states)
cudaError_t smat_launch_tabulate_alg2(const float* in, float* out, const SmatGeo& geo, int64_t state_elems, int bh,
                                      int transpose, cudaStream_t st);
// Largest slab (entries) the direct tabulation can hold in shared memory; 0 if none fits.
int smat_tabulate_alg2_slab(int64_t rows_in, int64_t state_elems);

cudaError_t smat_launch_mask(uint8_t* mask, const SmatGeo& geo, cudaStream_t st);

// Pooling of outer products into one fp32 state per group: state[bh][g] = Σ_{tokens of g} a_tᵀ b_t.
cudaError_t smat_launch_pool(const void* A, const void* Bm, int bf16, float* state, const SmatGroupSpec& grp,
                             int64_t Tlen, int64_t groups, int bh, int r, int p, cudaStream_t st);

// Routed read of per-group states: acc_out[t] = acc_in[t] + x_t · state[g(t)] for the tokens of every group.
cudaError_t smat_launch_state_read(const void* X, int bf16, const float* state, int transposed, const float* acc_in,
                                   float* acc_out, const SmatGroupSpec& grp, int64_t Tlen, int64_t groups, int bh,
                                   int r, int p, int* status, cudaStream_t st);

// Staged exact tabulation (same sums as Algorithm 2, one coordinate at a time). Slab = 0: not available.
int smat_tabulate_staged_slab(const SmatGeo& geo, int64_t state_elems, int transpose);
// out_bf16 = 1 writes the result table as bf16 (same layout, half the bytes) instead of fp32.
cudaError_t smat_launch_tabulate_staged(const float* in, void* out, const SmatGeo& geo, int64_t state_elems, int bh,
                                        int transpose, int out_bf16, cudaStream_t st);

// Tensor-core kernels of the causal branch (bf16, d_k = d_v = 128, 128-token tiles; n and T - n multiples of 128).
bool smat_tc_available();
// S_in[bh][tile] (bf16 [128][128]) = exclusive prefix sum of K_bᵀ V_b over the tiles of each block;
// through = 1 runs one scan over the whole sequence (d = 1), else the scan restarts at token n.
// reverse = 1 gives exclusive suffix sums instead (the scan adjoint, with K, V replaced by Q, dO).
// lam (gated variant): inclusive prefix sums of the log-gates [bh][T]; K then holds the rows rescaled to the end of
// their tile (forward order) or to its start (reverse order), and the running state decays by the tile's total gate.
cudaError_t smat_launch_chunk_scan_tc(const void* K, const void* V, void* Sin_bf16, int64_t T, int bh, int64_t n,
                                      int through, int reverse, int* status, cudaStream_t st, const float* lam = nullptr);
// Within-chunk adjoints on tensor cores (which = 0: dQ, 1: dK, 2: dV), see tile_product_tc_kernel.
cudaError_t smat_launch_chunk_adjoint_tc(int which, const void* Q, const void* K, const void* V, const void* dO,
                                         const void* Sin_bf16, const void* Dbar_bf16, const float* addend,
                                         int64_t add_lo, int64_t add_hi, void* Out, int64_t T, int bh, int* status,
                                         cudaStream_t st, int addend_bf16 = 0);
// The three adjoints of every tile in one launch (all operands of a tile loaded once, both score tiles formed once).
cudaError_t smat_launch_bwd_tiles_fused_tc(const void* Q, const void* K, const void* V, const void* dO,
                                           const void* Sin_bf16, const void* Dbar_bf16, const void* lr_q, const void* lr_k,
                                           const void* lr_v, int64_t n, void* dQ, void* dK, void* dV, int64_t T, int bh,
                                           int* status, cudaStream_t st, const float* lam = nullptr);
// O_b = Q_b S_in[b] + tril(Q_b K_bᵀ) V_b (+ ylr rows for tokens >= n_lr).
cudaError_t smat_launch_chunk_output_tc(const void* Q, const void* K, const void* V, const void* Sin_bf16,
                                        const float* ylr, int64_t n_lr, void* O, int64_t T, int bh, int* status,
                                        cudaStream_t st, const float* lam = nullptr);
// Typed read on tensor cores: ylr[t] = q_tᵀ U_type(t) for recent tokens, U kept as bf16 [bh][B][128][128].
// (transposed = 1 contracts the second state index instead: out[t] = state · x_t; grp selects types or profiles)
// (the rows go to `out` as fp32, or to `out_bf16` when that is non-null)
cudaError_t smat_launch_state_read_tc(const void* X, const void* state_bf16, float* out, void* out_bf16, int transposed,
                                      const SmatGroupSpec& grp, int64_t groups, int64_t T, int bh, int* status,
                                      cudaStream_t st);
// Both reads of the per-profile adjoint states in one launch (every state loaded once): out_t[t] = St x_t for rows Xt,
// out_n[t] = Stᵀ x_t for rows Xn; bf16 results.
cudaError_t smat_launch_state_read_dual_tc(const void* Xt, const void* Xn, const void* state_bf16, void* out_t_bf16,
                                           void* out_n_bf16, const SmatGroupSpec& grp, int64_t groups, int64_t T, int bh,
                                           int* status, cudaStream_t st);
// One step of cached decoding: S += k vᵀ, o = qᵀ (U_type + S) for every head (fp32 running state).
cudaError_t smat_launch_decode_step(const void* q, const void* k, const void* v, void* o, float* S, const void* U,
                                    int u_bf16, int in_bf16, int64_t type, int64_t types, int r, int p, int bh,
                                    cudaStream_t st, const float* log_a = nullptr, float* log_g = nullptr);
// d = 3 tabulation from a bf16 profile table on the fp32 ALUs (primes too large for the resident-matrix kernel).
int smat_tabulate_d3_bf16_slab(const SmatGeo& geo, int64_t state_elems);
cudaError_t smat_launch_tabulate_d3_bf16(const void* in, void* out, const SmatGeo& geo, int64_t state_elems, int bh,
                                         cudaStream_t st);
// The same tabulation with the sums held in registers (K slopes x q offsets per thread, every column value loaded
// once per K slopes); covers the primes it was instantiated for.
int smat_tabulate_d3_regs_supported(const SmatGeo& geo, int64_t state_elems);
cudaError_t smat_launch_tabulate_d3_regs(const void* in, void* out, const SmatGeo& geo, int64_t state_elems, int bh,
                                         int* status, cudaStream_t st);
// bf16 -> fp32 copy of a table (debug export).
// Tabulation on the tensor cores (bf16 tables; d = 3, 4 with a prime small enough for a resident Radon matrix).
int smat_tabulate_tc_supported(const SmatGeo& geo, int64_t state_elems);
int smat_tabulate_tc_layout_ok(int q);   // host-only self-check of the kernel's shared-memory map for prime q
int64_t smat_tabulate_tc_scratch_rows(const SmatGeo& geo);
int64_t smat_tabulate_tc_scratch_elems(const SmatGeo& geo, int64_t state_elems, int bh);
cudaError_t smat_launch_tabulate_tc(const void* in, void* out, void* scratch, const SmatGeo& geo, int64_t state_elems,
                                    int bh, int transpose, int* status, cudaStream_t st, int* launches);
cudaError_t smat_launch_widen_bf16(const void* src_bf16, float* dst, int64_t count, cudaStream_t st);
// Pooling on tensor cores: F[bh][x] = Σ_{t ≡ x (mod P), t < n} k_t v_tᵀ, stored as fp32 or bf16.
// slab_major = 1 (bf16 only): F is stored as [bh][rp / 32][groups][32], 32 consecutive entries of every state together.
cudaError_t smat_launch_pool_tc(const void* K, const void* V, void* F, int out_bf16, const SmatGroupSpec& grp,
                                int64_t groups, int64_t max_tokens, int64_t T, int bh, int* status, cudaStream_t st,
                                int slab_major = 0);
// bf16 table kept slab-major [bh][rp / 32][rows][32] -> fp32 [bh][rows][rp] (debug export).
cudaError_t smat_launch_widen_bf16_slabs(const void* src_bf16, float* dst, int64_t heads, int64_t rows, int64_t rp,
                                         cudaStream_t st);
// Gated variant (Sec. 3.2): prefix / suffix sums per head, rescaled copies, decayed chunk scan, gate gradient.
cudaError_t smat_launch_head_scan(const float* in, float* out, int64_t len, int bh, int reverse, cudaStream_t st);
cudaError_t smat_launch_gate_scale(const void* A, const void* B, void* out, const float* lam, int mode, int bf16,
                                   int64_t n, int64_t c, int64_t T, int dim, int bh, cudaStream_t st);
cudaError_t smat_launch_gated_scan(float* S, const float* lam, int64_t state_elems, int64_t NC, int64_t c, int bh,
                                   int64_t lo0, int64_t hi0, int64_t lo1, int64_t hi1, int reverse, cudaStream_t st);
cudaError_t smat_launch_gate_dlam(const void* Q, const void* dQ, const void* K, const void* dK, float* dlam, int bf16,
                                  int dim, int64_t T, int bh, cudaStream_t st);
// Normalised output (Sec. 2): elementwise steps around the linear pass (see smat_gated.cu).
cudaError_t smat_launch_normalize_step(int step, const void* a, const void* b, void* out, int bf16, int p, int64_t rows,
                                       cudaStream_t st);
// Token lists of user-supplied routing: prof [bh][n] (cells in [0, P)) and type [bh][m] (types in [0, B)) -> CSR lists
// (offsets [bh][G + 1], token positions [bh][count], ascending inside a group).  Keys out of range are dropped.
int64_t smat_routing_max_groups();
cudaError_t smat_launch_routing_lists(const int32_t* prof, const int32_t* type, int32_t* prof_list, int32_t* prof_offs,
                                      int32_t* type_list, int32_t* type_offs, const SmatGeo& geo, int bh,
                                      cudaStream_t st);
// Zeroes the row (row_bytes bytes at rows + (bh*T + first + i) * row_bytes) of every token i whose key lies outside [0, G).
cudaError_t smat_launch_zero_unrouted(const int32_t* key, int64_t count, int64_t G, int64_t first, void* rows, int64_t T,
                                      int row_bytes, int bh, cudaStream_t st);
// Two-level causal branch: segment totals, then (after an exclusive scan of the totals) per-segment fused output.
int smat_segment_tiles(int64_t tiles_block0, int64_t tiles_block1, int bh);
void smat_segment_counts(int64_t tiles0, int64_t tiles1, int bh, int L, int* nseg0, int* nseg1);
cudaError_t smat_launch_segment_state_tc(const void* K, const void* V, float* totals, int64_t tiles0, int64_t tiles1,
                                         int nseg0, int nseg1, int bh, int* status, cudaStream_t st);
cudaError_t smat_launch_segment_output_tc(const void* Q, const void* K, const void* V, const float* seg_in,
                                          const void* ylr_bf16, int64_t n_lr, void* O, int64_t tiles0, int64_t tiles1,
                                          int nseg0, int nseg1, int bh, int* status, cudaStream_t st,
                                          void* sin_tiles = nullptr);
