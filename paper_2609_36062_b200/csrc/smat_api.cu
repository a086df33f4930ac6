// Host side of libsmat: plan construction (geometry of Sec. 3, workspace layout) and the C entry
// points that sequence the kernels of Algorithm 1 and of the backward pass.
#include <cuda_runtime.h>

#include <cstdlib>
#include <cstring>
#include <new>

#include "../../include/smat.h"
#include "smat_internal.h"

#define SMAT_MAX_STAGES 40

struct smat_plan {
  int batch, heads, bh;
  int r, p;            // d_k, d_v
  int64_t T, c, NC;    // tokens, chunk width, chunks
  smat_dtype dtype;
  unsigned flags;
  SmatGeo geo;
  int64_t rp;          // state entries
  // workspace layout (byte offsets, 256-byte aligned)
  size_t off_status, off_sin, off_F, off_U, off_acc, off_tileA, off_W, off_fwd_end;
  size_t off_dbar, off_ubar, off_fbar, off_tileG, off_bwd_end;
  size_t off_plist, off_poffs, off_tlist, off_toffs;   // token lists of user-supplied routing (int32)
  size_t off_lr3;         // tensor-core backward: third buffer of bf16 long-range rows (the first two share off_acc)
  size_t off_sin_tiles;   // KEEP_FORWARD_TABLES on tensor-core plans: the bf16 state entering every tile, left by the forward
  size_t off_lam, off_dlam, off_gq, off_gk, off_glr, off_gdo, off_gv, off_gvlr;   // gated variant (SMAT_FLAG_GATED)
  size_t off_nv, off_ny, off_ndy;   // normalised output (SMAT_FLAG_NORMALIZED): V̄, ȳ and the upstream of the linear pass
  // Gated plans on tensor-core shapes run their FORWARD through a plan of its own (ungated flags, one state per tile)
  // whose workspace is the region at off_inner; the backward and every other shape use the fp32-ALU kernels.
  smat_plan* inner;
  size_t off_inner;
  bool tc;             // tensor-core kernels for the causal branch
  bool u_bf16;         // forward keeps the type table U in bf16 and reads it with the tensor-core typed read
  bool pool_tc;        // forward pools the profile table on the tensor cores (enough tokens per profile)
  bool f_bf16;         // the profile table is kept in bf16 (d = 2: it is the type table; tab_tc: it is an MMA operand)
  bool tab_tc;         // d = 3, 4: tabulation and its transpose on the tensor cores (bf16 tables, resident Radon matrix)
  bool tab_d3_bf16;    // d = 3 with a prime too large for that kernel: bf16 profile table, sums on the fp32 ALUs
  bool tab_d3_regs;    // ... with the sums held in registers; the profile table is then stored slab-major
  bool ubar_tc;        // backward pools the per-type adjoint states on the tensor cores
  bool ubar_bf16;      // ... and keeps them in bf16
  bool fbar_bf16;      // the per-profile adjoint states (transposed tabulation) are kept in bf16
  mutable int launches;
  mutable bool tile_states;       // the last call left one bf16 incoming state per 128-token tile at off_sin
  mutable bool kept_tile_states;  // the last forward left them at off_sin_tiles for the backward (KEEP_FORWARD_TABLES)
  mutable bool kept_gated_forward;  // the last call was the tensor-core gated forward: λ, the rescaled K copies, U and the
                                    // per-tile states are still in the workspace (used under KEEP_FORWARD_TABLES)
  // optional per-launch timing (smat_profile_enable): event k is recorded before launch k
  mutable bool profiling;
  mutable cudaEvent_t events[SMAT_MAX_STAGES + 1];
  mutable const char* stage_names[SMAT_MAX_STAGES];
  mutable int stages;
};


namespace {

bool is_prime(int64_t v) {
  if (v < 2) return false;
  for (int64_t f = 2; f * f <= v; ++f)
    if (v % f == 0) return false;
  return true;
}

// q^e >= n without overflow
bool pow_at_least(int64_t q, int e, int64_t n) {
  int64_t acc = 1;
  for (int i = 0; i < e; ++i) {
    acc *= q;
    if (acc >= n) return true;
  }
  return acc >= n;
}

size_t align_up(size_t v) { return (v + 255) & ~(size_t)255; }

smat_status build_geometry(SmatGeo* g, int64_t T, int64_t c, int d, int q_override) {
  memset(g, 0, sizeof(*g));
  g->T = T; g->c = c; g->d = d;
  g->n = c * (T / (2 * c));  // Sec. 3.1: n = c*floor(T/2c), so no chunk crosses the block boundary
  g->m = T - g->n;
  if (d == 1) {              // Sec. 3: B = 1, H_0 = F_q^0, G all ones
    g->dense_G = 1; g->q = 0; g->D = 0; g->P = 1; g->A = 1; g->B = 1; g->nnzC = 1;
    for (int k = 0; k < SMAT_MAX_D; ++k) g->qpow[k] = 1;
    return SMAT_OK;
  }
  if (g->n == 0) return SMAT_ERR_GEOMETRY;
  int64_t q = q_override;
  if (q == 0) {
    q = 2;
    while (!(is_prime(q) && pow_at_least(q, d, g->n))) ++q;
  } else if (!is_prime(q)) {
    return SMAT_ERR_GEOMETRY;
  }
  g->q = (int32_t)q; g->D = d - 1;
  int64_t acc = 1;
  for (int k = 0; k < SMAT_MAX_D; ++k) {
    g->qpow[k] = acc;
    if (k < g->D) {
      if (acc > (int64_t)1 << 40) return SMAT_ERR_GEOMETRY;
      acc *= q;
    }
  }
  g->P = g->qpow[g->D];
  g->A = (g->P - 1) / (q - 1);   // Eq. "Bcount"
  g->B = q * g->A;
  g->nnzC = g->B * g->qpow[g->D - 1];
  if (g->P > 60000 || g->B > 60000) return SMAT_ERR_GEOMETRY;  // grid.y carries the state index
  int64_t start = 0;
  for (int lead = 0; lead < g->D; ++lead) {
    g->dir_group_start[lead] = start;
    start += g->qpow[g->D - 1 - lead];
  }
  return SMAT_OK;
}

SmatOperand operand(const void* ptr, int bf16, int64_t s_bh, int64_t s_g, int64_t s0, int64_t s1, int tok0 = 0,
                    int tok1 = 0) {
  SmatOperand o; o.ptr = ptr; o.bf16 = bf16; o.s_bh = s_bh; o.s_g = s_g; o.s0 = s0; o.s1 = s1;
  o.tok0 = tok0; o.tok1 = tok1;
  return o;
}

SmatGroupSpec group(const smat_plan* pl, int mode) {
  SmatGroupSpec s; s.mode = mode; s.n = pl->geo.n; s.T = pl->T; s.c = pl->c;
  s.period = mode == SMAT_GM_PROFILE ? pl->geo.P : pl->geo.B;
  s.list = nullptr; s.offs = nullptr; s.list_stride = 0; s.offs_stride = 0;
  return s;
}

struct Ctx;
SmatGroupSpec group(const Ctx& cx, int mode);

struct Ctx {
  const smat_plan* pl;
  cudaStream_t st;
  char* ws;
  cudaError_t err;
  int launches;
  const smat_plan* rec = nullptr;   // plan whose stage timer records the launches (default: pl)
  bool routed = false;   // profile / type groups come from the token lists in the workspace, not from positions
  const int32_t* prof = nullptr;   // the caller's arrays of a routed call
  const int32_t* type = nullptr;
  float* f(size_t off) const { return reinterpret_cast<float*>(ws + off); }
};

SmatGroupSpec group(const Ctx& cx, int mode) {
  const smat_plan* pl = cx.pl;
  SmatGroupSpec s = group(pl, mode);
  if (cx.routed && mode != SMAT_GM_CHUNK) {
    const bool prof = mode == SMAT_GM_PROFILE;
    s.list = reinterpret_cast<const int32_t*>(cx.ws + (prof ? pl->off_plist : pl->off_tlist));
    s.offs = reinterpret_cast<const int32_t*>(cx.ws + (prof ? pl->off_poffs : pl->off_toffs));
    s.list_stride = prof ? pl->geo.n : pl->geo.m;
    s.offs_stride = (prof ? pl->geo.P : pl->geo.B) + 1;
  }
  return s;
}

// Every pass starts from clean device status words: the plan's own and, on gated plans whose forward runs through an
// inner plan, that plan's (smat_check_status reads both).
cudaError_t clear_status(const Ctx& cx) {
  const smat_plan* pl = cx.pl;
  pl->kept_gated_forward = false;   // whatever pass starts here may overwrite what a gated forward left behind
  cudaError_t err = cudaMemsetAsync(cx.ws + pl->off_status, 0, 256, cx.st);
  if (err == cudaSuccess && pl->inner)
    err = cudaMemsetAsync(cx.ws + pl->off_inner + pl->inner->off_status, 0, 256, cx.st);
  return err;
}

void mark_stage(const smat_plan* pl, cudaStream_t st, const char* name) {
  if (!pl->profiling || pl->stages >= SMAT_MAX_STAGES) return;
  if (pl->stages == 0) cudaEventRecord(pl->events[0], st);
  pl->stage_names[pl->stages] = name;
}
void end_stage(const smat_plan* pl, cudaStream_t st) {
  if (!pl->profiling || pl->stages >= SMAT_MAX_STAGES) return;
  ++pl->stages;
  cudaEventRecord(pl->events[pl->stages], st);
}

#define SMAT_TRY(ctx, name, call)                   \
  do {                                              \
    if ((ctx).err == cudaSuccess) {                 \
      mark_stage((ctx).rec ? (ctx).rec : (ctx).pl, (ctx).st, name);   \
      (ctx).err = (call);                           \
      end_stage((ctx).rec ? (ctx).rec : (ctx).pl, (ctx).st);          \
      ++(ctx).launches;                             \
    }                                               \
  } while (0)

int64_t max_group_tokens(const smat_plan* pl, int mode, bool routed = false) {
  const SmatGeo& g = pl->geo;
  if (routed && mode != SMAT_GM_CHUNK) {
    // Data-dependent: any size.  The kernels loop over passes of their tile height, so this is only a hint for which
    // height to instantiate: groups that hold few tokens on average get the small one (more CTAs per SM), and a heavy
    // group simply takes more passes.
    const int64_t tokens = mode == SMAT_GM_PROFILE ? g.n : g.m, groups = mode == SMAT_GM_PROFILE ? g.P : g.B;
    return 2 * tokens <= 32 * groups ? 32 : tokens;
  }
  if (mode == SMAT_GM_CHUNK) return pl->c;
  if (mode == SMAT_GM_PROFILE) return (g.n + g.P - 1) / g.P;
  return (g.m + g.B - 1) / g.B;
}
int64_t group_count(const smat_plan* pl, int mode) {
  if (mode == SMAT_GM_CHUNK) return pl->NC;
  return mode == SMAT_GM_PROFILE ? pl->geo.P : pl->geo.B;
}

// state[bh][g] (r x p, fp32) = Σ_{tokens of g} a_tᵀ b_t   with a: [T, r], b: [T, p]
void outer_sum(Ctx& cx, const char* name, int mode, const void* a, const void* b, float* state) {
  const smat_plan* pl = cx.pl;
  const int bf = pl->dtype == SMAT_BF16;
  const int64_t G = group_count(pl, mode);
  SMAT_TRY(cx, name, smat_launch_pool(a, b, bf, state, group(cx, mode), pl->T, G, pl->bh, pl->r, pl->p, cx.st));
}

// out[bh][t] (+)= x_t · state_g(t)  (transposed = 0: x: [T, r] contracts the first state index, out: [T, p];
//                                     transposed = 1: x: [T, p] contracts the second state index, out: [T, r])
// `out_final` (plan dtype) receives acc_in + product when non-null; otherwise the fp32 accumulator is updated.
void state_read(Ctx& cx, const char* name, int mode, const void* x, const float* state, int transposed, const float* acc_in,
                float* acc_out, void* out_final) {
  const smat_plan* pl = cx.pl;
  const int bf = pl->dtype == SMAT_BF16;
  const int64_t G = group_count(pl, mode);
  const int kdim = transposed ? pl->p : pl->r, odim = transposed ? pl->r : pl->p;
  if (mode != SMAT_GM_CHUNK && !out_final) {  // a handful of tokens per state: stream the state once
    SMAT_TRY(cx, name, smat_launch_state_read(x, bf, state, transposed, acc_in, acc_out, group(cx, mode), pl->T, G,
                                              pl->bh, pl->r, pl->p, reinterpret_cast<int*>(cx.ws + pl->off_status),
                                              cx.st));
    return;
  }
  SmatGemmArgs g{};
  g.A = operand(x, bf, pl->T * kdim, 0, kdim, 1, 1, 0);
  g.B = transposed ? operand(state, 0, G * pl->rp, pl->rp, 1, pl->p) : operand(state, 0, G * pl->rp, pl->rp, pl->p, 1);
  g.Cin = operand(acc_in, 0, pl->T * odim, 0, odim, 1, 1, 0);
  g.C = out_final ? operand(out_final, bf, pl->T * odim, 0, odim, 1, 1, 0)
                  : operand(acc_out, 0, pl->T * odim, 0, odim, 1, 1, 0);
  g.K = kdim; g.N = odim; g.tokM = 1; g.grp = group(cx, mode);
  SMAT_TRY(cx, name, smat_launch_gemm(g, (int)max_group_tokens(pl, mode), odim, G, pl->bh, cx.st));
}

// tile[bh][chunk] (c x c, fp32) = tril(X_b Y_bᵀ), X, Y: [T, dim]
void tril_scores(Ctx& cx, const char* name, const void* x, const void* y, int dim, float* tile, const float* lam = nullptr) {
  const smat_plan* pl = cx.pl;
  const int bf = pl->dtype == SMAT_BF16;
  SmatGemmArgs g{};
  g.A = operand(x, bf, pl->T * dim, 0, dim, 1, 1, 0);
  g.B = operand(y, bf, pl->T * dim, 0, 1, dim, 0, 1);
  g.C = operand(tile, 0, pl->NC * pl->c * pl->c, pl->c * pl->c, pl->c, 1);
  g.K = dim; g.tokM = 1; g.tokN = 1; g.tril = 1; g.grp = group(pl, SMAT_GM_CHUNK); g.lam = lam;
  SMAT_TRY(cx, name, smat_launch_gemm(g, (int)pl->c, (int)pl->c, pl->NC, pl->bh, cx.st));
}

// out[bh][t in chunk] = acc_in + tile_b(ᵀ) · Y_b     (tile c x c; Y: [T, dim])
void tile_apply(Ctx& cx, const char* name, const float* tile, int tile_transposed, const void* y, int dim, const float* acc_in,
                float* acc_out, void* out_final) {
  const smat_plan* pl = cx.pl;
  const int bf = pl->dtype == SMAT_BF16;
  const int64_t cc = pl->c * pl->c;
  SmatGemmArgs g{};
  g.A = tile_transposed ? operand(tile, 0, pl->NC * cc, cc, 1, pl->c) : operand(tile, 0, pl->NC * cc, cc, pl->c, 1);
  g.B = operand(y, bf, pl->T * dim, 0, dim, 1, 1, 0);
  g.Cin = operand(acc_in, 0, pl->T * dim, 0, dim, 1, 1, 0);
  g.C = out_final ? operand(out_final, bf, pl->T * dim, 0, dim, 1, 1, 0)
                  : operand(acc_out, 0, pl->T * dim, 0, dim, 1, 1, 0);
  g.N = dim; g.tokM = 1; g.tokK = 1; g.grp = group(pl, SMAT_GM_CHUNK);
  SMAT_TRY(cx, name, smat_launch_gemm(g, (int)pl->c, dim, pl->NC, pl->bh, cx.st));
}

void scan_states(Ctx& cx, const char* name, float* S, int reverse) {
  const smat_plan* pl = cx.pl;
  const int64_t ncd = pl->geo.n / pl->c;
  if (pl->geo.dense_G)  // d = 1: U_0 = F_0 is exactly the carry across the boundary, so the scan runs through
    SMAT_TRY(cx, name, smat_launch_scan(S, pl->rp, pl->NC, pl->bh, 0, pl->NC, 0, 0, reverse, cx.st));
  else
    SMAT_TRY(cx, name, smat_launch_scan(S, pl->rp, pl->NC, pl->bh, 0, ncd, ncd, pl->NC, reverse, cx.st));
}

smat_status check_common(const smat_plan* pl, const void* ws, size_t ws_bytes, int for_backward) {
  if (!pl || !ws) return SMAT_ERR_NULL;
  if (ws_bytes < smat_workspace_bytes(pl, for_backward)) return SMAT_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(ws) & 255) return SMAT_ERR_ALIGN;
  return SMAT_OK;
}

bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) != 0; }

// Every kernel of the library is sm_100a code: a call that would launch on another device reports it instead.
bool device_ok() {
  const bool ok = smat_tc_available();
  if (!ok) cudaGetLastError();  // a missing driver or device leaves a sticky-looking error code behind: clear it
  return ok;
}

// Step 3 of Algorithm 1 (transpose = 0) or F̄ = Cᵀ Ū (transpose = 1).
void tabulate(Ctx& cx, const char* name, const float* in, float* out, int transpose, int out_bf16 = 0) {
  const smat_plan* pl = cx.pl;
  if (in == out) return;  // d = 2: hyperplanes are single points, the type table is the profile table
  if (!(pl->flags & SMAT_FLAG_ALG2_TABULATION) && smat_tabulate_staged_slab(pl->geo, pl->rp, transpose) >= 4)
    SMAT_TRY(cx, name, smat_launch_tabulate_staged(in, out, pl->geo, pl->rp, pl->bh, transpose, out_bf16, cx.st));
  else
    SMAT_TRY(cx, name, smat_launch_tabulate_alg2(in, out, pl->geo, pl->rp, pl->bh, transpose, cx.st));
}

// The same two operations for plans whose tables are bf16: Radon stages on the tensor cores (one launch for d = 3, two for d = 4).
void tabulate_tc(Ctx& cx, const char* name, const void* in, void* out, int transpose) {
  const smat_plan* pl = cx.pl;
  int launches = 1;
  SMAT_TRY(cx, name, smat_launch_tabulate_tc(in, out, cx.ws + pl->off_W, pl->geo, pl->rp, pl->bh, transpose,
                                             reinterpret_cast<int*>(cx.ws + pl->off_status), cx.st, &launches));
  cx.launches += launches - 1;
}

// Steps 2-3 and 5-6 of Algorithm 1: the tables S_in, F, U.
void build_forward_tables(Ctx& cx, const void* K, const void* V) {
  const smat_plan* pl = cx.pl;
  if (!pl->geo.dense_G) {
    outer_sum(cx, "pool", SMAT_GM_PROFILE, K, V, cx.f(pl->off_F));                                         // step 2
    tabulate(cx, "tabulate", cx.f(pl->off_F), cx.f(pl->off_U), 0);                                 // step 3
  }
  outer_sum(cx, "chunk_state", SMAT_GM_CHUNK, K, V, cx.f(pl->off_sin));                                           // step 5
  scan_states(cx, "scan", cx.f(pl->off_sin), 0);                                                           // step 6
}

// Steps 2-3 of Algorithm 1 alone, as the plan's forward runs them: the type table U ends in the workspace at the
// returned offset (d = 1: the single state U_0 = F_0, fp32).
size_t build_type_table(Ctx& cx, const void* K, const void* V) {
  const smat_plan* pl = cx.pl;
  if (pl->geo.dense_G) {
    outer_sum(cx, "pool", SMAT_GM_PROFILE, K, V, cx.f(pl->off_sin));
    return pl->off_sin;
  }
  if (pl->tc) {
    int* status = reinterpret_cast<int*>(cx.ws + pl->off_status);
    if (pl->pool_tc)
      SMAT_TRY(cx, "pool_tc", smat_launch_pool_tc(K, V, cx.ws + pl->off_F, pl->f_bf16, group(cx, SMAT_GM_PROFILE),
                                                  pl->geo.P, max_group_tokens(pl, SMAT_GM_PROFILE, cx.routed), pl->T, pl->bh,
                                                  status, cx.st, pl->tab_d3_regs ? 1 : 0));
    else
      outer_sum(cx, "pool", SMAT_GM_PROFILE, K, V, cx.f(pl->off_F));
    if (pl->tab_tc)
      tabulate_tc(cx, "tabulate_tc", cx.ws + pl->off_F, cx.ws + pl->off_U, 0);
    else if (pl->tab_d3_regs)
      SMAT_TRY(cx, "tabulate_regs", smat_launch_tabulate_d3_regs(cx.ws + pl->off_F, cx.ws + pl->off_U, pl->geo, pl->rp,
                                                                  pl->bh, status, cx.st));
    else if (pl->tab_d3_bf16)
      SMAT_TRY(cx, "tabulate_bf16", smat_launch_tabulate_d3_bf16(cx.ws + pl->off_F, cx.ws + pl->off_U, pl->geo, pl->rp,
                                                                  pl->bh, cx.st));
    else
      tabulate(cx, "tabulate", cx.f(pl->off_F), cx.f(pl->off_U), 0, pl->u_bf16);
  } else {
    outer_sum(cx, "pool", SMAT_GM_PROFILE, K, V, cx.f(pl->off_F));
    tabulate(cx, "tabulate", cx.f(pl->off_F), cx.f(pl->off_U), 0);
  }
  return pl->off_U;
}

// The plan whose kernels build (and whose element type stores) the type table of the decode cache: a gated plan with
// a tensor-core inner plan tabulates through that one.
const smat_plan* decode_table_plan(const smat_plan* pl) {
  return (pl->flags & SMAT_FLAG_GATED) && pl->inner ? pl->inner : pl;
}
size_t decode_table_bytes(const smat_plan* pl) {
  return align_up((size_t)pl->bh * pl->geo.B * pl->rp * (decode_table_plan(pl)->u_bf16 ? 2 : 4));
}
size_t decode_state_bytes(const smat_plan* pl) { return align_up((size_t)pl->bh * pl->rp * sizeof(float)); }

}  // namespace

extern "C" {

smat_status smat_plan_create(smat_plan** out, int batch, int heads, int64_t T, int d_k, int d_v, int d, int chunk,
                             int q_override, smat_dtype dtype, unsigned flags) {
  if (!out) return SMAT_ERR_NULL;
  *out = nullptr;
  if (dtype != SMAT_F32 && dtype != SMAT_BF16) return SMAT_ERR_DTYPE;
  if (batch < 1 || heads < 1 || T < 1 || (int64_t)batch * heads > 65535) return SMAT_ERR_SHAPE;
  if ((d_k != 64 && d_k != 128) || (d_v != 64 && d_v != 128)) return SMAT_ERR_SHAPE;
  if (chunk != 16 && chunk != 32 && chunk != 64 && chunk != 128) return SMAT_ERR_SHAPE;
  if (T % chunk != 0 || T / chunk > 65535) return SMAT_ERR_SHAPE;
  if (d < 1 || d > SMAT_MAX_D || q_override < 0) return SMAT_ERR_GEOMETRY;
  smat_plan* pl = new (std::nothrow) smat_plan();
  if (!pl) return SMAT_ERR_LAUNCH;
  pl->batch = batch; pl->heads = heads; pl->bh = batch * heads;
  pl->r = d_k; pl->p = d_v; pl->T = T; pl->c = chunk; pl->NC = T / chunk;
  pl->dtype = dtype; pl->flags = flags; pl->rp = (int64_t)d_k * d_v; pl->launches = 0;
  pl->profiling = false; pl->stages = 0; pl->tile_states = false; pl->kept_tile_states = false;
  pl->kept_gated_forward = false;
  smat_status s = build_geometry(&pl->geo, T, chunk, d, q_override);
  if (s != SMAT_OK) { delete pl; return s; }
  const SmatGeo& g = pl->geo;
  // Which kernels a plan uses depends on the shape alone (no device work here); whether the current device can run
  // them is checked by the calls that launch.
  pl->tc = dtype == SMAT_BF16 && d_k == 128 && d_v == 128 && !(flags & (SMAT_FLAG_SIMT_ONLY | SMAT_FLAG_GATED)) && g.n % 128 == 0 &&
           g.m % 128 == 0 && g.n >= 128;
  if (!g.dense_G && (smat_tabulate_alg2_slab(g.B, pl->rp) < 1)) { delete pl; return SMAT_ERR_UNSUPPORTED; }
  // d >= 3 on the tensor-core path: U is only ever a bf16 MMA operand, so it is stored as bf16 (half the bytes)
  pl->tab_tc = pl->tc && !g.dense_G && !(flags & (SMAT_FLAG_ALG2_TABULATION | SMAT_FLAG_ALU_TABULATION)) &&
               smat_tabulate_tc_supported(g, pl->rp);
  pl->tab_d3_bf16 = pl->tc && g.D == 2 && !pl->tab_tc &&
                    !(flags & (SMAT_FLAG_ALG2_TABULATION | SMAT_FLAG_ALU_TABULATION)) &&
                    smat_tabulate_d3_bf16_slab(g, pl->rp) > 0;
  pl->tab_d3_regs = pl->tab_d3_bf16 && smat_tabulate_d3_regs_supported(g, pl->rp) && !(flags & SMAT_FLAG_D3_SHARED_SUMS);
  pl->pool_tc = pl->tc && !g.dense_G && (g.n / g.P >= 12 || pl->tab_tc || pl->tab_d3_bf16);
  pl->f_bf16 = pl->pool_tc && ((g.D == 1 && !(flags & SMAT_FLAG_ALG2_TABULATION)) || pl->tab_tc || pl->tab_d3_bf16);
  pl->u_bf16 = pl->f_bf16 || (pl->tc && g.D >= 2 && !(flags & SMAT_FLAG_ALG2_TABULATION) &&
                              smat_tabulate_staged_slab(g, pl->rp, 0) >= 4);
  // adjoint tables of the backward pass
  // F̄ readable by the tensor-core routed read: d = 2 (it is Ū), d = 3 when the staged transposed sums can write bf16
  const bool fbar_by_read = pl->u_bf16 && (g.D == 1 || (g.D == 2 && !(flags & SMAT_FLAG_ALG2_TABULATION) &&
                                                        smat_tabulate_staged_slab(g, pl->rp, 1) >= 4));
  pl->ubar_tc = pl->tc && !g.dense_G && (pl->tab_tc || g.m / g.B >= 12);
  pl->ubar_bf16 = pl->ubar_tc && ((g.D == 1 && fbar_by_read) || pl->tab_tc);   // d = 2: F̄ is Ū itself
  pl->fbar_bf16 = pl->tc && !g.dense_G && (pl->tab_tc || (g.D == 1 ? pl->ubar_bf16 : fbar_by_read));
  // Workspace regions, each sized for the element type the plan stores there.  Tensor-core plans keep the causal
  // states per 128-token tile in bf16 (or, in the two-level form, fewer fp32 segment states in the same region) and
  // have no score-tile buffers; the fp32-ALU plans keep one fp32 state per chunk and two fp32 score-tile buffers.
  const size_t entries = (size_t)pl->rp;
  const int wide = d_k > d_v ? d_k : d_v;
  const size_t causal = pl->tc ? (size_t)pl->bh * (T / 128) * entries * 2 : (size_t)pl->bh * pl->NC * entries * 4;
  const size_t tiles = pl->tc ? 0 : (size_t)pl->bh * T * chunk * sizeof(float);
  size_t off = 0;
  pl->off_status = off; off = align_up(off + 256);
  pl->off_sin = off;    off = align_up(off + causal);
  // d = 2: C is the identity (U_h = F_h), so the two tables share storage unless Algorithm 2 is forced
  const bool alias = g.D == 1 && !(flags & SMAT_FLAG_ALG2_TABULATION);
  pl->off_F = off;      off = align_up(off + (g.dense_G || alias ? 0 : (size_t)pl->bh * g.P * entries * (pl->f_bf16 ? 2 : 4)));
  pl->off_U = off;      off = align_up(off + (g.dense_G ? 0 : (size_t)pl->bh * g.B * entries * (pl->u_bf16 ? 2 : 4)));
  pl->off_acc = off;    off = align_up(off + (size_t)pl->bh * T * wide * sizeof(float));
  pl->off_tileA = off;  off = align_up(off + tiles);
  pl->off_W = off;      off = align_up(off + (pl->tab_tc ? (size_t)smat_tabulate_tc_scratch_elems(g, pl->rp, pl->bh) * 2 : 0));
  pl->off_sin_tiles = off;
  off = align_up(off + (pl->tc && (flags & SMAT_FLAG_KEEP_FORWARD_TABLES) ? (size_t)pl->bh * (T / 128) * entries * 2 : 0));
  const bool lists = !g.dense_G;
  pl->off_plist = off;  off = align_up(off + (lists ? (size_t)pl->bh * g.n * 4 : 0));
  pl->off_poffs = off;  off = align_up(off + (lists ? (size_t)pl->bh * (g.P + 1) * 4 : 0));
  pl->off_tlist = off;  off = align_up(off + (lists ? (size_t)pl->bh * g.m * 4 : 0));
  pl->off_toffs = off;  off = align_up(off + (lists ? (size_t)pl->bh * (g.B + 1) * 4 : 0));
  // gated variant: λ and the rescaled copies of Q, K (forward) and dO, V (backward), in the plan's dtype
  const size_t esz = dtype == SMAT_BF16 ? 2 : 4;
  const size_t gated = (flags & SMAT_FLAG_GATED) ? 1 : 0;
  pl->off_lam = off;    off = align_up(off + gated * (size_t)pl->bh * T * 4);
  pl->off_gq = off;     off = align_up(off + gated * (size_t)pl->bh * T * d_k * esz);
  pl->off_gk = off;     off = align_up(off + gated * (size_t)pl->bh * T * d_k * esz);
  pl->off_glr = off;    off = align_up(off + gated * (size_t)pl->bh * T * d_k * esz);
  const size_t normd = (flags & SMAT_FLAG_NORMALIZED) ? 1 : 0;
  pl->off_nv = off;     off = align_up(off + normd * (size_t)pl->bh * T * d_v * esz);
  pl->off_ny = off;     off = align_up(off + normd * (size_t)pl->bh * T * d_v * esz);
  pl->inner = nullptr;
  pl->off_inner = off;
  if ((flags & SMAT_FLAG_GATED) && !(flags & SMAT_FLAG_SIMT_ONLY) && dtype == SMAT_BF16 && d_k == 128 && d_v == 128) {
    smat_plan* in = nullptr;
    const unsigned keep = SMAT_FLAG_ALG2_TABULATION | SMAT_FLAG_ALU_TABULATION | SMAT_FLAG_D3_SHARED_SUMS;
    if (smat_plan_create(&in, batch, heads, T, d_k, d_v, d, chunk, q_override, dtype,
                         (flags & keep) | SMAT_FLAG_PER_TILE_STATES) == SMAT_OK && in->tc) {
      pl->inner = in;
      off = align_up(off + in->off_bwd_end);   // the gated backward runs through the same inner plan
    } else if (in) {
      smat_plan_destroy(in);
    }
  }
  pl->off_fwd_end = off;
  pl->off_lr3 = off;    off = align_up(off + (pl->tc ? (size_t)pl->bh * T * 128 * 2 : 0));
  pl->off_ndy = off;    off = align_up(off + normd * (size_t)pl->bh * T * d_v * esz);
  pl->off_dlam = off;   off = align_up(off + gated * (size_t)pl->bh * T * 4);
  pl->off_gdo = off;    off = align_up(off + gated * (size_t)pl->bh * T * d_v * esz);
  pl->off_gv = off;     off = align_up(off + gated * (size_t)pl->bh * T * d_v * esz);
  pl->off_gvlr = off;   off = align_up(off + gated * (size_t)pl->bh * T * d_v * esz);
  pl->off_dbar = off;   off = align_up(off + causal);
  pl->off_ubar = off;   off = align_up(off + (g.dense_G || alias ? 0 : (size_t)pl->bh * g.B * entries * (pl->ubar_bf16 ? 2 : 4)));
  pl->off_fbar = off;   off = align_up(off + (g.dense_G ? 0 : (size_t)pl->bh * g.P * entries * (pl->fbar_bf16 ? 2 : 4)));
  pl->off_tileG = off;  off = align_up(off + tiles);
  pl->off_bwd_end = off;
  *out = pl;
  return SMAT_OK;
}

void smat_plan_destroy(smat_plan* plan) {
  if (plan && plan->profiling) smat_profile_enable(plan, 0);
  if (plan && plan->inner) smat_plan_destroy(plan->inner);
  delete plan;
}

smat_status smat_profile_enable(smat_plan* pl, int enable) {
  if (!pl) return SMAT_ERR_NULL;
  if ((enable != 0) == pl->profiling) return SMAT_OK;
  if (enable) {
    for (int i = 0; i <= SMAT_MAX_STAGES; ++i)
      if (cudaEventCreate(&pl->events[i]) != cudaSuccess) return SMAT_ERR_LAUNCH;
    pl->profiling = true;
  } else {
    for (int i = 0; i <= SMAT_MAX_STAGES; ++i) cudaEventDestroy(pl->events[i]);
    pl->profiling = false;
  }
  pl->stages = 0;
  return SMAT_OK;
}

int smat_profile_read(const smat_plan* pl, const char** names, float* ms, int max_stages) {
  if (!pl || !pl->profiling || pl->stages == 0) return 0;
  if (cudaEventSynchronize(pl->events[pl->stages]) != cudaSuccess) return 0;
  int count = pl->stages < max_stages ? pl->stages : max_stages;
  for (int i = 0; i < count; ++i) {
    float t = 0.f;
    cudaEventElapsedTime(&t, pl->events[i], pl->events[i + 1]);
    if (ms) ms[i] = t;
    if (names) names[i] = pl->stage_names[i];
  }
  return count;
}

smat_status smat_get_geometry(const smat_plan* pl, smat_geometry* out) {
  if (!pl || !out) return SMAT_ERR_NULL;
  const SmatGeo& g = pl->geo;
  out->T = g.T; out->c = g.c; out->n = g.n; out->m = g.m; out->d = g.d; out->q = g.q;
  out->P = g.P; out->A = g.A; out->B = g.B; out->nnzC = g.nnzC;
  out->vc_conditions_met = g.dense_G ? 1 : (g.P <= g.n && 2 * g.B <= g.m);
  return SMAT_OK;
}

int smat_uses_tensor_cores(const smat_plan* pl) { return pl && pl->tc ? 1 : 0; }

int smat_gated_forward_uses_tensor_cores(const smat_plan* pl) { return pl && pl->inner ? 1 : 0; }

int smat_gated_backward_uses_tensor_cores(const smat_plan* pl) {
  return pl && pl->inner && (pl->geo.dense_G || (pl->inner->u_bf16 && pl->inner->fbar_bf16)) ? 1 : 0;
}

int smat_type_table_element_bytes(const smat_plan* pl) { return pl && pl->u_bf16 ? 2 : 4; }

int smat_profile_table_element_bytes(const smat_plan* pl) { return pl && pl->f_bf16 ? 2 : 4; }

size_t smat_workspace_bytes(const smat_plan* pl, int for_backward) {
  if (!pl) return 0;
  return for_backward ? pl->off_bwd_end : pl->off_fwd_end;
}

}  // extern "C"

namespace {

// Builds the token lists of a routed call in the workspace (or does nothing for a positional call).
smat_status begin_routing(Ctx& cx, const int32_t* prof, const int32_t* type) {
  const smat_plan* pl = cx.pl;
  if (!prof && !type) return SMAT_OK;
  if (!prof || !type) return SMAT_ERR_NULL;
  if (pl->geo.dense_G) return SMAT_OK;   // d = 1: one cell, one type; there is nothing to route
  if ((reinterpret_cast<uintptr_t>(prof) | reinterpret_cast<uintptr_t>(type)) & 3) return SMAT_ERR_ALIGN;
  const int64_t gmax = pl->geo.P > pl->geo.B ? pl->geo.P : pl->geo.B;
  if (gmax > smat_routing_max_groups()) return SMAT_ERR_UNSUPPORTED;
  auto i32 = [&](size_t off) { return reinterpret_cast<int32_t*>(cx.ws + off); };
  SMAT_TRY(cx, "routing_lists", smat_launch_routing_lists(prof, type, i32(pl->off_plist), i32(pl->off_poffs),
                                                          i32(pl->off_tlist), i32(pl->off_toffs), pl->geo, pl->bh, cx.st));
  cx.routed = true;
  cx.prof = prof; cx.type = type;
  return SMAT_OK;
}

// Routed calls on the tensor-core path: the rows a routed read does not visit (tokens of no group) must read as zero
// for the kernel that adds them.
void zero_unrouted(Ctx& cx, int mode, void* rows, int row_bytes) {
  if (!cx.routed) return;
  const smat_plan* pl = cx.pl;
  const bool prof = mode == SMAT_GM_PROFILE;
  SMAT_TRY(cx, "zero_unrouted", smat_launch_zero_unrouted(prof ? cx.prof : cx.type, prof ? pl->geo.n : pl->geo.m,
                                                           prof ? pl->geo.P : pl->geo.B, prof ? 0 : pl->geo.n, rows, pl->T,
                                                           row_bytes, pl->bh, cx.st));
}

smat_status forward_impl(const smat_plan* pl, const void* Q, const void* K, const void* V, void* O, const int32_t* prof,
                         const int32_t* type, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!Q || !K || !V || !O) return SMAT_ERR_NULL;
  smat_status s = check_common(pl, workspace, workspace_bytes, 0);
  if (s != SMAT_OK) return s;
  if (misaligned(Q) || misaligned(K) || misaligned(V) || misaligned(O)) return SMAT_ERR_ALIGN;
  if (!device_ok()) return SMAT_ERR_ARCH;
  Ctx cx{pl, static_cast<cudaStream_t>(cuda_stream), static_cast<char*>(workspace), cudaSuccess, 0};
  pl->stages = 0;
  cx.err = clear_status(cx);
  s = begin_routing(cx, prof, type);
  if (s != SMAT_OK) return s;
  if (pl->tc) {
    int* status = reinterpret_cast<int*>(cx.ws + pl->off_status);
    float* ylr = cx.f(pl->off_acc);
    const bool lr = !pl->geo.dense_G;
    if (lr) build_type_table(cx, K, V);                                                      // steps 2-3
    // The two-level causal branch takes the long-range rows as bf16 (half the bytes for the typed read to write and
    // for the output kernel to fetch); plans whose type table is fp32 use the per-tile form.
    const int64_t tiles0 = lr ? pl->geo.n / 128 : pl->T / 128, tiles1 = lr ? pl->geo.m / 128 : 0;
    const int L = ((pl->flags & SMAT_FLAG_PER_TILE_STATES) || (lr && !pl->u_bf16)) ? 1 : smat_segment_tiles(tiles0, tiles1, pl->bh);
    if (lr) {                                                                                // step 4
      zero_unrouted(cx, SMAT_GM_TYPE, ylr, L >= 2 && pl->u_bf16 ? 256 : 512);
      if (pl->u_bf16)
        SMAT_TRY(cx, "read_type_tc", smat_launch_state_read_tc(Q, cx.ws + pl->off_U, ylr, L >= 2 ? ylr : nullptr, 0,
                                                               group(cx, SMAT_GM_TYPE), pl->geo.B, pl->T, pl->bh, status,
                                                               cx.st));
      else
        state_read(cx, "read_type", SMAT_GM_TYPE, Q, cx.f(pl->off_U), 0, nullptr, ylr, nullptr);
    }
    pl->tile_states = L < 2;
    pl->kept_tile_states = false;
    if (L >= 2) {  // steps 5-7, two-level: segment totals, scan of the totals, fused per-segment output
      float* seg = cx.f(pl->off_sin);
      int nseg0 = 0, nseg1 = 0;
      smat_segment_counts(tiles0, tiles1, pl->bh, L, &nseg0, &nseg1);
      const int64_t nseg = nseg0 + nseg1;
      SMAT_TRY(cx, "segment_state_tc", smat_launch_segment_state_tc(K, V, seg, tiles0, tiles1, nseg0, nseg1, pl->bh, status, cx.st));
      SMAT_TRY(cx, "segment_scan", smat_launch_scan(seg, pl->rp, nseg, pl->bh, 0, nseg0, nseg0, nseg, 0, cx.st));
      const bool keep = (pl->flags & SMAT_FLAG_KEEP_FORWARD_TABLES) != 0;   // a backward will want the per-tile states
      SMAT_TRY(cx, "segment_output_tc", smat_launch_segment_output_tc(Q, K, V, seg, ylr, lr ? pl->geo.n : pl->T, O,
                                                                       tiles0, tiles1, nseg0, nseg1, pl->bh, status, cx.st,
                                                                       keep ? cx.ws + pl->off_sin_tiles : nullptr));
      pl->kept_tile_states = keep;
    } else {
      SMAT_TRY(cx, "chunk_scan_tc", smat_launch_chunk_scan_tc(K, V, cx.ws + pl->off_sin, pl->T, pl->bh, pl->geo.n,
                                                               lr ? 0 : 1, 0, status, cx.st));   // steps 5-6
      SMAT_TRY(cx, "chunk_output_tc", smat_launch_chunk_output_tc(Q, K, V, cx.ws + pl->off_sin, ylr,
                                                                   lr ? pl->geo.n : pl->T, O, pl->T, pl->bh, status,
                                                                   cx.st));                   // step 7
    }
    pl->launches = cx.launches;
    return cx.err == cudaSuccess ? SMAT_OK : SMAT_ERR_LAUNCH;
  }
  build_forward_tables(cx, K, V);
  float* acc = cx.f(pl->off_acc);
  float* tileA = cx.f(pl->off_tileA);
  tril_scores(cx, "scores", Q, K, pl->r, tileA);                           // within-chunk scores, Eq. "local"
  state_read(cx, "read_chunk", SMAT_GM_CHUNK, Q, cx.f(pl->off_sin), 0, nullptr, acc, nullptr);  // earlier chunks
  if (!pl->geo.dense_G)                                                    // step 4: typed read, rows in place
    state_read(cx, "read_type", SMAT_GM_TYPE, Q, cx.f(pl->off_U), 0, acc, acc, nullptr);
  tile_apply(cx, "output", tileA, 0, V, pl->p, acc, nullptr, O);                     // step 7
  pl->launches = cx.launches;
  return cx.err == cudaSuccess ? SMAT_OK : SMAT_ERR_LAUNCH;
}

smat_status backward_impl(const smat_plan* pl, const void* Q, const void* K, const void* V, const void* dO, void* dQ,
                          void* dK, void* dV, const int32_t* prof, const int32_t* type, void* workspace,
                          size_t workspace_bytes, void* cuda_stream) {
  if (!Q || !K || !V || !dO || !dQ || !dK || !dV) return SMAT_ERR_NULL;
  smat_status s = check_common(pl, workspace, workspace_bytes, 1);
  if (s != SMAT_OK) return s;
  if (misaligned(Q) || misaligned(K) || misaligned(V) || misaligned(dO) || misaligned(dQ) || misaligned(dK) ||
      misaligned(dV))
    return SMAT_ERR_ALIGN;
  if (!device_ok()) return SMAT_ERR_ARCH;
  Ctx cx{pl, static_cast<cudaStream_t>(cuda_stream), static_cast<char*>(workspace), cudaSuccess, 0};
  pl->stages = 0;
  cx.err = clear_status(cx);
  s = begin_routing(cx, prof, type);
  if (s != SMAT_OK) return s;
  const bool lr = !pl->geo.dense_G;
  if (pl->tc) {
    // Tensor-core backward.  Forward tables are rebuilt as in smat_forward (U in bf16 where the plan keeps it so);
    // the per-tile states S_in and D̄ are bf16 tiles; the long-range contributions go through one fp32 buffer
    // that each within-chunk adjoint adds to its rows.
    int* status = reinterpret_cast<int*>(cx.ws + pl->off_status);
    float* lrbuf = cx.f(pl->off_acc);
    // With KEEP_FORWARD_TABLES the preceding forward has left the state entering every tile: no second scan of K, V
    const bool kept = (pl->flags & SMAT_FLAG_KEEP_FORWARD_TABLES) && pl->kept_tile_states;
    void* sin_tiles = cx.ws + (kept ? pl->off_sin_tiles : pl->off_sin);
    pl->tile_states = !kept;
    const SmatGroupSpec types = group(cx, SMAT_GM_TYPE), profs = group(cx, SMAT_GM_PROFILE);
    const int64_t n = pl->geo.n;
    if (lr) {
      if (!(pl->flags & SMAT_FLAG_KEEP_FORWARD_TABLES)) build_type_table(cx, K, V);
      // Ū_h = Σ q dOᵀ over the type (Eq. "lr-adjoint"), then F̄ = Cᵀ Ū
      const bool ubar_tc = pl->ubar_tc, ubar_bf16 = pl->ubar_bf16;
      if (ubar_tc)
        SMAT_TRY(cx, "bwd_pool_type_tc", smat_launch_pool_tc(Q, dO, cx.ws + pl->off_ubar, ubar_bf16, types, pl->geo.B,
                                                             max_group_tokens(pl, SMAT_GM_TYPE, cx.routed), pl->T, pl->bh,
                                                             status, cx.st));
      else
        outer_sum(cx, "bwd_pool_type", SMAT_GM_TYPE, Q, dO, cx.f(pl->off_ubar));
      const bool fbar_is_bf16 = pl->fbar_bf16;
      if (pl->tab_tc)
        tabulate_tc(cx, "bwd_tabulate_t_tc", cx.ws + pl->off_ubar, cx.ws + pl->off_fbar, 1);
      else
        tabulate(cx, "bwd_tabulate_t", cx.f(pl->off_ubar), cx.f(pl->off_fbar), 1, pl->geo.D == 2 && pl->fbar_bf16);
      // per-tile states
      if (!kept)
        SMAT_TRY(cx, "bwd_state_scan_tc", smat_launch_chunk_scan_tc(K, V, sin_tiles, pl->T, pl->bh, n, 0, 0, status, cx.st));
      SMAT_TRY(cx, "bwd_suffix_scan_tc", smat_launch_chunk_scan_tc(Q, dO, cx.ws + pl->off_dbar, pl->T, pl->bh, n, 0, 1, status, cx.st));
      if (pl->u_bf16 && fbar_is_bf16 && !(pl->flags & SMAT_FLAG_SEPARATE_TILE_ADJOINTS)) {
        // All three long-range terms come from the tensor-core read as bf16 rows: one buffer each, then ONE kernel for
        // the three within-chunk adjoints (every operand of a tile loaded once, both score tiles formed once).
        char* lr_q = cx.ws + pl->off_acc;
        char* lr_k = lr_q + (size_t)pl->bh * pl->T * 128 * 2;
        char* lr_v = cx.ws + pl->off_lr3;
        zero_unrouted(cx, SMAT_GM_TYPE, lr_q, 256);
        SMAT_TRY(cx, "bwd_dq_type_tc", smat_launch_state_read_tc(dO, cx.ws + pl->off_U, nullptr, lr_q, 1, types, pl->geo.B,
                                                                 pl->T, pl->bh, status, cx.st));
        zero_unrouted(cx, SMAT_GM_PROFILE, lr_k, 256);
        zero_unrouted(cx, SMAT_GM_PROFILE, lr_v, 256);
        // dK's and dV's long-range rows read the same state F̄_x: one launch, every state loaded once
        SMAT_TRY(cx, "bwd_dkdv_profile_tc", smat_launch_state_read_dual_tc(V, K, cx.ws + pl->off_fbar, lr_k, lr_v, profs,
                                                                            pl->geo.P, pl->T, pl->bh, status, cx.st));
        SMAT_TRY(cx, "bwd_tiles_fused_tc", smat_launch_bwd_tiles_fused_tc(Q, K, V, dO, sin_tiles, cx.ws + pl->off_dbar, lr_q,
                                                                           lr_k, lr_v, n, dQ, dK, dV, pl->T, pl->bh, status,
                                                                           cx.st));
        pl->launches = cx.launches;
        return cx.err == cudaSuccess ? SMAT_OK : SMAT_ERR_LAUNCH;
      }
      // dQ: recent rows add U_type dO
      // (the rows travel as bf16 where the tensor-core read writes them: rounded once, added in fp32 by the tile kernel)
      zero_unrouted(cx, SMAT_GM_TYPE, lrbuf, pl->u_bf16 ? 256 : 512);
      if (pl->u_bf16)
        SMAT_TRY(cx, "bwd_dq_type_tc", smat_launch_state_read_tc(dO, cx.ws + pl->off_U, lrbuf, lrbuf, 1, types, pl->geo.B,
                                                                 pl->T, pl->bh, status, cx.st));
      else
        state_read(cx, "bwd_dq_type", SMAT_GM_TYPE, dO, cx.f(pl->off_U), 1, nullptr, lrbuf, nullptr);
      SMAT_TRY(cx, "bwd_dq_tile_tc", smat_launch_chunk_adjoint_tc(0, Q, K, V, dO, sin_tiles, cx.ws + pl->off_dbar,
                                                                  lrbuf, n, pl->T, dQ, pl->T, pl->bh, status, cx.st,
                                                                  pl->u_bf16 ? 1 : 0));
      // dK: distant rows add F̄_prof v
      zero_unrouted(cx, SMAT_GM_PROFILE, lrbuf, fbar_is_bf16 ? 256 : 512);
      if (fbar_is_bf16)
        SMAT_TRY(cx, "bwd_dk_profile_tc", smat_launch_state_read_tc(V, cx.ws + pl->off_fbar, lrbuf, lrbuf, 1, profs, pl->geo.P,
                                                                    pl->T, pl->bh, status, cx.st));
      else
        state_read(cx, "bwd_dk_profile", SMAT_GM_PROFILE, V, cx.f(pl->off_fbar), 1, nullptr, lrbuf, nullptr);
      SMAT_TRY(cx, "bwd_dk_tile_tc", smat_launch_chunk_adjoint_tc(1, Q, K, V, dO, sin_tiles, cx.ws + pl->off_dbar,
                                                                  lrbuf, 0, n, dK, pl->T, pl->bh, status, cx.st,
                                                                  fbar_is_bf16 ? 1 : 0));
      // dV: distant rows add F̄_profᵀ k
      zero_unrouted(cx, SMAT_GM_PROFILE, lrbuf, fbar_is_bf16 ? 256 : 512);
      if (fbar_is_bf16)
        SMAT_TRY(cx, "bwd_dv_profile_tc", smat_launch_state_read_tc(K, cx.ws + pl->off_fbar, lrbuf, lrbuf, 0, profs, pl->geo.P,
                                                                    pl->T, pl->bh, status, cx.st));
      else
        state_read(cx, "bwd_dv_profile", SMAT_GM_PROFILE, K, cx.f(pl->off_fbar), 0, nullptr, lrbuf, nullptr);
      SMAT_TRY(cx, "bwd_dv_tile_tc", smat_launch_chunk_adjoint_tc(2, Q, K, V, dO, sin_tiles, cx.ws + pl->off_dbar,
                                                                  lrbuf, 0, n, dV, pl->T, pl->bh, status, cx.st,
                                                                  fbar_is_bf16 ? 1 : 0));
    } else {
      if (!kept)
        SMAT_TRY(cx, "bwd_state_scan_tc", smat_launch_chunk_scan_tc(K, V, sin_tiles, pl->T, pl->bh, n, 1, 0, status, cx.st));
      SMAT_TRY(cx, "bwd_suffix_scan_tc", smat_launch_chunk_scan_tc(Q, dO, cx.ws + pl->off_dbar, pl->T, pl->bh, n, 1, 1, status, cx.st));
      if (!(pl->flags & SMAT_FLAG_SEPARATE_TILE_ADJOINTS)) {
        SMAT_TRY(cx, "bwd_tiles_fused_tc", smat_launch_bwd_tiles_fused_tc(Q, K, V, dO, sin_tiles, cx.ws + pl->off_dbar, nullptr,
                                                                           nullptr, nullptr, pl->T, dQ, dK, dV, pl->T, pl->bh,
                                                                           status, cx.st));
        pl->launches = cx.launches;
        return cx.err == cudaSuccess ? SMAT_OK : SMAT_ERR_LAUNCH;
      }
      for (int which = 0; which < 3; ++which)
        SMAT_TRY(cx, which == 0 ? "bwd_dq_tile_tc" : (which == 1 ? "bwd_dk_tile_tc" : "bwd_dv_tile_tc"),
                 smat_launch_chunk_adjoint_tc(which, Q, K, V, dO, sin_tiles, cx.ws + pl->off_dbar, lrbuf, 0, 0,
                                              which == 0 ? dQ : (which == 1 ? dK : dV), pl->T, pl->bh, status, cx.st));
    }
    pl->launches = cx.launches;
    return cx.err == cudaSuccess ? SMAT_OK : SMAT_ERR_LAUNCH;
  }
  build_forward_tables(cx, K, V);
  float* sin = cx.f(pl->off_sin);
  float* dbar = cx.f(pl->off_dbar);
  float* acc = cx.f(pl->off_acc);
  float* tileA = cx.f(pl->off_tileA);
  float* tileG = cx.f(pl->off_tileG);
  // S̄_in_b = Q_bᵀ dO_b, then D̄ = exclusive suffix scan (scan adjoint)
  outer_sum(cx, "bwd_chunk_state", SMAT_GM_CHUNK, Q, dO, dbar);
  scan_states(cx, "bwd_scan", dbar, 1);
  // long-range adjoints: Ū_h = Σ q dOᵀ over the type, F̄ = Cᵀ Ū   (Eq. "lr-adjoint")
  if (lr) {
    outer_sum(cx, "bwd_pool_type", SMAT_GM_TYPE, Q, dO, cx.f(pl->off_ubar));
    tabulate(cx, "bwd_tabulate_t", cx.f(pl->off_ubar), cx.f(pl->off_fbar), 1);
  }
  tril_scores(cx, "bwd_scores_qk", Q, K, pl->r, tileA);    // A = tril(Q Kᵀ)
  tril_scores(cx, "bwd_scores_gv", dO, V, pl->p, tileG);   // tril(dO Vᵀ)
  // dQ = dO S_inᵀ + U_type dO (recent) + tril(dO Vᵀ) K                      (Eq. "local-adjoint", Eq. "lr-adjoint")
  state_read(cx, "bwd_dq_chunk", SMAT_GM_CHUNK, dO, sin, 1, nullptr, acc, nullptr);
  if (lr) state_read(cx, "bwd_dq_type", SMAT_GM_TYPE, dO, cx.f(pl->off_U), 1, acc, acc, nullptr);
  tile_apply(cx, "bwd_dq_tile", tileG, 0, K, pl->r, acc, nullptr, dQ);
  // dK = tril(dO Vᵀ)ᵀ Q + F̄_prof v (distant) + D̄ v
  tile_apply(cx, "bwd_dk_tile", tileG, 1, Q, pl->r, nullptr, acc, nullptr);
  if (lr) state_read(cx, "bwd_dk_profile", SMAT_GM_PROFILE, V, cx.f(pl->off_fbar), 1, acc, acc, nullptr);
  state_read(cx, "bwd_dk_chunk", SMAT_GM_CHUNK, V, dbar, 1, acc, nullptr, dK);
  // dV = Aᵀ dO + F̄_profᵀ k (distant) + D̄ᵀ k
  tile_apply(cx, "bwd_dv_tile", tileA, 1, dO, pl->p, nullptr, acc, nullptr);
  if (lr) state_read(cx, "bwd_dv_profile", SMAT_GM_PROFILE, K, cx.f(pl->off_fbar), 0, acc, acc, nullptr);
  state_read(cx, "bwd_dv_chunk", SMAT_GM_CHUNK, K, dbar, 0, acc, nullptr, dV);
  pl->launches = cx.launches;
  return cx.err == cudaSuccess ? SMAT_OK : SMAT_ERR_LAUNCH;
}

// ---- scalar-gated variant (Sec. 3.2, Eq. "gated"; Lemma "Gated SMat") on the fp32-ALU kernels ------------------------
struct Gated {
  float* lam;
  void *qc, *kc, *lr, *doc, *vc, *vlr;
};

Gated gated_buffers(const Ctx& cx) {
  const smat_plan* pl = cx.pl;
  return Gated{cx.f(pl->off_lam), cx.ws + pl->off_gq, cx.ws + pl->off_gk, cx.ws + pl->off_glr,
               cx.ws + pl->off_gdo, cx.ws + pl->off_gv, cx.ws + pl->off_gvlr};
}

void gate_scale(Ctx& cx, const char* name, const void* a, const void* b, void* out, const float* lam, int mode, int dim) {
  const smat_plan* pl = cx.pl;
  SMAT_TRY(cx, name, smat_launch_gate_scale(a, b, out, lam, mode, pl->dtype == SMAT_BF16, pl->geo.n, pl->c, pl->T, dim,
                                            pl->bh, cx.st));
}

void gated_scan(Ctx& cx, const char* name, float* S, const float* lam, int reverse) {
  const smat_plan* pl = cx.pl;
  const int64_t ncd = pl->geo.n / pl->c;
  if (pl->geo.dense_G)   // d = 1: one causal block; the carried state crosses the boundary (it is U_0 decayed)
    SMAT_TRY(cx, name, smat_launch_gated_scan(S, lam, pl->rp, pl->NC, pl->c, pl->bh, 0, pl->NC, 0, 0, reverse, cx.st));
  else
    SMAT_TRY(cx, name, smat_launch_gated_scan(S, lam, pl->rp, pl->NC, pl->c, pl->bh, 0, ncd, ncd, pl->NC, reverse, cx.st));
}

// λ, the rescaled inputs and the forward tables (S_in, F, U) of the gated pass.
void gated_forward_tables(Ctx& cx, const Gated& gt, const void* Q, const void* K, const void* V, const float* log_a) {
  const smat_plan* pl = cx.pl;
  SMAT_TRY(cx, "gate_prefix", smat_launch_head_scan(log_a, gt.lam, pl->T, pl->bh, 0, cx.st));
  gate_scale(cx, "gate_scale_q", Q, nullptr, gt.qc, gt.lam, 0, pl->r);       // exp(λ_i - λ_{e(b-1)}) q_i
  gate_scale(cx, "gate_scale_k", K, nullptr, gt.kc, gt.lam, 1, pl->r);       // exp(λ_{e(b)} - λ_j) k_j
  if (!pl->geo.dense_G) {
    gate_scale(cx, "gate_scale_lr", K, Q, gt.lr, gt.lam, 2, pl->r);          // keys and queries split at the boundary
    outer_sum(cx, "pool", SMAT_GM_PROFILE, gt.lr, V, cx.f(pl->off_F));
    tabulate(cx, "tabulate", cx.f(pl->off_F), cx.f(pl->off_U), 0);
  }
  outer_sum(cx, "chunk_state", SMAT_GM_CHUNK, gt.kc, V, cx.f(pl->off_sin));
  gated_scan(cx, "gated_scan", cx.f(pl->off_sin), gt.lam, 0);
}

// Gated forward on the tensor cores (bf16, d_k = d_v = 128, blocks of whole 128-token tiles).  The long-range part is
// the ungated pipeline on the boundary-rescaled keys and queries; the causal part carries one state per tile: the scan
// adds the sums of keys rescaled to the end of their tile and decays the running state by the tile's total gate; the
// tile kernel multiplies the masked scores by exp(λ_i - λ_j) and the state product of row i by exp(λ_i - λ_{tile start - 1}).
// Every exponent is a non-positive difference.
smat_status forward_gated_tc(Ctx& cx, const Gated& gt, const void* Q, const void* K, const void* V, const float* log_a,
                             void* O) {
  const smat_plan* pl = cx.pl;
  const smat_plan* in = pl->inner;
  const bool lr = !pl->geo.dense_G;
  Ctx ci{in, cx.st, cx.ws + pl->off_inner, cudaSuccess, 0};
  ci.rec = pl;
  int* status = reinterpret_cast<int*>(ci.ws + in->off_status);
  SMAT_TRY(cx, "gate_prefix", smat_launch_head_scan(log_a, gt.lam, pl->T, pl->bh, 0, cx.st));
  SMAT_TRY(cx, "gate_scale_k", smat_launch_gate_scale(K, nullptr, gt.kc, gt.lam, 1, 1, pl->geo.n, 128, pl->T, pl->r, pl->bh,
                                                      cx.st));                                // exp(λ_{tile end} - λ_j) k_j
  if (lr) gate_scale(cx, "gate_scale_lr", K, Q, gt.lr, gt.lam, 2, pl->r);                    // split at the boundary
  ci.err = cx.err;
  float* ylr = ci.f(in->off_acc);
  if (lr) {
    build_type_table(ci, gt.lr, V);                                                          // steps 2-3 on the rescaled keys
    if (in->u_bf16)
      SMAT_TRY(ci, "read_type_tc", smat_launch_state_read_tc(gt.lr, ci.ws + in->off_U, ylr, nullptr, 0,
                                                             group(ci, SMAT_GM_TYPE), in->geo.B, in->T, in->bh, status,
                                                             ci.st));                        // step 4 on the rescaled queries
    else
      state_read(ci, "read_type", SMAT_GM_TYPE, gt.lr, ci.f(in->off_U), 0, nullptr, ylr, nullptr);
  }
  SMAT_TRY(ci, "gated_chunk_scan_tc", smat_launch_chunk_scan_tc(gt.kc, V, ci.ws + in->off_sin, in->T, in->bh, in->geo.n,
                                                                 lr ? 0 : 1, 0, status, ci.st, gt.lam));
  SMAT_TRY(ci, "gated_chunk_output_tc", smat_launch_chunk_output_tc(Q, K, V, ci.ws + in->off_sin, ylr, lr ? in->geo.n : in->T,
                                                                     O, in->T, in->bh, status, ci.st, gt.lam));
  pl->launches = cx.launches + ci.launches;
  pl->kept_gated_forward = ci.err == cudaSuccess;
  return ci.err == cudaSuccess ? SMAT_OK : SMAT_ERR_LAUNCH;
}

// The gated backward runs on the tensor cores when the forward does and the inner plan keeps bf16 tables (the fused
// tile kernel takes its long-range rows as bf16); d = 1 has no tables.
bool gated_backward_on_tc(const smat_plan* pl) {
  const smat_plan* in = pl->inner;
  return in && (pl->geo.dense_G || (in->u_bf16 && in->fbar_bf16));
}

// Gated backward on the tensor cores: the ungated adjoint pipeline on rescaled copies (Ū from the boundary-scaled
// queries, the reads of U and F̄ on the boundary-scaled dO, V and K), the decayed scans for S_in (keys rescaled to the
// end of their tile) and D̄ (queries rescaled to the start of theirs, reverse order), and the fused tile kernel with
// the decays on both score tiles and the row factors on the three state products.  dλ_t = q_t·dQ_t - k_t·dK_t.
smat_status backward_gated_tc(Ctx& cx, const Gated& gt, const void* Q, const void* K, const void* V, const float* log_a,
                              const void* dO, void* dQ, void* dK, void* dV, float* dlog_a, bool after_gated_forward) {
  const smat_plan* pl = cx.pl;
  const smat_plan* in = pl->inner;
  const bool lr = !pl->geo.dense_G;
  Ctx ci{in, cx.st, cx.ws + pl->off_inner, cudaSuccess, 0};
  ci.rec = pl;
  int* status = reinterpret_cast<int*>(ci.ws + in->off_status);
  const int64_t n = in->geo.n;
  // With KEEP_FORWARD_TABLES, right after the gated forward of the same inputs on this workspace: λ, the rescaled keys
  // and the boundary-split copy, U and the per-tile incoming states are all still there.
  const bool kept = (pl->flags & SMAT_FLAG_KEEP_FORWARD_TABLES) && after_gated_forward;
  if (!kept) {
    SMAT_TRY(cx, "gate_prefix", smat_launch_head_scan(log_a, gt.lam, pl->T, pl->bh, 0, cx.st));
    SMAT_TRY(cx, "gate_scale_k", smat_launch_gate_scale(K, nullptr, gt.kc, gt.lam, 1, 1, n, 128, pl->T, pl->r, pl->bh, cx.st));
    if (lr) gate_scale(cx, "gate_scale_lr", K, Q, gt.lr, gt.lam, 2, pl->r);
  }
  SMAT_TRY(cx, "bwd_gate_scale_q", smat_launch_gate_scale(Q, nullptr, gt.qc, gt.lam, 0, 1, n, 128, pl->T, pl->r, pl->bh, cx.st));
  if (lr) gate_scale(cx, "bwd_gate_scale_lr", V, dO, gt.vlr, gt.lam, 2, pl->p);
  ci.err = cx.err;
  char* sin = ci.ws + in->off_sin;
  char* dbar = ci.ws + in->off_dbar;
  char *lr_q = nullptr, *lr_k = nullptr, *lr_v = nullptr;
  if (lr) {
    const SmatGroupSpec types = group(ci, SMAT_GM_TYPE), profs = group(ci, SMAT_GM_PROFILE);
    if (!kept) build_type_table(ci, gt.lr, V);
    if (in->ubar_tc)
      SMAT_TRY(ci, "bwd_pool_type_tc", smat_launch_pool_tc(gt.lr, dO, ci.ws + in->off_ubar, in->ubar_bf16, types, in->geo.B,
                                                           max_group_tokens(in, SMAT_GM_TYPE), in->T, in->bh, status, ci.st));
    else
      outer_sum(ci, "bwd_pool_type", SMAT_GM_TYPE, gt.lr, dO, ci.f(in->off_ubar));
    if (in->tab_tc)
      tabulate_tc(ci, "bwd_tabulate_t_tc", ci.ws + in->off_ubar, ci.ws + in->off_fbar, 1);
    else
      tabulate(ci, "bwd_tabulate_t", ci.f(in->off_ubar), ci.f(in->off_fbar), 1, in->geo.D == 2 && in->fbar_bf16);
    lr_q = ci.ws + in->off_acc;
    lr_k = lr_q + (size_t)in->bh * in->T * 128 * 2;
    lr_v = ci.ws + in->off_lr3;
    SMAT_TRY(ci, "bwd_dq_type_tc", smat_launch_state_read_tc(gt.vlr, ci.ws + in->off_U, nullptr, lr_q, 1, types, in->geo.B,
                                                             in->T, in->bh, status, ci.st));
    SMAT_TRY(ci, "bwd_dkdv_profile_tc", smat_launch_state_read_dual_tc(gt.vlr, gt.lr, ci.ws + in->off_fbar, lr_k, lr_v, profs,
                                                                        in->geo.P, in->T, in->bh, status, ci.st));
  }
  if (!kept)
    SMAT_TRY(ci, "gated_chunk_scan_tc", smat_launch_chunk_scan_tc(gt.kc, V, sin, in->T, in->bh, n, lr ? 0 : 1, 0, status, ci.st,
                                                                   gt.lam));
  SMAT_TRY(ci, "bwd_gated_suffix_scan_tc", smat_launch_chunk_scan_tc(gt.qc, dO, dbar, in->T, in->bh, n, lr ? 0 : 1, 1, status,
                                                                      ci.st, gt.lam));
  SMAT_TRY(ci, "bwd_gated_tiles_fused_tc", smat_launch_bwd_tiles_fused_tc(Q, K, V, dO, sin, dbar, lr_q, lr_k, lr_v,
                                                                           lr ? n : in->T, dQ, dK, dV, in->T, in->bh, status,
                                                                           ci.st, gt.lam));
  cx.err = ci.err;
  cx.launches += ci.launches;
  float* dlam = cx.f(pl->off_dlam);
  SMAT_TRY(cx, "bwd_gate_dlam", smat_launch_gate_dlam(Q, dQ, K, dK, dlam, 1, pl->r, pl->T, pl->bh, cx.st));
  SMAT_TRY(cx, "bwd_gate_suffix", smat_launch_head_scan(dlam, dlog_a, pl->T, pl->bh, 1, cx.st));
  pl->launches = cx.launches;
  return cx.err == cudaSuccess ? SMAT_OK : SMAT_ERR_LAUNCH;
}

smat_status gated_check(const smat_plan* pl, const void* log_a, void* ws, size_t ws_bytes, int for_backward) {
  if (!log_a) return SMAT_ERR_NULL;
  smat_status s = check_common(pl, ws, ws_bytes, for_backward);
  if (s != SMAT_OK) return s;
  if (!(pl->flags & SMAT_FLAG_GATED)) return SMAT_ERR_UNSUPPORTED;
  if (reinterpret_cast<uintptr_t>(log_a) & 3) return SMAT_ERR_ALIGN;
  return SMAT_OK;
}

}  // namespace

extern "C" {

smat_status smat_forward_normalized(const smat_plan* pl, const void* Q, const void* K, const void* V, void* O,
                                    void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!pl) return SMAT_ERR_NULL;
  if (!(pl->flags & SMAT_FLAG_NORMALIZED)) return SMAT_ERR_UNSUPPORTED;
  if (!Q || !K || !V || !O || !workspace) return SMAT_ERR_NULL;
  char* ws = static_cast<char*>(workspace);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (workspace_bytes < smat_workspace_bytes(pl, 0)) return SMAT_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(ws) & 255) || misaligned(V) || misaligned(O)) return SMAT_ERR_ALIGN;
  if (!device_ok()) return SMAT_ERR_ARCH;
  const int bf = pl->dtype == SMAT_BF16;
  const int64_t rows = (int64_t)pl->bh * pl->T;
  // v̄ = [v; 1]: the last value column is the normaliser column (Eq. "augmented-kv-state")
  if (smat_launch_normalize_step(0, V, nullptr, ws + pl->off_nv, bf, pl->p, rows, st) != cudaSuccess) return SMAT_ERR_LAUNCH;
  smat_status s = forward_impl(pl, Q, K, ws + pl->off_nv, ws + pl->off_ny, nullptr, nullptr, workspace, workspace_bytes,
                               cuda_stream);
  if (s != SMAT_OK) return s;
  // the single final division (Eq. "augmented-attention-output")
  if (smat_launch_normalize_step(1, ws + pl->off_ny, nullptr, O, bf, pl->p, rows, st) != cudaSuccess) return SMAT_ERR_LAUNCH;
  pl->launches += 2;
  return SMAT_OK;
}

smat_status smat_backward_normalized(const smat_plan* pl, const void* Q, const void* K, const void* V, const void* O,
                                     const void* dO, void* dQ, void* dK, void* dV, void* workspace,
                                     size_t workspace_bytes, void* cuda_stream) {
  if (!pl) return SMAT_ERR_NULL;
  if (!(pl->flags & SMAT_FLAG_NORMALIZED)) return SMAT_ERR_UNSUPPORTED;
  if (!Q || !K || !V || !O || !dO || !dQ || !dK || !dV || !workspace) return SMAT_ERR_NULL;
  char* ws = static_cast<char*>(workspace);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (workspace_bytes < smat_workspace_bytes(pl, 1)) return SMAT_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(ws) & 255) || misaligned(V) || misaligned(O) || misaligned(dO) || misaligned(dV))
    return SMAT_ERR_ALIGN;
  if (!device_ok()) return SMAT_ERR_ARCH;
  const int bf = pl->dtype == SMAT_BF16;
  const int64_t rows = (int64_t)pl->bh * pl->T;
  if (smat_launch_normalize_step(0, V, nullptr, ws + pl->off_nv, bf, pl->p, rows, st) != cudaSuccess) return SMAT_ERR_LAUNCH;
  // backward of the final division, then the linear pass with the augmented upstream
  if (smat_launch_normalize_step(2, O, dO, ws + pl->off_ndy, bf, pl->p, rows, st) != cudaSuccess) return SMAT_ERR_LAUNCH;
  smat_status s = backward_impl(pl, Q, K, ws + pl->off_nv, ws + pl->off_ndy, dQ, dK, dV, nullptr, nullptr, workspace,
                                workspace_bytes, cuda_stream);
  if (s != SMAT_OK) return s;
  if (smat_launch_normalize_step(3, nullptr, nullptr, dV, bf, pl->p, rows, st) != cudaSuccess) return SMAT_ERR_LAUNCH;
  pl->launches += 3;
  return SMAT_OK;
}

smat_status smat_forward_gated(const smat_plan* pl, const void* Q, const void* K, const void* V, const float* log_a,
                               void* O, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!Q || !K || !V || !O) return SMAT_ERR_NULL;
  smat_status s = gated_check(pl, log_a, workspace, workspace_bytes, 0);
  if (s != SMAT_OK) return s;
  if (misaligned(Q) || misaligned(K) || misaligned(V) || misaligned(O)) return SMAT_ERR_ALIGN;
  if (!device_ok()) return SMAT_ERR_ARCH;
  Ctx cx{pl, static_cast<cudaStream_t>(cuda_stream), static_cast<char*>(workspace), cudaSuccess, 0};
  pl->stages = 0;
  pl->tile_states = false;
  cx.err = clear_status(cx);
  const Gated gt = gated_buffers(cx);
  if (pl->inner) return forward_gated_tc(cx, gt, Q, K, V, log_a, O);
  gated_forward_tables(cx, gt, Q, K, V, log_a);
  float* acc = cx.f(pl->off_acc);
  float* tileA = cx.f(pl->off_tileA);
  tril_scores(cx, "scores", Q, K, pl->r, tileA, gt.lam);                         // tril(QKᵀ) ⊙ exp(λ_i - λ_j)
  state_read(cx, "read_chunk", SMAT_GM_CHUNK, gt.qc, cx.f(pl->off_sin), 0, nullptr, acc, nullptr);
  if (!pl->geo.dense_G) state_read(cx, "read_type", SMAT_GM_TYPE, gt.lr, cx.f(pl->off_U), 0, acc, acc, nullptr);
  tile_apply(cx, "output", tileA, 0, V, pl->p, acc, nullptr, O);
  pl->launches = cx.launches;
  return cx.err == cudaSuccess ? SMAT_OK : SMAT_ERR_LAUNCH;
}

smat_status smat_backward_gated(const smat_plan* pl, const void* Q, const void* K, const void* V, const float* log_a,
                                const void* dO, void* dQ, void* dK, void* dV, float* dlog_a, void* workspace,
                                size_t workspace_bytes, void* cuda_stream) {
  if (!Q || !K || !V || !dO || !dQ || !dK || !dV || !dlog_a) return SMAT_ERR_NULL;
  smat_status s = gated_check(pl, log_a, workspace, workspace_bytes, 1);
  if (s != SMAT_OK) return s;
  if (misaligned(Q) || misaligned(K) || misaligned(V) || misaligned(dO) || misaligned(dQ) || misaligned(dK) ||
      misaligned(dV) || (reinterpret_cast<uintptr_t>(dlog_a) & 3))
    return SMAT_ERR_ALIGN;
  if (!device_ok()) return SMAT_ERR_ARCH;
  Ctx cx{pl, static_cast<cudaStream_t>(cuda_stream), static_cast<char*>(workspace), cudaSuccess, 0};
  pl->stages = 0;
  pl->tile_states = false;
  const bool after_gated_forward = pl->kept_gated_forward;   // read before the pass resets it
  cx.err = clear_status(cx);
  const bool lr = !pl->geo.dense_G;
  const Gated gt = gated_buffers(cx);
  if (gated_backward_on_tc(pl)) return backward_gated_tc(cx, gt, Q, K, V, log_a, dO, dQ, dK, dV, dlog_a, after_gated_forward);
  gated_forward_tables(cx, gt, Q, K, V, log_a);
  gate_scale(cx, "bwd_gate_scale_do", dO, nullptr, gt.doc, gt.lam, 0, pl->p);    // exp(λ_i - λ_{e(b-1)}) dO_i
  gate_scale(cx, "bwd_gate_scale_v", V, nullptr, gt.vc, gt.lam, 1, pl->p);       // exp(λ_{e(b)} - λ_j) v_j
  if (lr) gate_scale(cx, "bwd_gate_scale_lr", V, dO, gt.vlr, gt.lam, 2, pl->p);  // values / upstream rows at the boundary
  float* sin = cx.f(pl->off_sin);
  float* dbar = cx.f(pl->off_dbar);
  float* acc = cx.f(pl->off_acc);
  float* tileA = cx.f(pl->off_tileA);
  float* tileG = cx.f(pl->off_tileG);
  // adjoint of the carried state: S̄_in_b = Σ_i (scaled q_i) dO_iᵀ, then the decayed suffix recursion
  outer_sum(cx, "bwd_chunk_state", SMAT_GM_CHUNK, gt.qc, dO, dbar);
  gated_scan(cx, "bwd_gated_scan", dbar, gt.lam, 1);
  if (lr) {
    outer_sum(cx, "bwd_pool_type", SMAT_GM_TYPE, gt.lr, dO, cx.f(pl->off_ubar));
    tabulate(cx, "bwd_tabulate_t", cx.f(pl->off_ubar), cx.f(pl->off_fbar), 1);
  }
  tril_scores(cx, "bwd_scores_qk", Q, K, pl->r, tileA, gt.lam);
  tril_scores(cx, "bwd_scores_gv", dO, V, pl->p, tileG, gt.lam);
  // dQ_i = S_in (scaled dO_i) + U_type (boundary-scaled dO_i) + Σ_j G_ij k_j
  state_read(cx, "bwd_dq_chunk", SMAT_GM_CHUNK, gt.doc, sin, 1, nullptr, acc, nullptr);
  if (lr) state_read(cx, "bwd_dq_type", SMAT_GM_TYPE, gt.vlr, cx.f(pl->off_U), 1, acc, acc, nullptr);
  tile_apply(cx, "bwd_dq_tile", tileG, 0, K, pl->r, acc, nullptr, dQ);
  // dK_j = Σ_i G_ij q_i + F̄_prof (boundary-scaled v_j) + D̄ (chunk-scaled v_j)
  tile_apply(cx, "bwd_dk_tile", tileG, 1, Q, pl->r, nullptr, acc, nullptr);
  if (lr) state_read(cx, "bwd_dk_profile", SMAT_GM_PROFILE, gt.vlr, cx.f(pl->off_fbar), 1, acc, acc, nullptr);
  state_read(cx, "bwd_dk_chunk", SMAT_GM_CHUNK, gt.vc, dbar, 1, acc, nullptr, dK);
  // dV_j = Σ_i A_ij dO_i + F̄_profᵀ (boundary-scaled k_j) + D̄ᵀ (chunk-scaled k_j)
  tile_apply(cx, "bwd_dv_tile", tileA, 1, dO, pl->p, nullptr, acc, nullptr);
  if (lr) state_read(cx, "bwd_dv_profile", SMAT_GM_PROFILE, gt.lr, cx.f(pl->off_fbar), 0, acc, acc, nullptr);
  state_read(cx, "bwd_dv_chunk", SMAT_GM_CHUNK, gt.kc, dbar, 0, acc, nullptr, dV);
  // gates: dλ_t = q_t·dQ_t - k_t·dK_t, and log a_k enters every λ_t with t >= k
  float* dlam = cx.f(pl->off_dlam);
  SMAT_TRY(cx, "bwd_gate_dlam", smat_launch_gate_dlam(Q, dQ, K, dK, dlam, pl->dtype == SMAT_BF16, pl->r, pl->T, pl->bh, cx.st));
  SMAT_TRY(cx, "bwd_gate_suffix", smat_launch_head_scan(dlam, dlog_a, pl->T, pl->bh, 1, cx.st));
  pl->launches = cx.launches;
  return cx.err == cudaSuccess ? SMAT_OK : SMAT_ERR_LAUNCH;
}

smat_status smat_forward(const smat_plan* pl, const void* Q, const void* K, const void* V, void* O, void* workspace,
                         size_t workspace_bytes, void* cuda_stream) {
  return forward_impl(pl, Q, K, V, O, nullptr, nullptr, workspace, workspace_bytes, cuda_stream);
}

smat_status smat_backward(const smat_plan* pl, const void* Q, const void* K, const void* V, const void* dO, void* dQ,
                          void* dK, void* dV, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return backward_impl(pl, Q, K, V, dO, dQ, dK, dV, nullptr, nullptr, workspace, workspace_bytes, cuda_stream);
}

smat_status smat_forward_routed(const smat_plan* pl, const void* Q, const void* K, const void* V, void* O,
                                const int32_t* prof, const int32_t* type, void* workspace, size_t workspace_bytes,
                                void* cuda_stream) {
  if (!prof || !type) return SMAT_ERR_NULL;
  return forward_impl(pl, Q, K, V, O, prof, type, workspace, workspace_bytes, cuda_stream);
}

smat_status smat_backward_routed(const smat_plan* pl, const void* Q, const void* K, const void* V, const void* dO,
                                 void* dQ, void* dK, void* dV, const int32_t* prof, const int32_t* type, void* workspace,
                                 size_t workspace_bytes, void* cuda_stream) {
  if (!prof || !type) return SMAT_ERR_NULL;
  return backward_impl(pl, Q, K, V, dO, dQ, dK, dV, prof, type, workspace, workspace_bytes, cuda_stream);
}

smat_status smat_routing_indices(const smat_plan* pl, int32_t* prof, int32_t* type, int32_t* type_ab) {
  if (!pl) return SMAT_ERR_NULL;
  const SmatGeo& g = pl->geo;
  if (g.dense_G) {
    if (type) for (int64_t i = 0; i < g.m; ++i) type[i] = 0;
    if (type_ab) type_ab[0] = 0;
    return SMAT_OK;
  }
  if (prof)
    for (int64_t t = 0; t < g.n; ++t) {
      int64_t v = smat_profile_of(g, t);
      for (int k = 0; k < g.D; ++k) { prof[t * g.D + k] = (int32_t)(v % g.q); v /= g.q; }
    }
  if (type)
    for (int64_t t = g.n; t < g.T; ++t) type[t - g.n] = (int32_t)smat_type_of(g, t);
  if (type_ab)
    for (int64_t h = 0; h < g.B; ++h) {
      int32_t a[SMAT_MAX_DIM];
      smat_direction(g, h / g.q, a);
      for (int k = 0; k < g.D; ++k) type_ab[h * g.d + k] = a[k];
      type_ab[h * g.d + g.D] = (int32_t)(h % g.q);
    }
  return SMAT_OK;
}

smat_status smat_debug_mask(const smat_plan* pl, uint8_t* mask, void* cuda_stream) {
  if (!pl || !mask) return SMAT_ERR_NULL;
  if (pl->T > 8192) return SMAT_ERR_SHAPE;
  if (!device_ok()) return SMAT_ERR_ARCH;
  return smat_launch_mask(mask, pl->geo, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? SMAT_OK
                                                                                                 : SMAT_ERR_LAUNCH;
}

smat_status smat_debug_tables(const smat_plan* pl, const void* workspace, float* F, float* U, float* Sin,
                              void* cuda_stream) {
  if (!pl || !workspace) return SMAT_ERR_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const char* ws = static_cast<const char*>(workspace);
  const size_t state = (size_t)pl->rp * sizeof(float);
  cudaError_t err = cudaSuccess;
  if (pl->tc) {
    // Tensor-core plans: incoming states exist per 128-token tile (bf16) after a per-tile forward or a backward; the
    // two-level form keeps only one state per segment of tiles, which is no per-chunk table.
    const bool want_states = Sin || (pl->geo.dense_G && (F || U));
    if (want_states && !pl->tile_states) return SMAT_ERR_UNSUPPORTED;
    const int64_t tiles = pl->T / 128;
    if (Sin) err = smat_launch_widen_bf16(ws + pl->off_sin, Sin, (int64_t)pl->bh * tiles * pl->rp, st);
    if (pl->geo.dense_G) {  // d = 1: the state entering the first recent tile is U_0 = F_0
      for (int t = 0; t < 2; ++t) {
        float* dst = t ? U : F;
        for (int h = 0; dst && h < pl->bh && err == cudaSuccess; ++h)
          err = smat_launch_widen_bf16(ws + pl->off_sin + ((size_t)h * tiles + pl->geo.n / 128) * pl->rp * 2,
                                       dst + (size_t)h * pl->rp, pl->rp, st);
      }
      return err == cudaSuccess ? SMAT_OK : SMAT_ERR_LAUNCH;
    }
  } else if (Sin) {
    err = cudaMemcpyAsync(Sin, ws + pl->off_sin, (size_t)pl->bh * pl->NC * state, cudaMemcpyDeviceToDevice, st);
  }
  if (pl->geo.dense_G) {
    const int64_t first_recent = pl->geo.n / pl->c;
    for (int t = 0; t < 2; ++t) {
      float* dst = t ? U : F;
      if (!dst || err != cudaSuccess) continue;
      err = cudaMemcpy2DAsync(dst, state, ws + pl->off_sin + (size_t)first_recent * state, (size_t)pl->NC * state,
                              state, pl->bh, cudaMemcpyDeviceToDevice, st);
    }
  } else {
    if (F && err == cudaSuccess) {
      if (pl->tab_d3_regs)
        err = smat_launch_widen_bf16_slabs(ws + pl->off_F, F, pl->bh, pl->geo.P, pl->rp, st);
      else if (pl->f_bf16)
        err = smat_launch_widen_bf16(ws + pl->off_F, F, (int64_t)pl->bh * pl->geo.P * pl->rp, st);
      else
        err = cudaMemcpyAsync(F, ws + pl->off_F, (size_t)pl->bh * pl->geo.P * state, cudaMemcpyDeviceToDevice, st);
    }
    if (U && err == cudaSuccess) {
      if (pl->u_bf16)  // this plan keeps U in bf16: widen on export
        err = smat_launch_widen_bf16(ws + pl->off_U, U, (int64_t)pl->bh * pl->geo.B * pl->rp, st);
      else
        err = cudaMemcpyAsync(U, ws + pl->off_U, (size_t)pl->bh * pl->geo.B * state, cudaMemcpyDeviceToDevice, st);
    }
  }
  return err == cudaSuccess ? SMAT_OK : SMAT_ERR_LAUNCH;
}

smat_status smat_check_status(const smat_plan* pl, const void* workspace, void* cuda_stream) {
  if (!pl || !workspace) return SMAT_ERR_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int word = 0, word2 = 0;
  if (cudaMemcpyAsync(&word, static_cast<const char*>(workspace) + pl->off_status, sizeof(int), cudaMemcpyDeviceToHost,
                      st) != cudaSuccess)
    return SMAT_ERR_LAUNCH;
  if (pl->inner &&   // the tensor-core forward of a gated plan reports into the status word of its own region
      cudaMemcpyAsync(&word2, static_cast<const char*>(workspace) + pl->off_inner + pl->inner->off_status, sizeof(int),
                      cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return SMAT_ERR_LAUNCH;
  if (cudaStreamSynchronize(st) != cudaSuccess) return SMAT_ERR_LAUNCH;
  return (word | word2) == 0 ? SMAT_OK : SMAT_ERR_DEVICE_TIMEOUT;
}

int smat_last_launch_count(const smat_plan* pl) { return pl ? pl->launches : 0; }

int smat_debug_tabulation_layout_ok(int q) { return smat_tabulate_tc_layout_ok(q); }

size_t smat_decode_cache_bytes(const smat_plan* pl) {
  if (!pl) return 0;   // type table, running state, and on gated plans the running log-gate of every head
  return decode_table_bytes(pl) + decode_state_bytes(pl) + ((pl->flags & SMAT_FLAG_GATED) ? align_up((size_t)pl->bh * 4) : 0);
}

smat_status smat_decode_begin(const smat_plan* pl, const void* K, const void* V, void* cache, size_t cache_bytes,
                              void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!K || !V || !cache) return SMAT_ERR_NULL;
  if (pl && (pl->flags & SMAT_FLAG_GATED)) return SMAT_ERR_UNSUPPORTED;   // gated plans decode with the gated pair of calls
  smat_status s = check_common(pl, workspace, workspace_bytes, 0);
  if (s != SMAT_OK) return s;
  if (cache_bytes < smat_decode_cache_bytes(pl)) return SMAT_ERR_WORKSPACE;
  if (misaligned(K) || misaligned(V) || (reinterpret_cast<uintptr_t>(cache) & 255)) return SMAT_ERR_ALIGN;
  if (!device_ok()) return SMAT_ERR_ARCH;
  Ctx cx{pl, static_cast<cudaStream_t>(cuda_stream), static_cast<char*>(workspace), cudaSuccess, 0};
  pl->stages = 0;
  cx.err = clear_status(cx);
  const size_t off = build_type_table(cx, K, V);
  const size_t tbytes = (size_t)pl->bh * pl->geo.B * pl->rp * (pl->u_bf16 ? 2 : 4);
  if (cx.err == cudaSuccess)
    cx.err = cudaMemcpyAsync(cache, cx.ws + off, tbytes, cudaMemcpyDeviceToDevice, cx.st);
  if (cx.err == cudaSuccess)
    cx.err = cudaMemsetAsync(static_cast<char*>(cache) + decode_table_bytes(pl), 0, (size_t)pl->bh * pl->rp * sizeof(float),
                             cx.st);
  pl->launches = cx.launches;
  return cx.err == cudaSuccess ? SMAT_OK : SMAT_ERR_LAUNCH;
}

smat_status smat_decode_step(const smat_plan* pl, const void* q, const void* k, const void* v, int64_t t, void* o,
                             void* cache, size_t cache_bytes, void* cuda_stream) {
  if (!pl || !q || !k || !v || !o || !cache) return SMAT_ERR_NULL;
  if (pl->flags & SMAT_FLAG_GATED) return SMAT_ERR_UNSUPPORTED;
  if (cache_bytes < smat_decode_cache_bytes(pl)) return SMAT_ERR_WORKSPACE;
  if (t < pl->geo.n || t >= pl->T) return SMAT_ERR_SHAPE;
  if (reinterpret_cast<uintptr_t>(cache) & 255) return SMAT_ERR_ALIGN;
  if (!device_ok()) return SMAT_ERR_ARCH;
  float* S = reinterpret_cast<float*>(static_cast<char*>(cache) + decode_table_bytes(pl));
  const cudaError_t err = smat_launch_decode_step(q, k, v, o, S, cache, pl->u_bf16 ? 1 : 0, pl->dtype == SMAT_BF16 ? 1 : 0,
                                                  smat_type_of(pl->geo, t), pl->geo.B, pl->r, pl->p, pl->bh,
                                                  static_cast<cudaStream_t>(cuda_stream));
  pl->launches = 1;
  return err == cudaSuccess ? SMAT_OK : SMAT_ERR_LAUNCH;
}

smat_status smat_decode_begin_gated(const smat_plan* pl, const void* K, const void* V, const float* log_a, void* cache,
                                    size_t cache_bytes, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!K || !V || !cache) return SMAT_ERR_NULL;
  smat_status s = gated_check(pl, log_a, workspace, workspace_bytes, 0);
  if (s != SMAT_OK) return s;
  if (cache_bytes < smat_decode_cache_bytes(pl)) return SMAT_ERR_WORKSPACE;
  if (misaligned(K) || misaligned(V) || (reinterpret_cast<uintptr_t>(cache) & 255)) return SMAT_ERR_ALIGN;
  if (!device_ok()) return SMAT_ERR_ARCH;
  Ctx cx{pl, static_cast<cudaStream_t>(cuda_stream), static_cast<char*>(workspace), cudaSuccess, 0};
  pl->stages = 0;
  cx.err = clear_status(cx);
  const Gated gt = gated_buffers(cx);
  // λ, the keys rescaled to the block boundary (rows t < n of the split copy), then steps 2-3 of Algorithm 1 on them
  SMAT_TRY(cx, "gate_prefix", smat_launch_head_scan(log_a, gt.lam, pl->T, pl->bh, 0, cx.st));
  gate_scale(cx, "gate_scale_lr", K, K, gt.lr, gt.lam, 2, pl->r);
  const smat_plan* tp = decode_table_plan(pl);
  Ctx ct{tp, cx.st, cx.ws + (tp == pl ? 0 : pl->off_inner), cx.err, 0};
  ct.rec = pl;
  const size_t off = build_type_table(ct, gt.lr, V);
  cx.err = ct.err;
  const size_t tbytes = (size_t)pl->bh * pl->geo.B * pl->rp * (tp->u_bf16 ? 2 : 4);
  if (cx.err == cudaSuccess) cx.err = cudaMemcpyAsync(cache, ct.ws + off, tbytes, cudaMemcpyDeviceToDevice, cx.st);
  if (cx.err == cudaSuccess)   // S = 0 and log g = 0 (they follow the table)
    cx.err = cudaMemsetAsync(static_cast<char*>(cache) + decode_table_bytes(pl), 0,
                             smat_decode_cache_bytes(pl) - decode_table_bytes(pl), cx.st);
  pl->launches = cx.launches + ct.launches;
  return cx.err == cudaSuccess ? SMAT_OK : SMAT_ERR_LAUNCH;
}

smat_status smat_decode_step_gated(const smat_plan* pl, const void* q, const void* k, const void* v, const float* log_a_t,
                                   int64_t t, void* o, void* cache, size_t cache_bytes, void* cuda_stream) {
  if (!pl || !q || !k || !v || !o || !cache || !log_a_t) return SMAT_ERR_NULL;
  if (!(pl->flags & SMAT_FLAG_GATED)) return SMAT_ERR_UNSUPPORTED;
  if (cache_bytes < smat_decode_cache_bytes(pl)) return SMAT_ERR_WORKSPACE;
  if (t < pl->geo.n || t >= pl->T) return SMAT_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(cache) & 255) || (reinterpret_cast<uintptr_t>(log_a_t) & 3)) return SMAT_ERR_ALIGN;
  if (!device_ok()) return SMAT_ERR_ARCH;
  char* base = static_cast<char*>(cache);
  float* S = reinterpret_cast<float*>(base + decode_table_bytes(pl));
  float* log_g = reinterpret_cast<float*>(base + decode_table_bytes(pl) + decode_state_bytes(pl));
  const cudaError_t err = smat_launch_decode_step(q, k, v, o, S, cache, decode_table_plan(pl)->u_bf16 ? 1 : 0,
                                                  pl->dtype == SMAT_BF16 ? 1 : 0, smat_type_of(pl->geo, t), pl->geo.B, pl->r,
                                                  pl->p, pl->bh, static_cast<cudaStream_t>(cuda_stream), log_a_t, log_g);
  pl->launches = 1;
  return err == cudaSuccess ? SMAT_OK : SMAT_ERR_LAUNCH;
}

const char* smat_status_string(smat_status s) {
  switch (s) {
    case SMAT_OK: return "ok";
    case SMAT_ERR_NULL: return "null pointer";
    case SMAT_ERR_SHAPE: return "unsupported shape";
    case SMAT_ERR_DTYPE: return "unknown dtype";
    case SMAT_ERR_GEOMETRY: return "invalid mask geometry";
    case SMAT_ERR_WORKSPACE: return "workspace too small";
    case SMAT_ERR_ALIGN: return "misaligned pointer";
    case SMAT_ERR_ARCH: return "device is not sm_100";
    case SMAT_ERR_LAUNCH: return "CUDA launch or runtime failure";
    case SMAT_ERR_DEVICE_TIMEOUT: return "bounded device wait expired";
    case SMAT_ERR_UNSUPPORTED: return "no kernel path for this request";
  }
  return "unknown status";
}

}  // extern "C"
