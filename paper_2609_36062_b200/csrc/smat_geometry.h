// Integer geometry of the SMat mask family, shared by the host planner and the device kernels.
//
// Sec. 3 ("construction of G", "Scaling with sequence length"): hyperplanes H_{a,b} = {x : aᵀx = b}
// over F_q^{D}, D = d-1; positional assignment prof(t) = base-q digits of t mod q^D (least
// significant digit first), type(i) = i mod B with the paper's 1-based recent index i.
// Types are numbered h = dir*q + b; directions (first nonzero coordinate equal to one) are ordered
// by the position g of that leading one, and inside a group by the remaining coordinates read as a
// little-endian base-q integer.
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define SMAT_HD __host__ __device__ __forceinline__
#else
#define SMAT_HD inline
#endif

#define SMAT_MAX_D 8          // largest VC dimension accepted
#define SMAT_MAX_DIM (SMAT_MAX_D - 1)

struct SmatGeo {
  int64_t T, c, n, m;
  int32_t d, q, D;
  int64_t P, A, B, nnzC;
  int32_t dense_G;            // 1 when d == 1: one point, one hyperplane that contains it
  int64_t qpow[SMAT_MAX_D];   // qpow[k] = q^k
  int64_t dir_group_start[SMAT_MAX_D];  // first direction index of the group with leading one at position g (0-based)
};

// Direction number `dir` -> coordinates a[0..D).
SMAT_HD void smat_direction(const SmatGeo& g, int64_t dir, int32_t* a) {
  int lead = 0;
  while (lead + 1 < g.D && dir >= g.dir_group_start[lead + 1]) ++lead;
  int64_t tail = dir - g.dir_group_start[lead];
  for (int k = 0; k < g.D; ++k) a[k] = 0;
  a[lead] = 1;
  for (int k = lead + 1; k < g.D; ++k) {
    a[k] = (int32_t)(tail % g.q);
    tail /= g.q;
  }
}

// aᵀx mod q for the point with packed (little-endian) index v.
SMAT_HD int32_t smat_dot_point(const SmatGeo& g, const int32_t* a, int64_t v) {
  int64_t acc = 0;
  for (int k = 0; k < g.D; ++k) {
    acc += (int64_t)a[k] * (v % g.q);
    v /= g.q;
  }
  return (int32_t)(acc % g.q);
}

// Type of recent token t (t >= n).
SMAT_HD int64_t smat_type_of(const SmatGeo& g, int64_t t) { return g.dense_G ? 0 : (t - g.n + 1) % g.B; }

// Packed profile of distant token t (t < n).
SMAT_HD int64_t smat_profile_of(const SmatGeo& g, int64_t t) { return g.dense_G ? 0 : t % g.P; }

// One entry of M^(d) (Eq. "blockform", Eq. "Gdef").
SMAT_HD int smat_mask_entry(const SmatGeo& g, int64_t t, int64_t s) {
  if (s > t) return 0;
  if (t < g.n || s >= g.n) return 1;
  if (g.dense_G) return 1;
  int64_t h = smat_type_of(g, t);
  int32_t a[SMAT_MAX_DIM];
  smat_direction(g, h / g.q, a);
  return smat_dot_point(g, a, smat_profile_of(g, s)) == (int32_t)(h % g.q);
}
