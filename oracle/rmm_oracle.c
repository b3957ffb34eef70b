/*
 * CPU oracle for the randomized-matrix-multiplication (RMM) linear layer.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, fp64
 * restatement of what the layer computes, written from the paper's definitions
 * (Eq. 1-4, Algorithm 1, Eq. 5, Lemma 1, Lemma 2, Theorem 1's alpha) so that the
 * CUDA library can be compared against it.  It shares no code, header, table or
 * constant generator with the CUDA path.  Only the tests, the smoke check and the
 * benchmark's CPU-baseline leg may load it.
 *
 * Every contraction is the textbook triple loop in fp64, parallelised over output
 * rows with OpenMP and nothing else: no blocking, no BLAS, no reordering of the
 * sums (each output element adds its terms in index order).
 *
 * The sketch matrix S is defined by a counter-based generator (Philox4x32-10,
 * Salmon et al. 2011) plus a fixed sequence of correctly rounded fp32 operations,
 * so that an independent implementation reproduces every entry bit for bit.
 * Compile with -ffp-contract=off: the only fused multiply-adds are the explicit
 * fmaf() calls below.
 *
 * Pins (tests marked "not gpu"): Philox known-answer vectors cross-checked with an
 * independent implementation; the Gaussian transform against fp64 Box-Muller over
 * all 2^16 radius and angle inputs; brute-force numpy loops on tiny shapes; S = I
 * reproducing the exact gradient; Monte-Carlo unbiasedness and variance; the
 * paper's worked 2x2 example for the two variance estimators; the structured
 * sketches against scipy's Hadamard and DCT-II matrices.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_DIST_GAUSSIAN 0
#define ORACLE_DIST_RADEMACHER 1
#define ORACLE_DIST_IDENTITY 2
#define ORACLE_DIST_SORS 3
#define ORACLE_DIST_DCT 4
#define ORACLE_STORE_BF16 0
#define ORACLE_STORE_F32 1

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void oracle_set_num_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}

/* ---------------------------------------------------------------------------
 * Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy
 * as 1, 2, 3", SC'11).  One round maps (c0,c1,c2,c3) with round key (k0,k1) to
 * (hi(M1*c2)^c1^k0, lo(M1*c2), hi(M0*c0)^c3^k1, lo(M0*c0)); the key is bumped by
 * the Weyl constants between rounds; ten rounds.
 * ------------------------------------------------------------------------- */
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
  const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    uint64_t p0 = (uint64_t)M0 * c0;
    uint64_t p1 = (uint64_t)M1 * c2;
    uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    uint32_t n1 = (uint32_t)p1;
    uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    uint32_t n3 = (uint32_t)p0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += W0; k1 += W1;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

static inline uint32_t f32_bits(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }
static inline float bits_f32(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }

/* Round an fp32 value to the nearest bfloat16 (ties to even), returned as fp32. */
float oracle_bf16_round(float x) {
  uint32_t u = f32_bits(x);
  if ((u & 0x7fffffffu) > 0x7f800000u) return x; /* NaN: not produced here */
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7fffu + lsb;
  u &= 0xffff0000u;
  return bits_f32(u);
}

/* ---------------------------------------------------------------------------
 * One 32-bit Philox word -> two standard normals (Box-Muller on 16-bit uniforms).
 *
 * radius: hi = word >> 16, u_a = (2 hi + 1) / 2^17 in (0,1).  Write the odd
 *   integer v = 2 hi + 1 as 2^e * m with m in [1,2); then
 *   -2 ln u_a = 2 ln2 * (17 - e) - 2 ln m, with -2 ln m replaced by a degree-6
 *   polynomial in m (Horner, fmaf).  rad = sqrtf(.) correctly rounded.
 * angle: lo = word & 0xffff.  Bit 15 chooses the half plane (a sign on both
 *   outputs), the low 15 bits give y = (2 p + 1) / 2^15 - 1 in (-1,1) and the
 *   angle pi/2 * y; sin(pi/2 y) = y * S(y^2) and cos(pi/2 y) = C(y^2) with cubic
 *   S and C (Horner, fmaf).
 * even output = +-rad * cos, odd output = +-rad * sin.
 * All constants are part of the definition of S.
 * ------------------------------------------------------------------------- */
static const float LN_C[7] = {
    0x1.0db894p+2f, -0x1.0f2e02p+3f, 0x1.d9f4dap+2f, -0x1.239714p+2f,
    0x1.c19e4cp+0f, -0x1.869778p-2f, 0x1.23c2eep-5f};
static const float TWO_LN2 = 0x1.62e43p+0f;
static const float SIN_C[4] = {0x1.921fa2p+0f, -0x1.4ab6cep-1f, 0x1.45a27ap-4f, -0x1.1e7576p-8f};
static const float COS_C[4] = {0x1.ffff2p-1f, -0x1.3bc5a4p+0f, 0x1.02a464p-2f, -0x1.38dd52p-6f};

void oracle_gauss_pair(uint32_t word, float* z_even, float* z_odd) {
  /* radius */
  uint32_t hi = word >> 16;
  float fv = (float)(2u * hi + 1u);            /* exact: at most 17 bits */
  uint32_t fb = f32_bits(fv);
  float ef = (float)((int32_t)(fb >> 23) - 144); /* e - 17, exact small integer */
  float m = bits_f32((fb & 0x007fffffu) | 0x3f800000u);
  float p = LN_C[6];
  for (int i = 5; i >= 0; --i) p = fmaf(p, m, LN_C[i]);
  float t = fmaf(-TWO_LN2, ef, p);
  float rad = sqrtf(t);
  /* angle */
  uint32_t lo = word & 0xffffu;
  uint32_t pp = lo & 0x7fffu;
  float y = fmaf((float)(2u * pp + 1u), 0x1p-15f, -1.0f); /* exact */
  float z = y * y;
  float sp = fmaf(fmaf(fmaf(SIN_C[3], z, SIN_C[2]), z, SIN_C[1]), z, SIN_C[0]);
  float sn = y * sp;
  float cs = fmaf(fmaf(fmaf(COS_C[3], z, COS_C[2]), z, COS_C[1]), z, COS_C[0]);
  float rs = (lo >> 15) ? -rad : rad;
  *z_even = rs * cs;
  *z_odd = rs * sn;
}

/* Scale c such that S = c * P: 1/sqrt(k) for Gaussian and Rademacher entries
 * (Eq. 5; unit-variance entries need this factor for E[S S^T] = I), 1 for the
 * identity test matrix.  Computed in fp32 with correctly rounded operations. */
float oracle_scale(int64_t k, int dist) {
  if (dist == ORACLE_DIST_IDENTITY) return 1.0f;
  return 1.0f / sqrtf((float)k);
}

/* Unscaled entries P[n][j] for n in [0,N), j in [j0,j1), after rounding to the
 * storage type; out is [N, j1-j0] row-major fp32.
 * Gaussian: counter (n>>3, j, 0, 0) -> 4 words -> 8 normals for tokens
 *   8*(n>>3) .. +7 of column j (word i gives tokens 2i and 2i+1).
 * Rademacher: counter (n>>7, j, 0, 1) -> 128 bits; token n takes bit (n&31) of
 *   word ((n&127)>>5); a set bit means -1.
 * Identity: P[n][j] = (n == j).
 * SORS (subsampled orthonormal with random signs; the paper names the family in
 *   Section 2.1 and gives no construction; this one is defined here): with L the
 *   smallest power of two >= N and H the Sylvester Hadamard matrix of order L,
 *   H[n][r] = (-1)^popcount(n & r):  P[n][j] = d_n * H[n][r_j], where d_n = -1 when
 *   bit (n&31) of word ((n&127)>>5) of counter (n>>7, 0, 0, 2) is set, and r_j is the
 *   first word of counter (j, 0, 0, 3) modulo L. */
void oracle_generate_p_cols(uint64_t seed, int64_t N, int64_t k, int64_t j0, int64_t j1,
                            int dist, int storage, float* out) {
  const int64_t w = j1 - j0;
  uint32_t key[2] = {(uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32)};
  (void)k;
  if (dist == ORACLE_DIST_IDENTITY) {
    for (int64_t n = 0; n < N; ++n)
      for (int64_t j = j0; j < j1; ++j) out[n * w + (j - j0)] = (n == j) ? 1.0f : 0.0f;
    return;
  }
  if (dist == ORACLE_DIST_GAUSSIAN) {
    const int64_t nblk = (N + 7) / 8;
#pragma omp parallel for schedule(static)
    for (int64_t q = 0; q < nblk; ++q) {
      for (int64_t j = j0; j < j1; ++j) {
        uint32_t ctr[4] = {(uint32_t)q, (uint32_t)j, 0u, 0u}, r[4];
        oracle_philox4x32_10(ctr, key, r);
        for (int i = 0; i < 4; ++i) {
          float ze, zo;
          oracle_gauss_pair(r[i], &ze, &zo);
          if (storage == ORACLE_STORE_BF16) { ze = oracle_bf16_round(ze); zo = oracle_bf16_round(zo); }
          int64_t n = 8 * q + 2 * i;
          if (n < N) out[n * w + (j - j0)] = ze;
          if (n + 1 < N) out[(n + 1) * w + (j - j0)] = zo;
        }
      }
    }
    return;
  }
  if (dist == ORACLE_DIST_SORS) {
    uint64_t L = 1;
    while (L < (uint64_t)N) L <<= 1;
    for (int64_t j = j0; j < j1; ++j) {
      uint32_t cj[4] = {(uint32_t)j, 0u, 0u, 3u}, rj[4];
      oracle_philox4x32_10(cj, key, rj);
      const uint64_t col = (uint64_t)rj[0] % L;
      for (int64_t n = 0; n < N; ++n) {
        uint32_t cn[4] = {(uint32_t)(n >> 7), 0u, 0u, 2u}, rn[4];
        oracle_philox4x32_10(cn, key, rn);
        const int t = (int)(n & 127);
        const int d_neg = (int)((rn[t >> 5] >> (t & 31)) & 1u);
        int ones = 0;                                   /* popcount(n & col), bit by bit */
        for (uint64_t b = (uint64_t)n & col; b != 0; b >>= 1) ones += (int)(b & 1u);
        const float h = (ones & 1) ? -1.0f : 1.0f;
        out[n * w + (j - j0)] = d_neg ? -h : h;
      }
    }
    return;
  }
  if (dist == ORACLE_DIST_DCT) {
    /* Subsampled DCT-II with random signs (Section 3.5 compares DCT sketches, Section 2.1 names the SORS
     * family; the construction is defined here).  L = smallest power of two >= N; the orthonormal DCT-II
     * matrix of order L has rows C[0][n] = sqrt(1/L), C[r][n] = sqrt(2/L) cos(pi (2n+1) r / (2L)).
     * P[n][j] = d_n * sqrt(L) * C[r_j][n], with d_n and r_j drawn exactly as for the Hadamard variant
     * (counters (n>>7,0,0,2) and (j,0,0,3)): 1 for r_j = 0, else sqrt(2) cos(...), where the cosine is
     * evaluated in fp32: m = (2n+1) r mod 4L (exact integers), quadrant q = m / L, x = (m mod L) / L in
     * [0,1), and cos(pi/2 (q + x)) = c, -s, -c, s for q = 0..3 with s = x * S(x^2), c = C(x^2), S and C the
     * cubics of the Gaussian transform's angle step (Horner, fmaf). */
    uint64_t L = 1;
    int logL = 0;
    while (L < (uint64_t)N) { L <<= 1; ++logL; }
    const float inv_L = bits_f32((uint32_t)(127 - logL) << 23);   /* 2^-logL, exact */
    const float SQRT2 = 0x1.6a09e6p+0f;
    for (int64_t j = j0; j < j1; ++j) {
      uint32_t cj[4] = {(uint32_t)j, 0u, 0u, 3u}, rj[4];
      oracle_philox4x32_10(cj, key, rj);
      const uint64_t r = (uint64_t)rj[0] % L;
      for (int64_t n = 0; n < N; ++n) {
        uint32_t cn[4] = {(uint32_t)(n >> 7), 0u, 0u, 2u}, rn[4];
        oracle_philox4x32_10(cn, key, rn);
        const int t = (int)(n & 127);
        const int d_neg = (int)((rn[t >> 5] >> (t & 31)) & 1u);
        float g = 1.0f;
        if (r != 0) {
          const uint64_t m = ((2u * (uint64_t)n + 1u) * r) & (4u * L - 1u);
          const int q = (int)(m >> logL);
          const float x = (float)(uint32_t)(m & (L - 1u)) * inv_L;
          const float z = x * x;
          const float sp = fmaf(fmaf(fmaf(SIN_C[3], z, SIN_C[2]), z, SIN_C[1]), z, SIN_C[0]);
          const float sn = x * sp;
          const float cs = fmaf(fmaf(fmaf(COS_C[3], z, COS_C[2]), z, COS_C[1]), z, COS_C[0]);
          const float v = (q == 0) ? cs : (q == 1) ? -sn : (q == 2) ? -cs : sn;
          g = SQRT2 * v;
        }
        if (storage == ORACLE_STORE_BF16) g = oracle_bf16_round(g);
        out[n * w + (j - j0)] = d_neg ? -g : g;
      }
    }
    return;
  }
  /* Rademacher */
  const int64_t nblk = (N + 127) / 128;
#pragma omp parallel for schedule(static)
  for (int64_t q = 0; q < nblk; ++q) {
    for (int64_t j = j0; j < j1; ++j) {
      uint32_t ctr[4] = {(uint32_t)q, (uint32_t)j, 0u, 1u}, r[4];
      oracle_philox4x32_10(ctr, key, r);
      for (int t = 0; t < 128; ++t) {
        int64_t n = 128 * q + t;
        if (n >= N) break;
        uint32_t bit = (r[t >> 5] >> (t & 31)) & 1u;
        out[n * w + (j - j0)] = bit ? -1.0f : 1.0f;
      }
    }
  }
}

/* S = c * P as fp64, [N,k] row-major (Eq. 5 for the Gaussian case). */
void oracle_generate_s(uint64_t seed, int64_t N, int64_t k, int dist, int storage, double* S) {
  float* P = (float*)malloc(sizeof(float) * (size_t)N * (size_t)k);
  oracle_generate_p_cols(seed, N, k, 0, k, dist, storage, P);
  const double c = (double)oracle_scale(k, dist);
  for (int64_t i = 0; i < N * k; ++i) S[i] = (double)P[i] * c;
  free(P);
}

/* ---------------------------------------------------------------------------
 * Algorithm 1, FORWARD.  Y = X W^T + 1 b^T (Eq. 1); X_proj = S^T X.
 * X [N,Din], W [Dout,Din], b [Dout] or NULL, S [N,k]; Y [N,Dout], Xproj [k,Din].
 * ------------------------------------------------------------------------- */
void oracle_forward(const double* X, const double* W, const double* b, int64_t N, int64_t Din,
                    int64_t Dout, const double* S, int64_t k, double* Y, double* Xproj) {
  if (Y) {
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n)
      for (int64_t o = 0; o < Dout; ++o) {
        double acc = 0.0;
        for (int64_t i = 0; i < Din; ++i) acc += X[n * Din + i] * W[o * Din + i];
        Y[n * Dout + o] = acc + (b ? b[o] : 0.0);
      }
  }
  if (Xproj) {
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < k; ++j)
      for (int64_t i = 0; i < Din; ++i) {
        double acc = 0.0;
        for (int64_t n = 0; n < N; ++n) acc += S[n * k + j] * X[n * Din + i];
        Xproj[j * Din + i] = acc;
      }
  }
}

/* ---------------------------------------------------------------------------
 * Algorithm 1, BACKWARD.  dX = dY W (Eq. 2); G = S^T dY; dW = G^T X_proj
 * (the association Algorithm 1 fixes: (dY^T S) X_proj); db = dY^T 1 (Eq. 3).
 * dY [N,Dout], W [Dout,Din], Xproj [k,Din], S [N,k];
 * dX [N,Din], dW [Dout,Din], db [Dout], G [k,Dout]; any output may be NULL
 * (dW needs G: if G is NULL a temporary is used).
 * ------------------------------------------------------------------------- */
void oracle_backward(const double* dY, const double* W, const double* Xproj, int64_t N, int64_t Din,
                     int64_t Dout, const double* S, int64_t k, double* dX, double* dW, double* db,
                     double* G) {
  if (dX) {
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n)
      for (int64_t i = 0; i < Din; ++i) {
        double acc = 0.0;
        for (int64_t o = 0; o < Dout; ++o) acc += dY[n * Dout + o] * W[o * Din + i];
        dX[n * Din + i] = acc;
      }
  }
  if (dW || G) {
    double* Gt = G ? G : (double*)malloc(sizeof(double) * (size_t)k * (size_t)Dout);
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < k; ++j)
      for (int64_t o = 0; o < Dout; ++o) {
        double acc = 0.0;
        for (int64_t n = 0; n < N; ++n) acc += S[n * k + j] * dY[n * Dout + o];
        Gt[j * Dout + o] = acc;
      }
    if (dW) {
#pragma omp parallel for schedule(static)
      for (int64_t o = 0; o < Dout; ++o)
        for (int64_t i = 0; i < Din; ++i) {
          double acc = 0.0;
          for (int64_t j = 0; j < k; ++j) acc += Gt[j * Dout + o] * Xproj[j * Din + i];
          dW[o * Din + i] = acc;
        }
    }
    if (!G) free(Gt);
  }
  if (db) {
    for (int64_t o = 0; o < Dout; ++o) {
      double acc = 0.0;
      for (int64_t n = 0; n < N; ++n) acc += dY[n * Dout + o];
      db[o] = acc;
    }
  }
}

/* Exact weight gradient dW* = dY^T X (Eq. 3), [Dout,Din]. */
void oracle_exact_dw(const double* dY, const double* X, int64_t N, int64_t Din, int64_t Dout,
                     double* dW) {
#pragma omp parallel for schedule(static)
  for (int64_t o = 0; o < Dout; ++o)
    for (int64_t i = 0; i < Din; ++i) {
      double acc = 0.0;
      for (int64_t n = 0; n < N; ++n) acc += dY[n * Dout + o] * X[n * Din + i];
      dW[o * Din + i] = acc;
    }
}

/* --- pieces shared by the variance formulas: X [B,Nx], Y [B,My] ------------- */
static double frob2(const double* A, int64_t n) {
  double s = 0.0;
  for (int64_t i = 0; i < n; ++i) s += A[i] * A[i];
  return s;
}
static double xty_frob2(const double* X, const double* Y, int64_t B, int64_t Nx, int64_t My) {
  double s = 0.0;
  for (int64_t a = 0; a < Nx; ++a)
    for (int64_t c = 0; c < My; ++c) {
      double e = 0.0;
      for (int64_t r = 0; r < B; ++r) e += X[r * Nx + a] * Y[r * My + c];
      s += e * e;
    }
  return s;
}
static double rownorm_products(const double* X, const double* Y, int64_t B, int64_t Nx, int64_t My) {
  double s = 0.0;
  for (int64_t r = 0; r < B; ++r) s += frob2(X + r * Nx, Nx) * frob2(Y + r * My, My);
  return s;
}

/* Lemma 1 (Eq. 9): D^2_SGD = B/(B-1) sum_k |x_k|^2 |y_k|^2 - |X^T Y|_F^2 / (B-1). */
double oracle_d2_sgd(const double* X, const double* Y, int64_t B, int64_t Nx, int64_t My) {
  return (double)B / (double)(B - 1) * rownorm_products(X, Y, B, Nx, My) -
         xty_frob2(X, Y, B, Nx, My) / (double)(B - 1);
}

/* Lemma 2 (Eq. 11) exactly as printed: (|X|_F^2 |Y|_F^2 - |X^T Y|_F^2) / B_proj. */
double oracle_d2_rmm_printed(const double* X, const double* Y, int64_t B, int64_t Nx, int64_t My,
                             int64_t Bproj) {
  return (frob2(X, B * Nx) * frob2(Y, B * My) - xty_frob2(X, Y, B, Nx, My)) / (double)Bproj;
}

/* E_S |X^T S S^T Y - X^T Y|_F^2 for iid N(0,1/B_proj) entries, worked out with the
 * Gaussian fourth moment kept (the i = j case of the proof of Lemma 2 uses
 * E[C^4] = 3 E[C^2]^2): (|X|_F^2 |Y|_F^2 + |X^T Y|_F^2) / B_proj. */
double oracle_d2_rmm_gaussian(const double* X, const double* Y, int64_t B, int64_t Nx, int64_t My,
                              int64_t Bproj) {
  return (frob2(X, B * Nx) * frob2(Y, B * My) + xty_frob2(X, Y, B, Nx, My)) / (double)Bproj;
}

/* Same expectation for iid +-1/sqrt(B_proj) entries (fourth moment = second moment
 * squared): (|X|^2|Y|^2 + |X^T Y|^2 - 2 sum_n |x_n|^2 |y_n|^2) / B_proj. */
double oracle_d2_rmm_rademacher(const double* X, const double* Y, int64_t B, int64_t Nx, int64_t My,
                                int64_t Bproj) {
  return (frob2(X, B * Nx) * frob2(Y, B * My) + xty_frob2(X, Y, B, Nx, My) -
          2.0 * rownorm_products(X, Y, B, Nx, My)) / (double)Bproj;
}

/* Theorem 1 (Eq. 13): alpha = |X^T Y|_F^2 / (|X|_F^2 |Y|_F^2). */
double oracle_alpha(const double* X, const double* Y, int64_t B, int64_t Nx, int64_t My) {
  return xty_frob2(X, Y, B, Nx, My) / (frob2(X, B * Nx) * frob2(Y, B * My));
}
