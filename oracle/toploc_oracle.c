/*
 * toploc_oracle.c -- slow, plain CPU statement of the TopLoc proof path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the parity reference for the CUDA
 * library and the timed CPU baseline of the benchmark; nothing on the product
 * path may call it, and it shares no code, header, table or constant with the
 * CUDA side.  Every routine is written for being checked by eye against the
 * paper, not for speed: a full sort for top-k, a brute-force modulus search,
 * Gaussian elimination on the Vandermonde system for the interpolant.
 *
 * Readings of points the paper leaves open (each is repeated where it is used):
 *   - ranking key: the bit pattern with the sign bit cleared, compared as an
 *     unsigned integer; ties go to the lower flat index;
 *   - field prime p = 65521, the largest prime below 2^16 (Algorithm 3 needs a
 *     prime modulus, Section 4 fixes 2-byte coefficients);
 *   - a candidate modulus m is accepted only if (index mod m) mod p is
 *     injective, because m may exceed p;
 *   - proof layout: m & 0xFFFF little-endian (0 means 65536), then the k
 *     coefficients in ascending degree, 2 bytes little-endian each;
 *   - fp32 activations rank on the 31-bit magnitude and commit the upper 16
 *     bits of the pattern (Section 5.6, mantissa scaled to bf16), or, in the
 *     32-bit field variant further down (dtype code 2 of the batch drivers),
 *     the whole pattern over Z_q, q = 2^32 - 5; dtype code 3 validates fp32
 *     activations against a 16-bit field proof padded with 16 zero bits;
 *   - direct commitments (Section 4's 6 bytes per point, for k beyond what
 *     Algorithm 6 can serve): records in ascending index order, an index
 *     that was not committed counts as an exponent mismatch.
 *
 * Pins (tests/test_oracle_*.py): worked examples and the paper's printed
 * values under tests/golden/, brute force on tiny inputs, P(x_j) = y_j with
 * Python integers, exhaustive a * inverse(a) = 1, Lagrange's form against
 * elimination, the modulus distribution of Table 11.  Unpinned: byte
 * compatibility with the upstream project's proofs (its code is not
 * available here) -- "parity unpinned" for that claim only.
 */
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define P_FIELD 65521u /* largest prime below 2^16 */
#define M_HIGH 65536u  /* Algorithm 6 tries 65536 first and stops after 2^15 + 1 */
#define M_LOW 32769u

enum { ST_OK = 0, ST_NO_MODULUS = 1, ST_K_EXCEEDS = 2, ST_BAD_PROOF = 3, ST_NONFINITE = 4 };

typedef struct {
  uint32_t exp_mismatch;
  uint32_t n_match;
  uint32_t mant_diff_sum;
  int32_t topk_mismatch;
  double mant_mean;
  double mant_median;
  uint32_t modulus;
  uint8_t accept;
  uint8_t status;
  uint8_t pad[2];
} oracle_result;

/* ------------------------------------------------------------------ */
/* topk(h, k) of Algorithm 1; Section 5.3 ranks by magnitude. */
/* ------------------------------------------------------------------ */

typedef struct {
  uint32_t key;  /* magnitude: pattern without its sign bit */
  uint32_t flat; /* token_in_chunk * hidden + channel */
  uint16_t bits; /* the 16-bit pattern that gets committed */
} ranked;

static int by_magnitude_then_index(const void* a, const void* b) {
  const ranked* p = (const ranked*)a;
  const ranked* q = (const ranked*)b;
  if (p->key != q->key) return p->key > q->key ? -1 : 1; /* larger magnitude first */
  if (p->flat != q->flat) return p->flat < q->flat ? -1 : 1; /* then lower index */
  return 0;
}

/* chunk: first element of the chunk's first row; rows x hidden elements,
 * row_stride elements between rows.  dtype 0 = bf16 (uint16 patterns),
 * 1 = fp32 (uint32 patterns).  Writes k indices and 16-bit patterns in rank
 * order.  Returns ST_OK or ST_K_EXCEEDS. */
int oracle_topk(const void* chunk, int dtype, int rows, int hidden, int64_t row_stride, int k,
                uint32_t* idx_out, uint16_t* bits_out) {
  int64_t n = (int64_t)rows * hidden;
  if (k > n) return ST_K_EXCEEDS;
  ranked* all = (ranked*)malloc((size_t)n * sizeof(ranked));
  for (int t = 0; t < rows; ++t) {
    for (int c = 0; c < hidden; ++c) {
      ranked* r = &all[(int64_t)t * hidden + c];
      r->flat = (uint32_t)((int64_t)t * hidden + c);
      if (dtype == 0) {
        uint16_t v = ((const uint16_t*)chunk)[(int64_t)t * row_stride + c];
        r->key = v & 0x7FFFu;
        r->bits = v;
      } else {
        uint32_t v = ((const uint32_t*)chunk)[(int64_t)t * row_stride + c];
        r->key = v & 0x7FFFFFFFu;
        r->bits = (uint16_t)(v >> 16);
      }
    }
  }
  qsort(all, (size_t)n, sizeof(ranked), by_magnitude_then_index);
  for (int j = 0; j < k; ++j) {
    idx_out[j] = all[j].flat;
    bits_out[j] = all[j].bits;
  }
  free(all);
  return ST_OK;
}

/* ------------------------------------------------------------------ */
/* Algorithm 6, Find Injective Modulus.                                */
/* ------------------------------------------------------------------ */

/* Largest m in [2^15+1, 2^16] such that the residues are pairwise distinct.
 * field_distinct != 0: the residues compared are (idx mod m) mod p (the
 * reading used by the proof path, since two residues below m can differ by
 * exactly p); 0: idx mod m, Algorithm 6 as printed.  Returns 0 when no
 * candidate works (the algorithm's "raise"). */
uint32_t oracle_find_injective_modulus(const uint32_t* idx, int k, int field_distinct) {
  uint32_t* r = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
  uint32_t found = 0;
  for (uint32_t m = M_HIGH; m >= M_LOW && !found; --m) {
    for (int j = 0; j < k; ++j) {
      r[j] = idx[j] % m;
      if (field_distinct) r[j] %= P_FIELD;
    }
    int injective = 1;
    for (int a = 0; a < k && injective; ++a)
      for (int b = a + 1; b < k; ++b)
        if (r[a] == r[b]) {
          injective = 0;
          break;
        }
    if (injective) found = m;
  }
  free(r);
  return found;
}

/* ------------------------------------------------------------------ */
/* Arithmetic in Z_p.                                                  */
/* ------------------------------------------------------------------ */

static uint32_t mulp(uint32_t a, uint32_t b) { return (uint32_t)(((uint64_t)a * b) % P_FIELD); }
static uint32_t addp(uint32_t a, uint32_t b) { return (a + b) % P_FIELD; }
static uint32_t subp(uint32_t a, uint32_t b) { return (a + P_FIELD - b) % P_FIELD; }

/* Inverse in Z_p by Fermat's little theorem, a^(p-2).  (Algorithm 4 uses the
 * extended Euclidean algorithm; the inverse is unique, so the method is
 * free.)  a must be in [1, p). */
uint32_t oracle_mod_inverse(uint32_t a) {
  uint32_t result = 1, base = a % P_FIELD;
  uint32_t e = P_FIELD - 2;
  while (e) {
    if (e & 1u) result = mulp(result, base);
    base = mulp(base, base);
    e >>= 1;
  }
  return result;
}

/* The inverse by the extended Euclidean method (the method of Algorithm 4),
 * stated through the recursion  gcd(a, b) = gcd(b, a mod b):  if
 * g = b s' + (a mod b) t'  then  g = a t' + b (s' - floor(a / b) t').
 * bezout() returns g and the two cofactors. */
static int64_t bezout(int64_t a, int64_t b, int64_t* s, int64_t* t) {
  if (b == 0) {
    *s = 1;
    *t = 0;
    return a;
  }
  int64_t s1, t1;
  int64_t g = bezout(b, a % b, &s1, &t1);
  *s = t1;
  *t = s1 - (a / b) * t1;
  return g;
}

/* Inverse of a modulo m in [0, m).  Returns 0 when m <= 1 (no ring to invert
 * in) and m itself, an impossible inverse, when gcd(a, m) != 1: the two cases
 * in which Algorithm 4 has nothing to return. */
int64_t oracle_mod_inverse_euclid(int64_t a, int64_t m) {
  if (m <= 1) return 0;
  int64_t s, t;
  a %= m;
  if (a < 0) a += m;
  if (bezout(a, m, &s, &t) != 1) return m;
  s %= m;
  return s < 0 ? s + m : s;
}

/* Algorithm 5, Horner: c[0..k-1] ascending degree, result in [0, p). */
uint32_t oracle_horner(const uint16_t* c, int k, uint32_t x) {
  uint32_t acc = c[k - 1] % P_FIELD;
  x %= P_FIELD;
  for (int d = k - 2; d >= 0; --d) acc = addp(mulp(acc, x), c[d] % P_FIELD);
  return acc;
}

/* ------------------------------------------------------------------ */
/* Section 4 relies on the interpolant being unique: k points with     */
/* distinct x fix one polynomial of degree below k.  It solves the     */
/* Vandermonde system  sum_d c_d x_j^d = y_j  over Z_p; solved here by  */
/* Gaussian elimination.  x must be pairwise distinct mod p.           */
/* Returns 0 on success, 1 if the system is singular.                  */
/* ------------------------------------------------------------------ */
int oracle_interpolate(const uint32_t* x, const uint32_t* y, int k, uint16_t* c) {
  int w = k + 1;
  uint32_t* a = (uint32_t*)malloc((size_t)k * w * sizeof(uint32_t));
  for (int j = 0; j < k; ++j) {
    uint32_t pw = 1, xj = x[j] % P_FIELD;
    for (int d = 0; d < k; ++d) {
      a[j * w + d] = pw;
      pw = mulp(pw, xj);
    }
    a[j * w + k] = y[j] % P_FIELD;
  }
  /* forward elimination to upper-triangular with unit diagonal */
  for (int col = 0; col < k; ++col) {
    int piv = -1;
    for (int r = col; r < k; ++r)
      if (a[r * w + col] != 0) {
        piv = r;
        break;
      }
    if (piv < 0) {
      free(a);
      return 1;
    }
    if (piv != col)
      for (int d = 0; d < w; ++d) {
        uint32_t t = a[col * w + d];
        a[col * w + d] = a[piv * w + d];
        a[piv * w + d] = t;
      }
    uint32_t inv = oracle_mod_inverse(a[col * w + col]);
    for (int d = col; d < w; ++d) a[col * w + d] = mulp(a[col * w + d], inv);
    for (int r = col + 1; r < k; ++r) {
      uint32_t f = a[r * w + col];
      if (f == 0) continue;
      for (int d = col; d < w; ++d) a[r * w + d] = subp(a[r * w + d], mulp(f, a[col * w + d]));
    }
  }
  /* back substitution */
  uint32_t* sol = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
  for (int row = k - 1; row >= 0; --row) {
    uint32_t s = a[row * w + k];
    for (int d = row + 1; d < k; ++d) s = subp(s, mulp(a[row * w + d], sol[d]));
    sol[row] = s;
  }
  for (int d = 0; d < k; ++d) c[d] = (uint16_t)sol[d];
  free(sol);
  free(a);
  return 0;
}

/* A second statement of the same polynomial, kept beside the elimination as a
 * pin (the two must agree because the interpolant is unique, Section 4):
 * Lagrange's form
 *   P(x) = sum_j y_j L_j(x),   L_j(x) = prod_{i != j} (x - x_i) / (x_j - x_i).
 * The master polynomial M(x) = prod_i (x - x_i) is multiplied out once; for
 * every j the quotient Q_j = M / (x - x_j) comes from one synthetic division
 * and the denominator is Q_j(x_j).  Inverses by the extended Euclidean routine.
 * (The CUDA path uses Newton's divided differences, Algorithm 3: a third
 * route to the same coefficients.)  Returns 1 if two x coincide mod p. */
int oracle_interpolate_lagrange(const uint32_t* x, const uint32_t* y, int k, uint16_t* c) {
  uint32_t* master = (uint32_t*)calloc((size_t)k + 1, sizeof(uint32_t));
  uint32_t* quot = (uint32_t*)calloc((size_t)k, sizeof(uint32_t));
  uint32_t* sum = (uint32_t*)calloc((size_t)k, sizeof(uint32_t));
  int failed = 0;
  master[0] = 1; /* the constant polynomial 1, then one factor (x - x_i) at a time */
  for (int i = 0; i < k; ++i) {
    uint32_t xi = x[i] % P_FIELD;
    for (int d = i + 1; d >= 1; --d) master[d] = subp(master[d - 1], mulp(master[d], xi));
    master[0] = subp(0, mulp(master[0], xi));
  }
  for (int j = 0; j < k && !failed; ++j) {
    uint32_t xj = x[j] % P_FIELD;
    /* M = (x - x_j) Q_j:  q_{k-1} = M_k,  q_{d-1} = M_d + x_j q_d */
    quot[k - 1] = master[k];
    for (int d = k - 1; d >= 1; --d) quot[d - 1] = addp(master[d], mulp(xj, quot[d]));
    uint32_t den = 0; /* Q_j(x_j) = prod_{i != j} (x_j - x_i) */
    for (int d = k - 1; d >= 0; --d) den = addp(mulp(den, xj), quot[d]);
    int64_t inv = oracle_mod_inverse_euclid((int64_t)den, (int64_t)P_FIELD);
    if (den == 0 || inv == (int64_t)P_FIELD) {
      failed = 1;
      break;
    }
    uint32_t w = mulp(y[j] % P_FIELD, (uint32_t)inv);
    for (int d = 0; d < k; ++d) sum[d] = addp(sum[d], mulp(w, quot[d]));
  }
  if (!failed)
    for (int d = 0; d < k; ++d) c[d] = (uint16_t)sum[d];
  free(master);
  free(quot);
  free(sum);
  return failed;
}

/* ------------------------------------------------------------------ */
/* encode / decode (Algorithm 1 last step, Algorithm 2 first step).    */
/* 2 + 2k bytes: Section 4 (2-byte coefficients), Section 5.7 (256 B of */
/* coefficients per interval), abstract (258 B).                       */
/* ------------------------------------------------------------------ */
void oracle_encode(uint32_t m, const uint16_t* c, int k, uint8_t* proof) {
  uint32_t m16 = m & 0xFFFFu; /* 65536 -> 0 */
  proof[0] = (uint8_t)(m16 & 0xFF);
  proof[1] = (uint8_t)(m16 >> 8);
  for (int d = 0; d < k; ++d) {
    proof[2 + 2 * d] = (uint8_t)(c[d] & 0xFF);
    proof[3 + 2 * d] = (uint8_t)(c[d] >> 8);
  }
}

/* Returns ST_OK or ST_BAD_PROOF (odd or too short length, modulus outside
 * the search range, a coefficient >= p).  *k_out = (len - 2) / 2. */
int oracle_decode(const uint8_t* proof, int64_t len, int* k_out, uint32_t* m_out, uint16_t* c) {
  if (len < 4 || (len & 1)) return ST_BAD_PROOF;
  int k = (int)((len - 2) / 2);
  uint32_t m = (uint32_t)proof[0] | ((uint32_t)proof[1] << 8);
  if (m == 0) m = 65536u;
  *k_out = k;
  *m_out = m;
  int bad = (m < M_LOW || m > M_HIGH);
  for (int d = 0; d < k; ++d) {
    c[d] = (uint16_t)(proof[2 + 2 * d] | (proof[3 + 2 * d] << 8));
    if (c[d] >= P_FIELD) bad = 1;
  }
  return bad ? ST_BAD_PROOF : ST_OK;
}

/* ------------------------------------------------------------------ */
/* Algorithm 1 for one chunk.                                          */
/* ------------------------------------------------------------------ */
/* Algorithm 1 after its topk line: idx / bits are the k selected elements in rank order. */
static int build_from_selection(const uint32_t* idx, const uint16_t* bits, int k, uint8_t* proof,
                                int32_t* indices_opt) {
  uint32_t* xs = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
  uint32_t* ys = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
  uint16_t* coef = (uint16_t*)malloc((size_t)k * sizeof(uint16_t));
  int status = ST_OK;
  if (indices_opt)
    for (int j = 0; j < k; ++j) indices_opt[j] = (int32_t)idx[j];
  uint32_t m = oracle_find_injective_modulus(idx, k, 1);
  if (m == 0) {
    status = ST_NO_MODULUS;
  } else {
    for (int j = 0; j < k; ++j) {
      xs[j] = (idx[j] % m) % P_FIELD;
      ys[j] = (uint32_t)bits[j] % P_FIELD; /* Algorithm 3 reduces every y mod M first */
      if (bits[j] >= P_FIELD) status = ST_NONFINITE;
    }
    oracle_interpolate(xs, ys, k, coef);
    oracle_encode(m, coef, k, proof);
  }
  free(xs);
  free(ys);
  free(coef);
  return status;
}

int oracle_build_chunk(const void* chunk, int dtype, int rows, int hidden, int64_t row_stride, int k,
                       uint8_t* proof, int32_t* indices_opt) {
  size_t nbytes = 2 + 2 * (size_t)k;
  memset(proof, 0, nbytes);
  if (indices_opt) memset(indices_opt, 0, (size_t)k * sizeof(int32_t));
  uint32_t* idx = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
  uint16_t* bits = (uint16_t*)malloc((size_t)k * sizeof(uint16_t));
  int status = oracle_topk(chunk, dtype, rows, hidden, row_stride, k, idx, bits);
  if (status == ST_OK) status = build_from_selection(idx, bits, k, proof, indices_opt);
  free(idx);
  free(bits);
  return status;
}

static int ascending_u32(const void* a, const void* b) {
  uint32_t p = *(const uint32_t*)a, q = *(const uint32_t*)b;
  return p < q ? -1 : (p > q ? 1 : 0);
}

/* ------------------------------------------------------------------ */
/* Algorithm 2 for one chunk.  Thresholds: Section 5.2.                */
/* 16-bit pattern: bit 15 sign, bits 14..7 exponent, bits 6..0         */
/* mantissa (bf16 has 7 mantissa bits, Section 5.2).                   */
/* ------------------------------------------------------------------ */
/* Algorithm 2 from its second line on.  select: the topk line -- either sorts the chunk (chunk
 * != NULL) or, when the caller has already ranked the chunk's elements, takes the first k of that
 * ranking (ranked_idx / ranked_bits hold at least k entries, or n_ranked < k of them when the
 * chunk has fewer than k elements). */
static void verify_with_selection(const void* chunk, int dtype, int rows, int hidden, int64_t row_stride,
                                  const uint32_t* ranked_idx, const uint16_t* ranked_bits, int64_t n_ranked, int k,
                                  const uint8_t* proof, int t_exp, double t_mean, double t_median,
                                  int sign_in_exponent, const int32_t* gen_indices_opt, oracle_result* out) {
  memset(out, 0, sizeof(*out));
  out->topk_mismatch = -1;
  uint32_t* idx = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
  uint16_t* bits = (uint16_t*)malloc((size_t)k * sizeof(uint16_t));
  uint16_t* coef = (uint16_t*)malloc((size_t)k * sizeof(uint16_t));
  uint32_t* diffs = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
  int kk = 0;
  uint32_t m = 0;
  int status = oracle_decode(proof, 2 + 2 * (int64_t)k, &kk, &m, coef);
  out->modulus = m;
  if (status == ST_OK) {
    if (chunk != NULL) {
      status = oracle_topk(chunk, dtype, rows, hidden, row_stride, k, idx, bits);
    } else if (n_ranked < k) {
      status = ST_K_EXCEEDS;
    } else {
      memcpy(idx, ranked_idx, (size_t)k * sizeof(uint32_t));
      memcpy(bits, ranked_bits, (size_t)k * sizeof(uint16_t));
    }
  }
  if (status == ST_OK) {
    uint32_t err_e = 0, n = 0, sum = 0;
    for (int j = 0; j < k; ++j) {
      uint32_t xj = (idx[j] % m) % P_FIELD;
      uint32_t committed = oracle_horner(coef, k, xj); /* P[i_m[j]] */
      uint32_t seen = bits[j];
      uint32_t e_p, e_v;
      if (sign_in_exponent) {
        e_p = committed >> 7; /* sign + exponent, 9 bits */
        e_v = seen >> 7;
      } else {
        e_p = (committed >> 7) & 0xFFu;
        e_v = (seen >> 7) & 0xFFu;
      }
      uint32_t m_p = committed & 0x7Fu, m_v = seen & 0x7Fu;
      if (e_p == e_v) {
        uint32_t d = m_p > m_v ? m_p - m_v : m_v - m_p;
        diffs[n++] = d;
        sum += d;
      } else {
        ++err_e;
      }
    }
    out->exp_mismatch = err_e;
    out->n_match = n;
    out->mant_diff_sum = sum;
    if (n > 0) {
      out->mant_mean = (double)sum / (double)n;
      qsort(diffs, n, sizeof(uint32_t), ascending_u32);
      out->mant_median = (n & 1u) ? (double)diffs[n / 2] : ((double)diffs[n / 2 - 1] + (double)diffs[n / 2]) / 2.0;
    }
    int reject = ((int64_t)err_e > (int64_t)t_exp) || (out->mant_mean > t_mean) || (out->mant_median > t_median);
    if (n == 0) reject = 1; /* nothing matched: no statistic to accept on */
    out->accept = reject ? 0 : 1;
    if (gen_indices_opt) {
      int common = 0;
      for (int a = 0; a < k; ++a)
        for (int b = 0; b < k; ++b)
          if ((uint32_t)gen_indices_opt[a] == idx[b]) {
            ++common;
            break;
          }
      out->topk_mismatch = k - common;
    }
  }
  out->status = (uint8_t)status;
  if (status != ST_OK) out->accept = 0;
  free(idx);
  free(bits);
  free(coef);
  free(diffs);
}

void oracle_verify_chunk(const void* chunk, int dtype, int rows, int hidden, int64_t row_stride, int k,
                         const uint8_t* proof, int t_exp, double t_mean, double t_median,
                         int sign_in_exponent, const int32_t* gen_indices_opt, oracle_result* out) {
  verify_with_selection(chunk, dtype, rows, hidden, row_stride, NULL, NULL, 0, k, proof, t_exp, t_mean, t_median,
                        sign_in_exponent, gen_indices_opt, out);
}

/* ================================================================== */
/* 32-bit field variant: an fp32 chunk commits the full 32-bit pattern */
/* of each selected value.  The paper uses it without printing its     */
/* layout: Section 5.2 gives thresholds for fp32 inference (8 / 256 /   */
/* 128, on 23-bit mantissas, cf. the fp32 rows of the precision table   */
/* in Section 5.6), and the subroutines appendix puts the modulus of   */
/* 32-bit types at 2^32.  Readings used here:                          */
/*   - field prime q = 4294967291 = 2^32 - 5, the largest prime below  */
/*     2^32 (a prime that fits 4-byte coefficients, as p fits 2 bytes); */
/*   - proof: the same 2 modulus bytes, then k coefficients of 4 bytes  */
/*     little-endian, ascending degree: 2 + 4k bytes;                  */
/*   - x = index mod m needs no second reduction (m <= 2^16 < q), so    */
/*     Algorithm 6 applies as printed;                                 */
/*   - y = the 32-bit pattern mod q; the five patterns >= q (negative   */
/*     NaNs) are flagged like their 16-bit counterparts;               */
/*   - extractBits: bit 31 sign, bits 30..23 exponent, bits 22..0       */
/*     mantissa (fp32 has 23 mantissa bits, Section 5.2).              */
/* Everything else (ranking, ties, statistics, verdict) is as above.   */
/* ================================================================== */
#define Q_FIELD 4294967291u

static uint32_t mulq(uint32_t a, uint32_t b) { return (uint32_t)(((uint64_t)a * b) % Q_FIELD); }
static uint32_t addq(uint32_t a, uint32_t b) { return (uint32_t)(((uint64_t)a + b) % Q_FIELD); }
static uint32_t subq(uint32_t a, uint32_t b) { return (uint32_t)(((uint64_t)a + Q_FIELD - b) % Q_FIELD); }

/* a^(q-2) in Z_q; a in [1, q). */
uint32_t oracle_mod_inverse32(uint32_t a) {
  uint32_t result = 1, base = a % Q_FIELD;
  uint32_t e = Q_FIELD - 2;
  while (e) {
    if (e & 1u) result = mulq(result, base);
    base = mulq(base, base);
    e >>= 1;
  }
  return result;
}

/* Algorithm 5 over Z_q. */
uint32_t oracle_horner32(const uint32_t* c, int k, uint32_t x) {
  uint32_t acc = c[k - 1] % Q_FIELD;
  x %= Q_FIELD;
  for (int d = k - 2; d >= 0; --d) acc = addq(mulq(acc, x), c[d] % Q_FIELD);
  return acc;
}

/* The unique interpolant over Z_q: Gaussian elimination on the Vandermonde
 * system, as oracle_interpolate.  Returns 1 if the system is singular. */
int oracle_interpolate32(const uint32_t* x, const uint32_t* y, int k, uint32_t* c) {
  int w = k + 1;
  uint32_t* a = (uint32_t*)malloc((size_t)k * w * sizeof(uint32_t));
  for (int j = 0; j < k; ++j) {
    uint32_t pw = 1, xj = x[j] % Q_FIELD;
    for (int d = 0; d < k; ++d) {
      a[j * w + d] = pw;
      pw = mulq(pw, xj);
    }
    a[j * w + k] = y[j] % Q_FIELD;
  }
  for (int col = 0; col < k; ++col) {
    int piv = -1;
    for (int r = col; r < k; ++r)
      if (a[r * w + col] != 0) {
        piv = r;
        break;
      }
    if (piv < 0) {
      free(a);
      return 1;
    }
    if (piv != col)
      for (int d = 0; d < w; ++d) {
        uint32_t t = a[col * w + d];
        a[col * w + d] = a[piv * w + d];
        a[piv * w + d] = t;
      }
    uint32_t inv = oracle_mod_inverse32(a[col * w + col]);
    for (int d = col; d < w; ++d) a[col * w + d] = mulq(a[col * w + d], inv);
    for (int r = col + 1; r < k; ++r) {
      uint32_t f = a[r * w + col];
      if (f == 0) continue;
      for (int d = col; d < w; ++d) a[r * w + d] = subq(a[r * w + d], mulq(f, a[col * w + d]));
    }
  }
  for (int row = k - 1; row >= 0; --row) {
    uint32_t s = a[row * w + k];
    for (int d = row + 1; d < k; ++d) s = subq(s, mulq(a[row * w + d], c[d]));
    c[row] = s;
  }
  free(a);
  return 0;
}

/* Lagrange's form over Z_q (see oracle_interpolate_lagrange): the second
 * statement of the same polynomial. */
int oracle_interpolate32_lagrange(const uint32_t* x, const uint32_t* y, int k, uint32_t* c) {
  uint32_t* master = (uint32_t*)calloc((size_t)k + 1, sizeof(uint32_t));
  uint32_t* quot = (uint32_t*)calloc((size_t)k, sizeof(uint32_t));
  uint32_t* sum = (uint32_t*)calloc((size_t)k, sizeof(uint32_t));
  int failed = 0;
  master[0] = 1;
  for (int i = 0; i < k; ++i) {
    uint32_t xi = x[i] % Q_FIELD;
    for (int d = i + 1; d >= 1; --d) master[d] = subq(master[d - 1], mulq(master[d], xi));
    master[0] = subq(0, mulq(master[0], xi));
  }
  for (int j = 0; j < k && !failed; ++j) {
    uint32_t xj = x[j] % Q_FIELD;
    quot[k - 1] = master[k];
    for (int d = k - 1; d >= 1; --d) quot[d - 1] = addq(master[d], mulq(xj, quot[d]));
    uint32_t den = 0;
    for (int d = k - 1; d >= 0; --d) den = addq(mulq(den, xj), quot[d]);
    int64_t inv = oracle_mod_inverse_euclid((int64_t)den, (int64_t)Q_FIELD);
    if (den == 0 || inv == (int64_t)Q_FIELD) {
      failed = 1;
      break;
    }
    uint32_t w = mulq(y[j] % Q_FIELD, (uint32_t)inv);
    for (int d = 0; d < k; ++d) sum[d] = addq(sum[d], mulq(w, quot[d]));
  }
  if (!failed)
    for (int d = 0; d < k; ++d) c[d] = sum[d];
  free(master);
  free(quot);
  free(sum);
  return failed;
}

/* 2 + 4k bytes. */
void oracle_encode32(uint32_t m, const uint32_t* c, int k, uint8_t* proof) {
  uint32_t m16 = m & 0xFFFFu; /* 65536 -> 0 */
  proof[0] = (uint8_t)(m16 & 0xFF);
  proof[1] = (uint8_t)(m16 >> 8);
  for (int d = 0; d < k; ++d)
    for (int b = 0; b < 4; ++b) proof[2 + 4 * d + b] = (uint8_t)(c[d] >> (8 * b));
}

/* ST_OK or ST_BAD_PROOF (length not 2 + 4k, modulus outside the search
 * range, a coefficient >= q).  *k_out = (len - 2) / 4. */
int oracle_decode32(const uint8_t* proof, int64_t len, int* k_out, uint32_t* m_out, uint32_t* c) {
  if (len < 6 || ((len - 2) & 3)) return ST_BAD_PROOF;
  int k = (int)((len - 2) / 4);
  uint32_t m = (uint32_t)proof[0] | ((uint32_t)proof[1] << 8);
  if (m == 0) m = 65536u;
  *k_out = k;
  *m_out = m;
  int bad = (m < M_LOW || m > M_HIGH);
  for (int d = 0; d < k; ++d) {
    c[d] = 0;
    for (int b = 0; b < 4; ++b) c[d] |= (uint32_t)proof[2 + 4 * d + b] << (8 * b);
    if (c[d] >= Q_FIELD) bad = 1;
  }
  return bad ? ST_BAD_PROOF : ST_OK;
}

/* top-k of an fp32 chunk with the full patterns of the selected elements. */
static int topk_patterns32(const void* chunk, int rows, int hidden, int64_t row_stride, int k, uint32_t* idx,
                           uint32_t* pattern) {
  uint16_t* upper = (uint16_t*)malloc((size_t)k * sizeof(uint16_t));
  int status = oracle_topk(chunk, 1, rows, hidden, row_stride, k, idx, upper);
  free(upper);
  if (status != ST_OK) return status;
  for (int j = 0; j < k; ++j) {
    int64_t t = idx[j] / (uint32_t)hidden, col = idx[j] % (uint32_t)hidden;
    pattern[j] = ((const uint32_t*)chunk)[t * row_stride + col];
  }
  return ST_OK;
}

/* Algorithm 1 for one fp32 chunk over Z_q. */
int oracle_build_chunk32(const void* chunk, int rows, int hidden, int64_t row_stride, int k, uint8_t* proof,
                         int32_t* indices_opt) {
  memset(proof, 0, 2 + 4 * (size_t)k);
  if (indices_opt) memset(indices_opt, 0, (size_t)k * sizeof(int32_t));
  uint32_t* idx = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
  uint32_t* pattern = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
  uint32_t* xs = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
  uint32_t* ys = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
  uint32_t* coef = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
  int status = topk_patterns32(chunk, rows, hidden, row_stride, k, idx, pattern);
  if (status == ST_OK) {
    if (indices_opt)
      for (int j = 0; j < k; ++j) indices_opt[j] = (int32_t)idx[j];
    uint32_t m = oracle_find_injective_modulus(idx, k, 0); /* residues below 2^16 are distinct in Z_q */
    if (m == 0) {
      status = ST_NO_MODULUS;
    } else {
      for (int j = 0; j < k; ++j) {
        xs[j] = idx[j] % m;
        ys[j] = pattern[j] % Q_FIELD;
        if (pattern[j] >= Q_FIELD) status = ST_NONFINITE;
      }
      oracle_interpolate32(xs, ys, k, coef);
      oracle_encode32(m, coef, k, proof);
    }
  }
  free(idx);
  free(pattern);
  free(xs);
  free(ys);
  free(coef);
  return status;
}

/* Algorithm 2 for one fp32 chunk over Z_q (thresholds of Section 5.2 for
 * fp32 inference: 8 / 256 / 128 at k = 128). */
void oracle_verify_chunk32(const void* chunk, int rows, int hidden, int64_t row_stride, int k,
                           const uint8_t* proof, int t_exp, double t_mean, double t_median,
                           int sign_in_exponent, const int32_t* gen_indices_opt, oracle_result* out) {
  memset(out, 0, sizeof(*out));
  out->topk_mismatch = -1;
  uint32_t* idx = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
  uint32_t* pattern = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
  uint32_t* coef = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
  uint32_t* diffs = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
  int kk = 0;
  uint32_t m = 0;
  int status = oracle_decode32(proof, 2 + 4 * (int64_t)k, &kk, &m, coef);
  out->modulus = m;
  if (status == ST_OK) status = topk_patterns32(chunk, rows, hidden, row_stride, k, idx, pattern);
  if (status == ST_OK) {
    uint32_t err_e = 0, n = 0;
    uint64_t sum = 0;
    for (int j = 0; j < k; ++j) {
      uint32_t committed = oracle_horner32(coef, k, idx[j] % m);
      uint32_t seen = pattern[j];
      uint32_t e_p = committed >> 23, e_v = seen >> 23; /* sign + exponent, 9 bits */
      if (!sign_in_exponent) {
        e_p &= 0xFFu;
        e_v &= 0xFFu;
      }
      uint32_t m_p = committed & 0x7FFFFFu, m_v = seen & 0x7FFFFFu;
      if (e_p == e_v) {
        uint32_t d = m_p > m_v ? m_p - m_v : m_v - m_p;
        diffs[n++] = d;
        sum += d;
      } else {
        ++err_e;
      }
    }
    out->exp_mismatch = err_e;
    out->n_match = n;
    out->mant_diff_sum = (uint32_t)sum; /* k <= 256 differences below 2^23 */
    if (n > 0) {
      out->mant_mean = (double)sum / (double)n;
      qsort(diffs, n, sizeof(uint32_t), ascending_u32);
      out->mant_median = (n & 1u) ? (double)diffs[n / 2] : ((double)diffs[n / 2 - 1] + (double)diffs[n / 2]) / 2.0;
    }
    int reject = ((int64_t)err_e > (int64_t)t_exp) || (out->mant_mean > t_mean) || (out->mant_median > t_median);
    if (n == 0) reject = 1;
    out->accept = reject ? 0 : 1;
    if (gen_indices_opt) {
      int common = 0;
      for (int a = 0; a < k; ++a)
        for (int b = 0; b < k; ++b)
          if ((uint32_t)gen_indices_opt[a] == idx[b]) {
            ++common;
            break;
          }
      out->topk_mismatch = k - common;
    }
  }
  out->status = (uint8_t)status;
  if (status != ST_OK) out->accept = 0;
  free(idx);
  free(pattern);
  free(coef);
  free(diffs);
}

/* Algorithm 2 for an fp32 validator against the proof of a bf16 generator
 * (Section 5.6 validates a bf16 model in fp32 by widening each bf16 pattern
 * with 16 zero bits).  The proof is an ordinary 16-bit
 * field proof; the validator ranks its fp32 chunk on the full magnitude,
 * evaluates the polynomial over Z_p, pads the committed 16-bit pattern with 16
 * zero bits and compares fp32 bit fields (23-bit mantissas), which is what the
 * fp32 thresholds of Section 5.2 apply to. */
void oracle_verify_chunk_padded(const void* chunk, int rows, int hidden, int64_t row_stride, int k,
                                const uint8_t* proof, int t_exp, double t_mean, double t_median,
                                int sign_in_exponent, const int32_t* gen_indices_opt, oracle_result* out) {
  memset(out, 0, sizeof(*out));
  out->topk_mismatch = -1;
  uint32_t* idx = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
  uint32_t* pattern = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
  uint16_t* coef = (uint16_t*)malloc((size_t)k * sizeof(uint16_t));
  uint32_t* diffs = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
  int kk = 0;
  uint32_t m = 0;
  int status = oracle_decode(proof, 2 + 2 * (int64_t)k, &kk, &m, coef);
  out->modulus = m;
  if (status == ST_OK) status = topk_patterns32(chunk, rows, hidden, row_stride, k, idx, pattern);
  if (status == ST_OK) {
    uint32_t err_e = 0, n = 0;
    uint64_t sum = 0;
    for (int j = 0; j < k; ++j) {
      uint32_t committed = oracle_horner(coef, k, (idx[j] % m) % P_FIELD) << 16; /* padded with 16 zero bits */
      uint32_t seen = pattern[j];
      uint32_t e_p = committed >> 23, e_v = seen >> 23;
      if (!sign_in_exponent) {
        e_p &= 0xFFu;
        e_v &= 0xFFu;
      }
      uint32_t m_p = committed & 0x7FFFFFu, m_v = seen & 0x7FFFFFu;
      if (e_p == e_v) {
        uint32_t d = m_p > m_v ? m_p - m_v : m_v - m_p;
        diffs[n++] = d;
        sum += d;
      } else {
        ++err_e;
      }
    }
    out->exp_mismatch = err_e;
    out->n_match = n;
    out->mant_diff_sum = (uint32_t)sum;
    if (n > 0) {
      out->mant_mean = (double)sum / (double)n;
      qsort(diffs, n, sizeof(uint32_t), ascending_u32);
      out->mant_median = (n & 1u) ? (double)diffs[n / 2] : ((double)diffs[n / 2 - 1] + (double)diffs[n / 2]) / 2.0;
    }
    int reject = ((int64_t)err_e > (int64_t)t_exp) || (out->mant_mean > t_mean) || (out->mant_median > t_median);
    if (n == 0) reject = 1;
    out->accept = reject ? 0 : 1;
    if (gen_indices_opt) {
      int common = 0;
      for (int a = 0; a < k; ++a)
        for (int b = 0; b < k; ++b)
          if ((uint32_t)gen_indices_opt[a] == idx[b]) {
            ++common;
            break;
          }
      out->topk_mismatch = k - common;
    }
  }
  out->status = (uint8_t)status;
  if (status != ST_OK) out->accept = 0;
  free(idx);
  free(pattern);
  free(coef);
  free(diffs);
}

/* ================================================================== */
/* Direct commitments: Section 4 opens with the plain alternative to   */
/* the polynomial: keep the top-k indices and values as they are, at 6 */
/* bytes per point (4 for the index, 2 for the value).  It is the only */
/* form that exists for the larger k of the exponent-error table in    */
/* Section 3 (k up to 4096): k indices below 2^16 residues collide for */
/* every candidate modulus once k reaches the thousands, so Algorithm  */
/* 6 has nothing to return there.  Readings used here:                 */
/*   - a commitment is k records of 6 bytes, record j = flat index     */
/*     (4 bytes little-endian) then the 16-bit pattern (2 bytes        */
/*     little-endian), records in ascending index order (the paper     */
/*     fixes no order; this one makes the bytes unique);               */
/*   - validation is Algorithm 2 with "evaluate the polynomial at the  */
/*     index" replaced by "look the index up": a recomputed top-k      */
/*     index that was not committed has nothing to agree with and      */
/*     counts as an exponent mismatch;                                 */
/*   - a commitment whose indices are not strictly ascending or reach  */
/*     beyond the chunk is malformed (ST_BAD_PROOF);                   */
/*   - exponent deviation (the columns of the table in Section 3):     */
/*     d = exponent field seen - exponent field committed, for every   */
/*     index both sides selected, counted in nine bins: 0, -1, +1, -2, */
/*     +2, -10..-3, 3..10, 11 <= |d| <= 99, |d| >= 100.                */
/* ================================================================== */

static int by_flat_index(const void* a, const void* b) {
  const ranked* p = (const ranked*)a;
  const ranked* q = (const ranked*)b;
  return p->flat < q->flat ? -1 : (p->flat > q->flat ? 1 : 0);
}

/* commit: 6k bytes.  Returns ST_OK or ST_K_EXCEEDS (commit zero-filled). */
int oracle_commit_direct_chunk(const void* chunk, int dtype, int rows, int hidden, int64_t row_stride, int k,
                               uint8_t* commit) {
  memset(commit, 0, 6 * (size_t)k);
  uint32_t* idx = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
  uint16_t* bits = (uint16_t*)malloc((size_t)k * sizeof(uint16_t));
  int status = oracle_topk(chunk, dtype, rows, hidden, row_stride, k, idx, bits);
  if (status == ST_OK) {
    ranked* pts = (ranked*)malloc((size_t)k * sizeof(ranked));
    for (int j = 0; j < k; ++j) {
      pts[j].key = 0;
      pts[j].flat = idx[j];
      pts[j].bits = bits[j];
    }
    qsort(pts, (size_t)k, sizeof(ranked), by_flat_index);
    for (int j = 0; j < k; ++j) {
      uint8_t* rec = commit + 6 * (size_t)j;
      rec[0] = (uint8_t)(pts[j].flat & 0xFFu);
      rec[1] = (uint8_t)((pts[j].flat >> 8) & 0xFFu);
      rec[2] = (uint8_t)((pts[j].flat >> 16) & 0xFFu);
      rec[3] = (uint8_t)(pts[j].flat >> 24);
      rec[4] = (uint8_t)(pts[j].bits & 0xFFu);
      rec[5] = (uint8_t)(pts[j].bits >> 8);
    }
    free(pts);
  }
  free(idx);
  free(bits);
  return status;
}

/* exp_dev: 9 counters (see above), may be NULL.  out->modulus stays 0 and
 * out->topk_mismatch is always filled (the commitment carries the indices). */
void oracle_verify_direct_chunk(const void* chunk, int dtype, int rows, int hidden, int64_t row_stride, int k,
                                const uint8_t* commit, int t_exp, double t_mean, double t_median,
                                int sign_in_exponent, oracle_result* out, uint32_t* exp_dev) {
  memset(out, 0, sizeof(*out));
  if (exp_dev) memset(exp_dev, 0, 9 * sizeof(uint32_t));
  uint32_t* c_idx = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
  uint16_t* c_bits = (uint16_t*)malloc((size_t)k * sizeof(uint16_t));
  uint32_t* idx = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
  uint16_t* bits = (uint16_t*)malloc((size_t)k * sizeof(uint16_t));
  uint32_t* diffs = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
  int64_t n_elems = (int64_t)rows * hidden;
  int status = ST_OK;
  for (int j = 0; j < k; ++j) {
    const uint8_t* rec = commit + 6 * (size_t)j;
    c_idx[j] = (uint32_t)rec[0] | ((uint32_t)rec[1] << 8) | ((uint32_t)rec[2] << 16) | ((uint32_t)rec[3] << 24);
    c_bits[j] = (uint16_t)(rec[4] | (rec[5] << 8));
  }
  if (k > n_elems) status = ST_K_EXCEEDS;
  if (status == ST_OK) {
    for (int j = 0; j < k; ++j) {
      if ((int64_t)c_idx[j] >= n_elems) status = ST_BAD_PROOF;
      if (j > 0 && c_idx[j] <= c_idx[j - 1]) status = ST_BAD_PROOF;
    }
  }
  if (status == ST_OK) status = oracle_topk(chunk, dtype, rows, hidden, row_stride, k, idx, bits);
  if (status == ST_OK) {
    uint32_t err_e = 0, n = 0, sum = 0;
    int common = 0;
    for (int j = 0; j < k; ++j) {
      int at = -1;
      for (int a = 0; a < k; ++a)
        if (c_idx[a] == idx[j]) at = a;
      if (at < 0) {
        ++err_e; /* nothing was committed for this index */
        continue;
      }
      ++common;
      uint32_t committed = c_bits[at], seen = bits[j];
      uint32_t e_p, e_v;
      if (sign_in_exponent) {
        e_p = committed >> 7;
        e_v = seen >> 7;
      } else {
        e_p = (committed >> 7) & 0xFFu;
        e_v = (seen >> 7) & 0xFFu;
      }
      uint32_t m_p = committed & 0x7Fu, m_v = seen & 0x7Fu;
      if (e_p == e_v) {
        uint32_t d = m_p > m_v ? m_p - m_v : m_v - m_p;
        diffs[n++] = d;
        sum += d;
      } else {
        ++err_e;
      }
      if (exp_dev) {
        int d = (int)((seen >> 7) & 0xFFu) - (int)((committed >> 7) & 0xFFu);
        int a = d < 0 ? -d : d;
        int bin;
        if (d == 0) bin = 0;
        else if (a == 1) bin = d < 0 ? 1 : 2;
        else if (a == 2) bin = d < 0 ? 3 : 4;
        else if (a <= 10) bin = d < 0 ? 5 : 6;
        else if (a <= 99) bin = 7;
        else bin = 8;
        ++exp_dev[bin];
      }
    }
    out->exp_mismatch = err_e;
    out->n_match = n;
    out->mant_diff_sum = sum;
    out->topk_mismatch = k - common;
    if (n > 0) {
      out->mant_mean = (double)sum / (double)n;
      qsort(diffs, n, sizeof(uint32_t), ascending_u32);
      out->mant_median = (n & 1u) ? (double)diffs[n / 2] : ((double)diffs[n / 2 - 1] + (double)diffs[n / 2]) / 2.0;
    }
    int reject = ((int64_t)err_e > (int64_t)t_exp) || (out->mant_mean > t_mean) || (out->mant_median > t_median);
    if (n == 0) reject = 1;
    out->accept = reject ? 0 : 1;
  } else {
    out->topk_mismatch = -1;
  }
  out->status = (uint8_t)status;
  if (status != ST_OK) out->accept = 0;
  free(c_idx);
  free(c_bits);
  free(idx);
  free(bits);
  free(diffs);
}

/* ------------------------------------------------------------------ */
/* Batch drivers: chunks of chunk_len rows per sequence (Section 5.5:   */
/* one proof per 32 new tokens), the last chunk of a sequence may be    */
/* shorter.  seq_offsets: num_seqs + 1 row offsets, or NULL for        */
/* uniform sequences of tokens_per_seq rows.  Threads split chunks.    */
/* ------------------------------------------------------------------ */

typedef struct {
  int64_t row0;
  int32_t rows;
} chunk_span;

static int64_t enumerate_chunks(int num_seqs, int64_t tokens_per_seq, const int64_t* seq_offsets,
                                int chunk_len, chunk_span* out) {
  int64_t n = 0;
  for (int s = 0; s < num_seqs; ++s) {
    int64_t begin = seq_offsets ? seq_offsets[s] : (int64_t)s * tokens_per_seq;
    int64_t end = seq_offsets ? seq_offsets[s + 1] : begin + tokens_per_seq;
    for (int64_t r = begin; r < end; r += chunk_len) {
      if (out) {
        out[n].row0 = r;
        out[n].rows = (int32_t)((end - r) < chunk_len ? (end - r) : chunk_len);
      }
      ++n;
    }
  }
  return n;
}

int64_t oracle_num_chunks(int num_seqs, int64_t tokens_per_seq, const int64_t* seq_offsets, int chunk_len) {
  return enumerate_chunks(num_seqs, tokens_per_seq, seq_offsets, chunk_len, NULL);
}

typedef struct {
  int tid, nthreads, verify;
  const uint8_t* act;
  int dtype, hidden, k;
  int64_t row_stride;
  const chunk_span* spans;
  int64_t count; /* chunks of the batch */
  uint8_t* proofs;
  uint8_t* status;
  int32_t* indices;
  const uint8_t* proofs_in;
  const int32_t* gen_indices;
  oracle_result* results;
  int t_exp, sign_in_exponent;
  double t_mean, t_median;
  /* optional, one entry per chunk (Section 6 suggests thresholds chosen per generation);
   * where absent the scalars above hold for every chunk */
  const int32_t* t_exp_each;
  const double* t_mean_each;
  const double* t_median_each;
} job;

static void* worker(void* arg) {
  job* jb = (job*)arg;
  size_t esz = jb->dtype == 0 ? 2 : 4;
  int wide = jb->dtype == 2; /* fp32 chunks committed over Z_q */
  size_t pbytes = 2 + (wide ? 4 : 2) * (size_t)jb->k;
  for (int64_t c = jb->tid; c < jb->count; c += jb->nthreads) {
    const void* chunk = jb->act + (size_t)jb->spans[c].row0 * (size_t)jb->row_stride * esz;
    const int t_exp = jb->t_exp_each ? jb->t_exp_each[c] : jb->t_exp;
    const double t_mean = jb->t_mean_each ? jb->t_mean_each[c] : jb->t_mean;
    const double t_median = jb->t_median_each ? jb->t_median_each[c] : jb->t_median;
    if (!jb->verify && wide) {
      jb->status[c] = (uint8_t)oracle_build_chunk32(chunk, jb->spans[c].rows, jb->hidden, jb->row_stride, jb->k,
                                                    jb->proofs + (size_t)c * pbytes,
                                                    jb->indices ? jb->indices + (size_t)c * jb->k : NULL);
    } else if (jb->verify && jb->dtype == 3) {
      oracle_verify_chunk_padded(chunk, jb->spans[c].rows, jb->hidden, jb->row_stride, jb->k,
                                 jb->proofs_in + (size_t)c * pbytes, t_exp, t_mean, t_median,
                                 jb->sign_in_exponent,
                                 jb->gen_indices ? jb->gen_indices + (size_t)c * jb->k : NULL, &jb->results[c]);
    } else if (wide) {
      oracle_verify_chunk32(chunk, jb->spans[c].rows, jb->hidden, jb->row_stride, jb->k,
                            jb->proofs_in + (size_t)c * pbytes, t_exp, t_mean, t_median,
                            jb->sign_in_exponent,
                            jb->gen_indices ? jb->gen_indices + (size_t)c * jb->k : NULL, &jb->results[c]);
    } else if (!jb->verify) {
      int st = oracle_build_chunk(chunk, jb->dtype, jb->spans[c].rows, jb->hidden, jb->row_stride, jb->k,
                                  jb->proofs + (size_t)c * pbytes,
                                  jb->indices ? jb->indices + (size_t)c * jb->k : NULL);
      jb->status[c] = (uint8_t)st;
    } else {
      oracle_verify_chunk(chunk, jb->dtype, jb->spans[c].rows, jb->hidden, jb->row_stride, jb->k,
                          jb->proofs_in + (size_t)c * pbytes, t_exp, t_mean, t_median,
                          jb->sign_in_exponent,
                          jb->gen_indices ? jb->gen_indices + (size_t)c * jb->k : NULL, &jb->results[c]);
    }
  }
  return NULL;
}

static int run_jobs(job* proto, int nthreads) {
  if (nthreads < 1) nthreads = 1;
  pthread_t* th = (pthread_t*)malloc((size_t)nthreads * sizeof(pthread_t));
  job* jobs = (job*)malloc((size_t)nthreads * sizeof(job));
  for (int t = 0; t < nthreads; ++t) {
    jobs[t] = *proto;
    jobs[t].tid = t;
    jobs[t].nthreads = nthreads;
    pthread_create(&th[t], NULL, worker, &jobs[t]);
  }
  for (int t = 0; t < nthreads; ++t) pthread_join(th[t], NULL);
  free(jobs);
  free(th);
  return 0;
}

/* Proofs for every chunk of the batch, in batch order. */
int oracle_build_proofs(const void* act, int dtype, int hidden, int chunk_len, int k, int num_seqs,
                        int64_t tokens_per_seq, const int64_t* seq_offsets, int64_t row_stride,
                        uint8_t* proofs, uint8_t* status,
                        int32_t* indices_opt, int nthreads) {
  int64_t n = enumerate_chunks(num_seqs, tokens_per_seq, seq_offsets, chunk_len, NULL);
  chunk_span* spans = (chunk_span*)malloc((size_t)(n > 0 ? n : 1) * sizeof(chunk_span));
  enumerate_chunks(num_seqs, tokens_per_seq, seq_offsets, chunk_len, spans);
  job jb;
  memset(&jb, 0, sizeof(jb));
  jb.act = (const uint8_t*)act;
  jb.dtype = dtype;
  jb.hidden = hidden;
  jb.k = k;
  jb.row_stride = row_stride;
  jb.spans = spans;
  jb.count = n;
  jb.proofs = proofs;
  jb.status = status;
  jb.indices = indices_opt;
  run_jobs(&jb, nthreads);
  free(spans);
  return 0;
}

int oracle_verify_proofs(const void* act, int dtype, int hidden, int chunk_len, int k, int num_seqs,
                         int64_t tokens_per_seq, const int64_t* seq_offsets, int64_t row_stride,
                         const uint8_t* proofs, int t_exp, double t_mean, double t_median,
                         int sign_in_exponent, const int32_t* t_exp_each_opt, const double* t_mean_each_opt,
                         const double* t_median_each_opt, const int32_t* gen_indices_opt,
                         oracle_result* results, int nthreads) {
  int64_t n = enumerate_chunks(num_seqs, tokens_per_seq, seq_offsets, chunk_len, NULL);
  chunk_span* spans = (chunk_span*)malloc((size_t)(n > 0 ? n : 1) * sizeof(chunk_span));
  enumerate_chunks(num_seqs, tokens_per_seq, seq_offsets, chunk_len, spans);
  job jb;
  memset(&jb, 0, sizeof(jb));
  jb.verify = 1;
  jb.act = (const uint8_t*)act;
  jb.dtype = dtype;
  jb.hidden = hidden;
  jb.k = k;
  jb.row_stride = row_stride;
  jb.spans = spans;
  jb.count = n;
  jb.proofs_in = proofs;
  jb.gen_indices = gen_indices_opt;
  jb.results = results;
  jb.t_exp = t_exp;
  jb.t_mean = t_mean;
  jb.t_median = t_median;
  jb.sign_in_exponent = sign_in_exponent;
  jb.t_exp_each = t_exp_each_opt;
  jb.t_mean_each = t_mean_each_opt;
  jb.t_median_each = t_median_each_opt;
  run_jobs(&jb, nthreads);
  free(spans);
  return 0;
}

/* ------------------------------------------------------------------ */
/* Several k over the same batch (a parameter sweep).  topk(h, k) is    */
/* the first k of the chunk's elements in rank order, so the selections */
/* of all the k are prefixes of one ranking: each chunk is sorted once, */
/* for the largest k, and Algorithm 1 or 2 then runs once per k on its  */
/* prefix.  16-bit field only (dtype 0 or 1).  Arrays indexed by the    */
/* position of k in ks; a chunk with fewer than k elements gets         */
/* ST_K_EXCEEDS for that k, as in the single-k drivers.                 */
/* ------------------------------------------------------------------ */
typedef struct {
  int tid, nthreads, verify;
  const uint8_t* act;
  int dtype, hidden, nk;
  const int32_t* ks;
  int64_t row_stride;
  const chunk_span* spans;
  int64_t count;
  uint8_t* const* proofs;
  uint8_t* const* status;
  int32_t* const* indices;
  const uint8_t* const* proofs_in;
  const int32_t* const* gen_indices;
  oracle_result* const* results;
  const int32_t* t_exp; /* one per k */
  double t_mean, t_median;
  int sign_in_exponent;
} sweep_job;

static void* sweep_worker(void* arg) {
  sweep_job* jb = (sweep_job*)arg;
  size_t esz = jb->dtype == 0 ? 2 : 4;
  int kmax = 0;
  for (int i = 0; i < jb->nk; ++i)
    if (jb->ks[i] > kmax) kmax = jb->ks[i];
  uint32_t* idx = (uint32_t*)malloc((size_t)kmax * sizeof(uint32_t));
  uint16_t* bits = (uint16_t*)malloc((size_t)kmax * sizeof(uint16_t));
  for (int64_t c = jb->tid; c < jb->count; c += jb->nthreads) {
    const void* chunk = jb->act + (size_t)jb->spans[c].row0 * (size_t)jb->row_stride * esz;
    int64_t n = (int64_t)jb->spans[c].rows * jb->hidden;
    int ranked = (int)(n < kmax ? n : kmax); /* the whole (short) chunk, or the largest k */
    oracle_topk(chunk, jb->dtype, jb->spans[c].rows, jb->hidden, jb->row_stride, ranked, idx, bits);
    for (int i = 0; i < jb->nk; ++i) {
      int k = jb->ks[i];
      size_t pbytes = 2 + 2 * (size_t)k;
      if (!jb->verify) {
        uint8_t* proof = jb->proofs[i] + (size_t)c * pbytes;
        int32_t* ind = (jb->indices && jb->indices[i]) ? jb->indices[i] + (size_t)c * k : NULL;
        memset(proof, 0, pbytes);
        if (ind) memset(ind, 0, (size_t)k * sizeof(int32_t));
        jb->status[i][c] = (uint8_t)(k > n ? ST_K_EXCEEDS : build_from_selection(idx, bits, k, proof, ind));
      } else {
        const int32_t* gen = (jb->gen_indices && jb->gen_indices[i]) ? jb->gen_indices[i] + (size_t)c * k : NULL;
        verify_with_selection(NULL, jb->dtype, jb->spans[c].rows, jb->hidden, jb->row_stride, idx, bits, ranked, k,
                              jb->proofs_in[i] + (size_t)c * pbytes, jb->t_exp[i], jb->t_mean, jb->t_median,
                              jb->sign_in_exponent, gen, &jb->results[i][c]);
      }
    }
  }
  free(idx);
  free(bits);
  return NULL;
}

static int run_sweep(sweep_job* proto, int num_seqs, int64_t tokens_per_seq, const int64_t* seq_offsets,
                     int chunk_len, int nthreads) {
  if (proto->dtype != 0 && proto->dtype != 1) return -1;
  int64_t n = enumerate_chunks(num_seqs, tokens_per_seq, seq_offsets, chunk_len, NULL);
  chunk_span* spans = (chunk_span*)malloc((size_t)(n > 0 ? n : 1) * sizeof(chunk_span));
  enumerate_chunks(num_seqs, tokens_per_seq, seq_offsets, chunk_len, spans);
  proto->spans = spans;
  proto->count = n;
  if (nthreads < 1) nthreads = 1;
  pthread_t* th = (pthread_t*)malloc((size_t)nthreads * sizeof(pthread_t));
  sweep_job* jobs = (sweep_job*)malloc((size_t)nthreads * sizeof(sweep_job));
  for (int t = 0; t < nthreads; ++t) {
    jobs[t] = *proto;
    jobs[t].tid = t;
    jobs[t].nthreads = nthreads;
    pthread_create(&th[t], NULL, sweep_worker, &jobs[t]);
  }
  for (int t = 0; t < nthreads; ++t) pthread_join(th[t], NULL);
  free(jobs);
  free(th);
  free(spans);
  return 0;
}

int oracle_build_proofs_ks(const void* act, int dtype, int hidden, int chunk_len, const int32_t* ks, int nk,
                           int num_seqs, int64_t tokens_per_seq, const int64_t* seq_offsets, int64_t row_stride,
                           uint8_t* const* proofs, uint8_t* const* status, int32_t* const* indices_opt,
                           int nthreads) {
  sweep_job jb;
  memset(&jb, 0, sizeof(jb));
  jb.act = (const uint8_t*)act;
  jb.dtype = dtype;
  jb.hidden = hidden;
  jb.ks = ks;
  jb.nk = nk;
  jb.row_stride = row_stride;
  jb.proofs = proofs;
  jb.status = status;
  jb.indices = indices_opt;
  return run_sweep(&jb, num_seqs, tokens_per_seq, seq_offsets, chunk_len, nthreads);
}

int oracle_verify_proofs_ks(const void* act, int dtype, int hidden, int chunk_len, const int32_t* ks, int nk,
                            int num_seqs, int64_t tokens_per_seq, const int64_t* seq_offsets, int64_t row_stride,
                            const uint8_t* const* proofs, const int32_t* t_exp_per_k, double t_mean,
                            double t_median, int sign_in_exponent, const int32_t* const* gen_indices_opt,
                            oracle_result* const* results, int nthreads) {
  sweep_job jb;
  memset(&jb, 0, sizeof(jb));
  jb.verify = 1;
  jb.act = (const uint8_t*)act;
  jb.dtype = dtype;
  jb.hidden = hidden;
  jb.ks = ks;
  jb.nk = nk;
  jb.row_stride = row_stride;
  jb.proofs_in = proofs;
  jb.gen_indices = gen_indices_opt;
  jb.results = results;
  jb.t_exp = t_exp_per_k;
  jb.t_mean = t_mean;
  jb.t_median = t_median;
  jb.sign_in_exponent = sign_in_exponent;
  return run_sweep(&jb, num_seqs, tokens_per_seq, seq_offsets, chunk_len, nthreads);
}
