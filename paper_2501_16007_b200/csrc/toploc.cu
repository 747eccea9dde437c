// TopLoc proof hot path for sm_100a: one thread block per chunk streams the
// chunk from HBM once, keeps the exact top-k on chip, and finishes the chunk in
// the same kernel (build: injective modulus, interpolation over Z_p, packing;
// verify: Horner evaluation, bit-field comparison, statistics, verdict).
//
// The path is a selection over data read once plus integer modular arithmetic:
// HBM bandwidth is the roofline, there is no dense contraction and therefore no
// tensor-core work.  Blocks of 128 threads, many per SM, so that blocks that
// are in their arithmetic tail overlap with blocks that are streaming.
#include "toploc.h"

#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

namespace {

// ---------------------------------------------------------------------------
// constants of the method
// ---------------------------------------------------------------------------
constexpr uint32_t kPrime = 65521u;      // field modulus: largest prime below 2^16
constexpr uint32_t kModHigh = 65536u;    // Algorithm 6 scans 65536 down to 2^15 + 1
constexpr uint32_t kModLow = 32769u;

// ---------------------------------------------------------------------------
// launch shape
// ---------------------------------------------------------------------------
constexpr int kThreads = 128;            // threads per block
constexpr int kUnroll = 4;               // 16-byte loads in flight per thread and tile
constexpr int kCandCap = 1536;           // candidate buffer entries (8 bytes each)
constexpr int kMaxK = TOPLOC_MAX_K;
constexpr int kEntriesPerThread = kMaxK / kThreads;  // tail arrays: entries owned per thread
constexpr int kIdxBits = 24;             // flat index field of a candidate
constexpr uint32_t kIdxMask = (1u << kIdxBits) - 1u;

static_assert(kMaxK % kThreads == 0, "tail loops assume whole entries per thread");
static_assert(kCandCap >= kMaxK + kThreads * 8, "a safe sub-tile must fit after a compaction");
static_assert(kCandCap * 8 >= 8192 && kCandCap * 8 >= 6 * kMaxK * 4, "buffer is reused by the tail");

struct ChunkSpan {   // one per chunk of a ragged batch, built on the host
  long long row0;
  int rows;
  int pad;
};

struct BatchParams {
  const void* act;
  long long row_stride;        // elements
  long long tokens_per_seq;    // uniform batches
  const ChunkSpan* spans;      // ragged batches (device), else nullptr
  int hidden;
  int chunk_len;
  int k;
  int chunks_per_seq;
};

struct BuildOut {
  uint8_t* proofs;
  uint8_t* status;
  int32_t* indices;            // optional
};

struct VerifyIo {
  const uint8_t* proofs;
  toploc_chunk_result* results;
  const int32_t* gen_indices;  // optional
  int t_exp;
  int sign_in_exponent;
  double t_mean;
  double t_median;
};

// A candidate is one 64-bit word whose unsigned order is the ranking order:
// magnitude key (bit pattern without sign) descending, then flat index
// ascending.  Layout: key << 25 | (kIdxMask - index) << 1 | sign.
__device__ __forceinline__ unsigned long long make_candidate(uint32_t key, uint32_t flat, uint32_t sign) {
  return ((unsigned long long)key << (kIdxBits + 1)) | ((unsigned long long)(kIdxMask - flat) << 1) | sign;
}

struct __align__(16) BlockShared {
  unsigned long long cand[kCandCap];  // candidates; later the modulus bitmap, then the tail arrays
  uint32_t hist[256];
  uint32_t idx[kMaxK];                // selected flat indices in rank order
  uint16_t bits[kMaxK];               // selected 16-bit patterns in rank order
  int count;
  uint32_t digit;
  int want;
  uint32_t err_e;
  uint32_t diff_sum;
  uint32_t common;
};

__device__ __forceinline__ uint4 load_streaming(const uint4* p) {
  uint4 v;
  asm("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
      : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
      : "l"(p));
  return v;
}

__device__ __forceinline__ void push_candidate(BlockShared& sh, unsigned long long c, int& max_pos) {
  int pos = atomicAdd(&sh.count, 1);
  if (pos < kCandCap) sh.cand[pos] = c;
  max_pos = max(max_pos, pos);
}

// ---------------------------------------------------------------------------
// Where a chunk's elements live.  MODE 0: rows are contiguous (row_stride ==
// hidden) and 16-byte aligned, the chunk is one flat array of vectors.
// MODE 1: 16-byte aligned rows with padding between them.  MODE 2: anything
// else, one element at a time.  DT 0 = bf16, 1 = fp32.
// ---------------------------------------------------------------------------
template <int DT, int MODE>
struct ChunkSource {
  static constexpr int kVec = (MODE == 2) ? 1 : (DT == 0 ? 8 : 4);
  static constexpr int kElemBytes = (DT == 0) ? 2 : 4;
  const char* base;
  long long row_stride;
  int hidden;
  int vecs_per_row;

  __device__ __forceinline__ uint4 load(int v) const {
    if (MODE == 0) {
      return load_streaming(reinterpret_cast<const uint4*>(base) + v);
    } else if (MODE == 1) {
      int t = v / vecs_per_row;
      int c = v - t * vecs_per_row;
      const char* p = base + ((long long)t * row_stride + (long long)c * kVec) * kElemBytes;
      return load_streaming(reinterpret_cast<const uint4*>(p));
    } else {
      int t = v / hidden;
      int c = v - t * hidden;
      const char* p = base + ((long long)t * row_stride + c) * kElemBytes;
      uint4 w = make_uint4(0, 0, 0, 0);
      if (DT == 0) w.x = *reinterpret_cast<const unsigned short*>(p);
      else w.x = *reinterpret_cast<const uint32_t*>(p);
      return w;
    }
  }
};

// Appends every element of one vector whose key is >= thr.  flat0 = flat index
// of the vector's first element.  bf16 fast test: with both 15-bit keys of a
// word in separate 16-bit lanes, adding (0x8000 - thr) to each lane sets the
// lane's top bit exactly when key >= thr (no carry leaves a lane).
template <int DT, int VEC>
__device__ __forceinline__ void filter_vector(BlockShared& sh, const uint4& w, uint32_t thr, uint32_t flat0,
                                              int& max_pos) {
  if (VEC == 1) {
    uint32_t key = DT == 0 ? (w.x & 0x7FFFu) : (w.x & 0x7FFFFFFFu);
    uint32_t sign = DT == 0 ? (w.x >> 15) & 1u : (w.x >> 31);
    if (key >= thr) push_candidate(sh, make_candidate(key, flat0, sign), max_pos);
  } else if (DT == 0) {
    const uint32_t add = (0x8000u - thr) * 0x00010001u;
    uint32_t t0 = (w.x & 0x7FFF7FFFu) + add;
    uint32_t t1 = (w.y & 0x7FFF7FFFu) + add;
    uint32_t t2 = (w.z & 0x7FFF7FFFu) + add;
    uint32_t t3 = (w.w & 0x7FFF7FFFu) + add;
    if ((t0 | t1 | t2 | t3) & 0x80008000u) {
      const uint32_t words[4] = {w.x, w.y, w.z, w.w};
      const uint32_t tests[4] = {t0, t1, t2, t3};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (tests[i] & 0x00008000u)
          push_candidate(sh, make_candidate(words[i] & 0x7FFFu, flat0 + 2 * i, (words[i] >> 15) & 1u), max_pos);
        if (tests[i] & 0x80000000u)
          push_candidate(sh, make_candidate((words[i] >> 16) & 0x7FFFu, flat0 + 2 * i + 1, words[i] >> 31),
                         max_pos);
      }
    }
  } else {
    const uint32_t words[4] = {w.x, w.y, w.z, w.w};
    bool any = false;
#pragma unroll
    for (int i = 0; i < 4; ++i) any |= (words[i] & 0x7FFFFFFFu) >= thr;
    if (any) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        uint32_t key = words[i] & 0x7FFFFFFFu;
        if (key >= thr) push_candidate(sh, make_candidate(key, flat0 + i, words[i] >> 31), max_pos);
      }
    }
  }
}

// Keeps the k best candidates (radix select on the 56 meaningful bits, most
// significant digit first) and raises the threshold to "strictly better than
// the k-th": every later element of the chunk has a higher flat index, so one
// that only ties the k-th key can no longer be selected.  All threads call it.
template <int DT>
__device__ void compact_candidates(BlockShared& sh, int k, uint32_t& thr) {
  const int tid = threadIdx.x;
  __syncthreads();
  const int n = min(sh.count, kCandCap);
  __syncthreads();
  if (n <= k) return;
  constexpr int kPer = kCandCap / kThreads;
  unsigned long long mine[kPer];
#pragma unroll
  for (int i = 0; i < kPer; ++i) {
    int e = tid + i * kThreads;
    mine[i] = e < n ? sh.cand[e] : 0ull;
  }
  unsigned long long prefix = 0ull, mask = 0ull;
  int want = k;
  // bf16 keys have 15 bits: candidate bits 40..55 are zero, two digit passes fewer
  for (int shift = (DT == 0 ? 32 : 48); shift >= 0; shift -= 8) {
    sh.hist[tid] = 0;
    sh.hist[tid + kThreads] = 0;
    __syncthreads();
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
      int e = tid + i * kThreads;
      if (e < n && (mine[i] & mask) == prefix) atomicAdd(&sh.hist[(uint32_t)(mine[i] >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (tid < 32) {
      // lane l owns digits 8l..8l+7; find the largest digit d with
      // (#candidates with digit >= d) >= want
      uint32_t local[8];
      uint32_t sum = 0;
#pragma unroll
      for (int b = 0; b < 8; ++b) {
        local[b] = sh.hist[tid * 8 + b];
        sum += local[b];
      }
      uint32_t incl = sum;  // becomes the sum over lanes >= this one
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        uint32_t other = __shfl_down_sync(0xFFFFFFFFu, incl, off);
        if (tid + off < 32) incl += other;
      }
      uint32_t above = incl - sum;  // candidates in higher lanes
      if (above < (uint32_t)want && incl >= (uint32_t)want) {
        uint32_t acc = above;
#pragma unroll
        for (int b = 7; b >= 0; --b) {
          if (acc < (uint32_t)want && acc + local[b] >= (uint32_t)want) {
            sh.digit = (uint32_t)(tid * 8 + b);
            sh.want = want - (int)acc;
          }
          acc += local[b];
        }
      }
    }
    __syncthreads();
    prefix |= (unsigned long long)sh.digit << shift;
    mask |= 255ull << shift;
    want = sh.want;
  }
  const unsigned long long pivot = prefix;  // the k-th best candidate itself
  if (tid == 0) sh.count = 0;
  __syncthreads();
#pragma unroll
  for (int i = 0; i < kPer; ++i) {
    int e = tid + i * kThreads;
    if (e < n && mine[i] >= pivot) sh.cand[atomicAdd(&sh.count, 1)] = mine[i];
  }
  __syncthreads();
  thr = (uint32_t)(pivot >> (kIdxBits + 1)) + 1u;
}

// Processes vectors [vb, ve) one vector per thread at a time, compacting
// whenever another round might not fit.  Precondition: count <= k.
template <int DT, int MODE>
__device__ void select_carefully(BlockShared& sh, const ChunkSource<DT, MODE>& src, int vb, int ve, int k,
                                 uint32_t& thr) {
  constexpr int VEC = ChunkSource<DT, MODE>::kVec;
  const int tid = threadIdx.x;
  int max_pos = -1;
  for (int s = vb; s < ve; s += kThreads) {
    int v = s + tid;
    if (v < ve) filter_vector<DT, VEC>(sh, src.load(v), thr, (uint32_t)v * VEC, max_pos);
    if (__syncthreads_or(max_pos + 1 + kThreads * VEC > kCandCap)) {
      compact_candidates<DT>(sh, k, thr);
      max_pos = -1;
    }
  }
}

// Exact top-k of one chunk.  On return sh.idx / sh.bits hold the k selected
// flat indices and 16-bit patterns in rank order (magnitude descending, index
// ascending).  n_elems >= k is the caller's business.
template <int DT, int MODE>
__device__ void select_topk(BlockShared& sh, const ChunkSource<DT, MODE>& src, int n_elems, int k) {
  constexpr int VEC = ChunkSource<DT, MODE>::kVec;
  constexpr int kTileVecs = kThreads * kUnroll;
  const int tid = threadIdx.x;
  const int n_vecs = n_elems / VEC;
  const int trigger = max(4 * k, 256);  // compact once this many candidates are held

  if (tid == 0) sh.count = 0;
  __syncthreads();
  uint32_t thr = 0;  // accept everything until k candidates exist

  // Warm-up on the first tile, then raise the threshold as far as it goes.
  const int first = min(n_vecs, kTileVecs);
  select_carefully<DT, MODE>(sh, src, 0, first, k, thr);
  compact_candidates<DT>(sh, k, thr);

  // Streaming tiles: kUnroll independent 16-byte loads per thread, then the
  // filter.  The block only synchronises to agree on whether to compact.
  int v0 = first;
  int max_pos = -1;
  bool overflow = false;
  for (; v0 + kTileVecs <= n_vecs; v0 += kTileVecs) {
    uint4 w[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) w[u] = src.load(v0 + u * kThreads + tid);
#pragma unroll
    for (int u = 0; u < kUnroll; ++u)
      filter_vector<DT, VEC>(sh, w[u], thr, (uint32_t)(v0 + u * kThreads + tid) * VEC, max_pos);
    if (__syncthreads_or(max_pos + 1 >= trigger)) {
      if (sh.count > kCandCap) {  // uniform: nobody appends until the next tile
        overflow = true;
        break;
      }
      compact_candidates<DT>(sh, k, thr);
      max_pos = -1;
    }
  }
  if (overflow) {
    // More candidates than the buffer holds arrived within one tile (e.g.
    // magnitudes that keep growing).  Start over, carefully.
    __syncthreads();
    if (tid == 0) sh.count = 0;
    __syncthreads();
    thr = 0;
    select_carefully<DT, MODE>(sh, src, 0, n_vecs, k, thr);
  } else {
    compact_candidates<DT>(sh, k, thr);
    select_carefully<DT, MODE>(sh, src, v0, n_vecs, k, thr);
  }
  compact_candidates<DT>(sh, k, thr);  // exactly k remain

  // Rank by counting: position = number of better candidates.
  __syncthreads();
  for (int j = tid; j < k; j += kThreads) {
    const unsigned long long cj = sh.cand[j];
    int rank = 0;
    for (int i = 0; i < k; ++i) rank += sh.cand[i] > cj;
    const uint32_t key = (uint32_t)(cj >> (kIdxBits + 1));
    const uint32_t sign = (uint32_t)cj & 1u;
    sh.idx[rank] = kIdxMask - ((uint32_t)(cj >> 1) & kIdxMask);
    sh.bits[rank] = (uint16_t)((sign << 15) | (DT == 0 ? key : (key >> 16)));
  }
  __syncthreads();
}

// ---------------------------------------------------------------------------
// arithmetic in Z_p (all operands < p < 2^16, so a * b + c fits 32 bits)
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t mul_mod(uint32_t a, uint32_t b) { return (a * b) % kPrime; }
__device__ __forceinline__ uint32_t mad_mod(uint32_t a, uint32_t b, uint32_t c) { return (a * b + c) % kPrime; }
__device__ __forceinline__ uint32_t sub_mod(uint32_t a, uint32_t b) { return a >= b ? a - b : a + kPrime - b; }

// a^(p-2): the inverse of a != 0 (the inverse is unique, Algorithm 4 computes
// the same value by the extended Euclidean algorithm).
__device__ uint32_t inverse_mod(uint32_t a) {
  uint32_t result = 1, base = a;
  uint32_t e = kPrime - 2u;
#pragma unroll 1
  while (e) {
    if (e & 1u) result = mul_mod(result, base);
    base = mul_mod(base, base);
    e >>= 1;
  }
  return result;
}

// Algorithm 6: largest m in [2^15 + 1, 2^16] for which the selected indices
// stay distinct as (index mod m) mod p -- the second reduction because the
// x-coordinates live in Z_p and m may exceed p.  Returns 0 if there is none.
// x_out[e] receives the residue of entry tid + e * kThreads.  Uses the
// candidate buffer as a 65536-bit set.
__device__ uint32_t find_injective_modulus(BlockShared& sh, int k, uint32_t (&x_out)[kEntriesPerThread]) {
  const int tid = threadIdx.x;
  uint32_t* seen = reinterpret_cast<uint32_t*>(sh.cand);
  for (int i = tid; i < 2048; i += kThreads) seen[i] = 0;
  __syncthreads();
  uint32_t found = 0;
#pragma unroll 1
  for (uint32_t m = kModHigh; m >= kModLow; --m) {
    uint32_t dup = 0;
#pragma unroll
    for (int e = 0; e < kEntriesPerThread; ++e) {
      int j = tid + e * kThreads;
      if (j < k) {
        uint32_t r = sh.idx[j] % m;
        if (r >= kPrime) r -= kPrime;
        x_out[e] = r;
        uint32_t bit = 1u << (r & 31u);
        dup |= atomicOr(&seen[r >> 5], bit) & bit;
      }
    }
    const int clash = __syncthreads_or(dup != 0);
#pragma unroll
    for (int e = 0; e < kEntriesPerThread; ++e) {
      int j = tid + e * kThreads;
      if (j < k) seen[x_out[e] >> 5] = 0;
    }
    __syncthreads();
    if (!clash) {
      found = m;
      break;
    }
  }
  return found;
}

// Algorithm 3 (Newton interpolation over Z_p) with the divisions postponed:
// every divided difference is carried as a fraction num / den, one level per
// block-wide step, and each Newton coefficient takes a single inverse at the
// end.  The Newton form is then multiplied out from the innermost bracket:
//   P <- a_{k-1};  P <- P * (x - x_i) + a_i  for i = k-2 .. 0.
// Entry j of every array belongs to thread j % kThreads.  On return coef[]
// (shared, k entries, ascending degree) holds the polynomial.
__device__ uint32_t* interpolate(BlockShared& sh, int k, const uint32_t (&x_in)[kEntriesPerThread]) {
  const int tid = threadIdx.x;
  uint32_t* X = reinterpret_cast<uint32_t*>(sh.cand);
  uint32_t* A = X + kMaxK;
  uint32_t* num[2] = {A + kMaxK, A + 2 * kMaxK};
  uint32_t* den[2] = {A + 3 * kMaxK, A + 4 * kMaxK};
  uint32_t fin_num[kEntriesPerThread], fin_den[kEntriesPerThread];
#pragma unroll
  for (int e = 0; e < kEntriesPerThread; ++e) {
    int j = tid + e * kThreads;
    fin_num[e] = 0;
    fin_den[e] = 1;
    if (j < k) {
      uint32_t y = sh.bits[j];
      if (y >= kPrime) y -= kPrime;  // "dd <- y mod M"
      X[j] = x_in[e];
      num[0][j] = y;
      den[0][j] = 1;
      fin_num[e] = y;  // entry 0 is already final; the others are overwritten at level j
    }
  }
  __syncthreads();
  int cur = 0;
#pragma unroll 1
  for (int level = 1; level < k; ++level) {
    const uint32_t* nc = num[cur];
    const uint32_t* dc = den[cur];
    uint32_t* nn = num[cur ^ 1];
    uint32_t* dn = den[cur ^ 1];
#pragma unroll
    for (int e = 0; e < kEntriesPerThread; ++e) {
      int j = tid + e * kThreads;
      if (j < k && j >= level) {
        // (n_j/d_j - n_{j-1}/d_{j-1}) / (x_j - x_{j-level})
        uint32_t nj = nc[j], np = nc[j - 1], dj = dc[j], dp = dc[j - 1];
        uint32_t span = sub_mod(X[j], X[j - level]);
        uint32_t n_new = mad_mod(kPrime - np, dj, mul_mod(nj, dp));
        uint32_t d_new = mul_mod(mul_mod(dj, dp), span);
        nn[j] = n_new;
        dn[j] = d_new;
        if (j == level) {
          fin_num[e] = n_new;
          fin_den[e] = d_new;
        }
      }
    }
    __syncthreads();
    cur ^= 1;
  }
#pragma unroll
  for (int e = 0; e < kEntriesPerThread; ++e) {
    int j = tid + e * kThreads;
    if (j < k) A[j] = mul_mod(fin_num[e], inverse_mod(fin_den[e]));
  }
  uint32_t* poly[2] = {num[0], num[1]};
  __syncthreads();  // A complete; num[] free for reuse (every level's reads are done)
  for (int d = tid; d < k; d += kThreads) poly[0][d] = (d == 0) ? A[k - 1] : 0u;
  __syncthreads();
  cur = 0;
#pragma unroll 1
  for (int i = k - 2; i >= 0; --i) {
    const uint32_t neg_x = (kPrime - X[i]) % kPrime;
    const uint32_t a_i = A[i];
    const int top = k - 1 - i;  // degree after this step
    const uint32_t* pc = poly[cur];
    uint32_t* pn = poly[cur ^ 1];
#pragma unroll
    for (int e = 0; e < kEntriesPerThread; ++e) {
      int d = tid + e * kThreads;
      if (d <= top) {
        const uint32_t carry = d > 0 ? pc[d - 1] : a_i;
        const uint32_t here = d < top ? pc[d] : 0u;  // the old polynomial has degree top - 1
        pn[d] = mad_mod(here, neg_x, carry);
      }
    }
    __syncthreads();
    cur ^= 1;
  }
  return poly[cur];
}

struct ChunkPlace {
  const char* base;
  int rows;
};

template <int DT>
__device__ __forceinline__ ChunkPlace locate_chunk(const BatchParams& bp, long long chunk) {
  long long row0;
  int rows;
  if (bp.spans != nullptr) {
    row0 = bp.spans[chunk].row0;
    rows = bp.spans[chunk].rows;
  } else {
    long long seq = chunk / bp.chunks_per_seq;
    long long j = chunk - seq * bp.chunks_per_seq;
    row0 = seq * bp.tokens_per_seq + j * bp.chunk_len;
    long long left = bp.tokens_per_seq - j * bp.chunk_len;
    rows = (int)(left < bp.chunk_len ? left : bp.chunk_len);
  }
  ChunkPlace pl;
  pl.base = static_cast<const char*>(bp.act) + row0 * bp.row_stride * (DT == 0 ? 2 : 4);
  pl.rows = rows;
  return pl;
}

// ---------------------------------------------------------------------------
// Algorithm 1 for one chunk per block.
// ---------------------------------------------------------------------------
template <int DT, int MODE>
__global__ void __launch_bounds__(kThreads) toploc_build_kernel(BatchParams bp, BuildOut out) {
  __shared__ BlockShared sh;
  const int tid = threadIdx.x;
  const long long chunk = blockIdx.x;
  const int k = bp.k;
  const size_t proof_bytes = 2 + 2 * (size_t)k;
  uint16_t* proof = reinterpret_cast<uint16_t*>(out.proofs + chunk * proof_bytes);
  int32_t* indices = out.indices ? out.indices + chunk * k : nullptr;

  const ChunkPlace pl = locate_chunk<DT>(bp, chunk);
  const long long n_elems = (long long)pl.rows * bp.hidden;
  if (n_elems < k) {
    for (int i = tid; i < k + 1; i += kThreads) proof[i] = 0;
    if (indices)
      for (int i = tid; i < k; i += kThreads) indices[i] = 0;
    if (tid == 0) out.status[chunk] = TOPLOC_CHUNK_K_EXCEEDS_CHUNK;
    return;
  }
  ChunkSource<DT, MODE> src;
  src.base = pl.base;
  src.row_stride = bp.row_stride;
  src.hidden = bp.hidden;
  src.vecs_per_row = bp.hidden / ChunkSource<DT, MODE>::kVec;
  select_topk<DT, MODE>(sh, src, (int)n_elems, k);

  if (indices)
    for (int j = tid; j < k; j += kThreads) indices[j] = (int32_t)sh.idx[j];
  uint32_t unrepresentable = 0;
  for (int j = tid; j < k; j += kThreads) unrepresentable |= sh.bits[j] >= kPrime;
  const int nonfinite = __syncthreads_or(unrepresentable != 0);

  uint32_t x[kEntriesPerThread];
  const uint32_t m = find_injective_modulus(sh, k, x);
  if (m == 0) {
    for (int i = tid; i < k + 1; i += kThreads) proof[i] = 0;
    if (tid == 0) out.status[chunk] = TOPLOC_CHUNK_NO_INJECTIVE_MODULUS;
    return;
  }
  const uint32_t* coef = interpolate(sh, k, x);
  // proof: m & 0xFFFF (65536 -> 0), then k coefficients, little-endian 16-bit words
  if (tid == 0) {
    proof[0] = (uint16_t)(m & 0xFFFFu);
    out.status[chunk] = nonfinite ? TOPLOC_CHUNK_NONFINITE_COMMITTED : TOPLOC_CHUNK_OK;
  }
  for (int d = tid; d < k; d += kThreads) proof[1 + d] = (uint16_t)coef[d];
}

// ---------------------------------------------------------------------------
// Algorithm 2 for one chunk per block.
// ---------------------------------------------------------------------------
template <int DT, int MODE>
__global__ void __launch_bounds__(kThreads) toploc_verify_kernel(BatchParams bp, VerifyIo io) {
  __shared__ BlockShared sh;
  const int tid = threadIdx.x;
  const long long chunk = blockIdx.x;
  const int k = bp.k;
  const size_t proof_bytes = 2 + 2 * (size_t)k;
  const uint16_t* proof = reinterpret_cast<const uint16_t*>(io.proofs + chunk * proof_bytes);

  toploc_chunk_result res;
  res.exp_mismatch = 0;
  res.n_match = 0;
  res.mant_diff_sum = 0;
  res.topk_mismatch = -1;
  res.mant_mean = 0.0;
  res.mant_median = 0.0;
  res.accept = 0;
  res.status = TOPLOC_CHUNK_OK;
  res.pad[0] = res.pad[1] = 0;

  // decode
  uint32_t m = proof[0];
  if (m == 0) m = 65536u;
  res.modulus = m;
  uint32_t bad = (m < kModLow || m > kModHigh);
  for (int d = tid; d < k; d += kThreads) bad |= proof[1 + d] >= kPrime;
  if (__syncthreads_or(bad != 0)) {
    res.status = TOPLOC_CHUNK_BAD_PROOF;
    if (tid == 0) io.results[chunk] = res;
    return;
  }
  const ChunkPlace pl = locate_chunk<DT>(bp, chunk);
  const long long n_elems = (long long)pl.rows * bp.hidden;
  if (n_elems < k) {
    res.status = TOPLOC_CHUNK_K_EXCEEDS_CHUNK;
    if (tid == 0) io.results[chunk] = res;
    return;
  }
  ChunkSource<DT, MODE> src;
  src.base = pl.base;
  src.row_stride = bp.row_stride;
  src.hidden = bp.hidden;
  src.vecs_per_row = bp.hidden / ChunkSource<DT, MODE>::kVec;
  select_topk<DT, MODE>(sh, src, (int)n_elems, k);

  // the candidate buffer is free now: coefficients, then the generator's indices
  uint32_t* coef = reinterpret_cast<uint32_t*>(sh.cand);
  uint32_t* gen = coef + kMaxK;
  for (int d = tid; d < k; d += kThreads) coef[d] = proof[1 + d];
  if (io.gen_indices)
    for (int j = tid; j < k; j += kThreads) gen[j] = (uint32_t)io.gen_indices[chunk * k + j];
  sh.hist[tid] = 0;  // 128 bins: a 7-bit mantissa difference is at most 127
  if (tid == 0) {
    sh.err_e = 0;
    sh.diff_sum = 0;
    sh.common = 0;
  }
  __syncthreads();
  for (int j = tid; j < k; j += kThreads) {
    uint32_t x = sh.idx[j] % m;
    if (x >= kPrime) x -= kPrime;
    // Algorithm 5 (Horner), highest degree first
    uint32_t acc = coef[k - 1];
#pragma unroll 4
    for (int d = k - 2; d >= 0; --d) acc = mad_mod(acc, x, coef[d]);
    const uint32_t seen = sh.bits[j];
    uint32_t e_p = acc >> 7, e_v = seen >> 7;  // sign + 8 exponent bits
    if (!io.sign_in_exponent) {
      e_p &= 0xFFu;
      e_v &= 0xFFu;
    }
    if (e_p == e_v) {
      int diff = (int)(acc & 0x7Fu) - (int)(seen & 0x7Fu);
      diff = diff < 0 ? -diff : diff;
      atomicAdd(&sh.hist[diff], 1u);
      atomicAdd(&sh.diff_sum, (uint32_t)diff);
    } else {
      atomicAdd(&sh.err_e, 1u);
    }
    if (io.gen_indices) {
      const uint32_t mine = sh.idx[j];
      uint32_t hit = 0;
      for (int i = 0; i < k; ++i) hit |= gen[i] == mine;
      if (hit) atomicAdd(&sh.common, 1u);
    }
  }
  __syncthreads();
  if (tid == 0) {
    const uint32_t n = (uint32_t)k - sh.err_e;
    res.exp_mismatch = sh.err_e;
    res.n_match = n;
    res.mant_diff_sum = sh.diff_sum;
    if (io.gen_indices) res.topk_mismatch = k - (int)sh.common;
    bool reject = true;  // nothing matched: nothing to accept on
    if (n > 0) {
      res.mant_mean = (double)sh.diff_sum / (double)n;
      // median from the histogram: sorted positions (n-1)/2 and n/2
      const uint32_t lo_pos = (n - 1) / 2, hi_pos = n / 2;
      uint32_t seen_cnt = 0;
      int lo_val = -1, hi_val = -1;
      for (int v = 0; v < 128 && hi_val < 0; ++v) {
        seen_cnt += sh.hist[v];
        if (lo_val < 0 && seen_cnt > lo_pos) lo_val = v;
        if (seen_cnt > hi_pos) hi_val = v;
      }
      res.mant_median = ((double)lo_val + (double)hi_val) * 0.5;
      reject = (res.exp_mismatch > (uint32_t)io.t_exp) || (res.mant_mean > io.t_mean) ||
               (res.mant_median > io.t_median);
    }
    res.accept = reject ? 0 : 1;
    io.results[chunk] = res;
  }
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
struct HostPlan {
  long long num_chunks;
  long long max_seq_rows;
  int chunks_per_seq;  // uniform only
  bool ragged;
};

int plan_layout(const toploc_layout* lay, HostPlan* plan) {
  if (lay == nullptr) return TOPLOC_ERR_INVALID_ARGUMENT;
  if (lay->dtype != TOPLOC_DTYPE_BF16 && lay->dtype != TOPLOC_DTYPE_FP32) return TOPLOC_ERR_UNSUPPORTED;
  if (lay->hidden <= 0 || lay->chunk_len <= 0 || lay->num_seqs <= 0 || lay->reserved != 0)
    return TOPLOC_ERR_INVALID_ARGUMENT;
  if (lay->k < 1) return TOPLOC_ERR_INVALID_ARGUMENT;
  if (lay->k > TOPLOC_MAX_K) return TOPLOC_ERR_UNSUPPORTED;
  if (lay->row_stride < lay->hidden) return TOPLOC_ERR_INVALID_ARGUMENT;
  if ((long long)lay->hidden * lay->chunk_len > TOPLOC_MAX_CHUNK_ELEMS) return TOPLOC_ERR_UNSUPPORTED;
  plan->ragged = lay->seq_offsets != nullptr;
  plan->chunks_per_seq = 0;
  long long n = 0, longest = 0;
  if (plan->ragged) {
    if (lay->seq_offsets[0] < 0) return TOPLOC_ERR_INVALID_ARGUMENT;
    for (int s = 0; s < lay->num_seqs; ++s) {
      long long len = lay->seq_offsets[s + 1] - lay->seq_offsets[s];
      if (len < 0) return TOPLOC_ERR_INVALID_ARGUMENT;
      n += (len + lay->chunk_len - 1) / lay->chunk_len;
      if (len > longest) longest = len;
    }
  } else {
    if (lay->tokens_per_seq <= 0) return TOPLOC_ERR_INVALID_ARGUMENT;
    long long cps = (lay->tokens_per_seq + lay->chunk_len - 1) / lay->chunk_len;
    if (cps > 0x7FFFFFFFll) return TOPLOC_ERR_UNSUPPORTED;
    plan->chunks_per_seq = (int)cps;
    n = cps * lay->num_seqs;
    longest = lay->tokens_per_seq;
  }
  if (n > 0x7FFFFFFFll) return TOPLOC_ERR_UNSUPPORTED;
  plan->num_chunks = n;
  plan->max_seq_rows = longest;
  return TOPLOC_OK;
}

int check_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return TOPLOC_ERR_CUDA;
  static int major_of[64];
  static bool known[64];
  if (dev < 0 || dev >= 64) return TOPLOC_ERR_UNSUPPORTED;
  if (!known[dev]) {
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
      return TOPLOC_ERR_CUDA;
    major_of[dev] = major;
    known[dev] = true;
  }
  return major_of[dev] == 10 ? TOPLOC_OK : TOPLOC_ERR_ARCH;
}

// 0: flat vectors, 1: aligned rows with padding, 2: element-wise
int pick_mode(const void* act, const toploc_layout* lay) {
  const int esz = lay->dtype == TOPLOC_DTYPE_BF16 ? 2 : 4;
  const int vec = 16 / esz;
  const bool aligned = (reinterpret_cast<uintptr_t>(act) % 16 == 0) && (lay->hidden % vec == 0) &&
                       (lay->row_stride % vec == 0);
  if (!aligned) return 2;
  return lay->row_stride == lay->hidden ? 0 : 1;
}

// Fills the device row table of a ragged batch (in the caller's workspace).
int upload_spans(const toploc_layout* lay, const HostPlan& plan, void* d_workspace, size_t workspace_bytes,
                 cudaStream_t stream, const ChunkSpan** d_spans) {
  *d_spans = nullptr;
  if (!plan.ragged || plan.num_chunks == 0) return TOPLOC_OK;
  const size_t need = (size_t)plan.num_chunks * sizeof(ChunkSpan);
  if (d_workspace == nullptr || workspace_bytes < need) return TOPLOC_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(d_workspace) % 8 != 0) return TOPLOC_ERR_INVALID_ARGUMENT;
  ChunkSpan* spans = static_cast<ChunkSpan*>(malloc(need));
  if (spans == nullptr) return TOPLOC_ERR_INVALID_ARGUMENT;
  long long c = 0;
  for (int s = 0; s < lay->num_seqs; ++s) {
    for (long long r = lay->seq_offsets[s]; r < lay->seq_offsets[s + 1]; r += lay->chunk_len) {
      long long left = lay->seq_offsets[s + 1] - r;
      spans[c].row0 = r;
      spans[c].rows = (int)(left < lay->chunk_len ? left : lay->chunk_len);
      spans[c].pad = 0;
      ++c;
    }
  }
  // pageable source: the runtime has staged the bytes by the time this returns
  cudaError_t err = cudaMemcpyAsync(d_workspace, spans, need, cudaMemcpyHostToDevice, stream);
  free(spans);
  if (err != cudaSuccess) return TOPLOC_ERR_CUDA;
  *d_spans = static_cast<const ChunkSpan*>(d_workspace);
  return TOPLOC_OK;
}

BatchParams make_params(const void* d_act, const toploc_layout* lay, const HostPlan& plan,
                        const ChunkSpan* d_spans) {
  BatchParams bp;
  bp.act = d_act;
  bp.row_stride = lay->row_stride;
  bp.tokens_per_seq = lay->tokens_per_seq;
  bp.spans = d_spans;
  bp.hidden = lay->hidden;
  bp.chunk_len = lay->chunk_len;
  bp.k = lay->k;
  bp.chunks_per_seq = plan.chunks_per_seq;
  return bp;
}

template <int DT>
void launch_build(int mode, unsigned grid, cudaStream_t stream, const BatchParams& bp, const BuildOut& out) {
  if (mode == 0) toploc_build_kernel<DT, 0><<<grid, kThreads, 0, stream>>>(bp, out);
  else if (mode == 1) toploc_build_kernel<DT, 1><<<grid, kThreads, 0, stream>>>(bp, out);
  else toploc_build_kernel<DT, 2><<<grid, kThreads, 0, stream>>>(bp, out);
}

template <int DT>
void launch_verify(int mode, unsigned grid, cudaStream_t stream, const BatchParams& bp, const VerifyIo& io) {
  if (mode == 0) toploc_verify_kernel<DT, 0><<<grid, kThreads, 0, stream>>>(bp, io);
  else if (mode == 1) toploc_verify_kernel<DT, 1><<<grid, kThreads, 0, stream>>>(bp, io);
  else toploc_verify_kernel<DT, 2><<<grid, kThreads, 0, stream>>>(bp, io);
}

size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Carves the staging buffer of the *_host entry points for a group of
// sequences: activations, per-chunk outputs, proofs, ragged row table.
struct StagingPlan {
  size_t act_off, small_off, proofs_off, spans_off, total;
};

StagingPlan carve_staging(const toploc_layout* lay, long long rows, long long chunks, size_t small_elem) {
  const size_t esz = lay->dtype == TOPLOC_DTYPE_BF16 ? 2 : 4;
  StagingPlan sp;
  sp.act_off = 0;
  size_t off = round_up((size_t)rows * (size_t)lay->row_stride * esz, 256);
  sp.small_off = off;
  off += round_up((size_t)chunks * small_elem, 256);
  sp.proofs_off = off;
  off += round_up((size_t)chunks * (2 + 2 * (size_t)lay->k), 256);
  sp.spans_off = off;
  off += round_up((size_t)chunks * sizeof(ChunkSpan), 256);
  sp.total = off;
  return sp;
}

long long seq_begin(const toploc_layout* lay, int s) {
  return lay->seq_offsets ? lay->seq_offsets[s] : (long long)s * lay->tokens_per_seq;
}

long long chunks_between(const toploc_layout* lay, int s0, int s1) {
  long long n = 0;
  for (int s = s0; s < s1; ++s) {
    long long len = seq_begin(lay, s + 1) - seq_begin(lay, s);
    n += (len + lay->chunk_len - 1) / lay->chunk_len;
  }
  return n;
}

}  // namespace

// ===========================================================================
// C ABI
// ===========================================================================
extern "C" {

int64_t toploc_num_chunks(const toploc_layout* lay) {
  HostPlan plan;
  int rc = plan_layout(lay, &plan);
  return rc != TOPLOC_OK ? (int64_t)rc : (int64_t)plan.num_chunks;
}

size_t toploc_proof_bytes(int32_t k) { return k > 0 ? 2 + 2 * (size_t)k : 0; }

size_t toploc_workspace_bytes(const toploc_layout* lay) {
  HostPlan plan;
  if (plan_layout(lay, &plan) != TOPLOC_OK || !plan.ragged) return 0;
  return (size_t)plan.num_chunks * sizeof(ChunkSpan);
}

size_t toploc_staging_bytes(const toploc_layout* lay) {
  HostPlan plan;
  if (plan_layout(lay, &plan) != TOPLOC_OK) return 0;
  long long chunks = (plan.max_seq_rows + lay->chunk_len - 1) / lay->chunk_len;
  return carve_staging(lay, plan.max_seq_rows, chunks, sizeof(toploc_chunk_result)).total;
}

void toploc_get_constants(uint32_t* p, uint32_t* m_lo, uint32_t* m_hi) {
  if (p) *p = kPrime;
  if (m_lo) *m_lo = kModLow;
  if (m_hi) *m_hi = kModHigh;
}

const char* toploc_status_string(int s) {
  switch (s) {
    case TOPLOC_CHUNK_OK: return "ok";
    case TOPLOC_CHUNK_NO_INJECTIVE_MODULUS: return "no injective modulus in [32769, 65536]";
    case TOPLOC_CHUNK_K_EXCEEDS_CHUNK: return "chunk has fewer than k elements";
    case TOPLOC_CHUNK_BAD_PROOF: return "malformed proof (modulus or coefficient out of range)";
    case TOPLOC_CHUNK_NONFINITE_COMMITTED: return "a committed 16-bit pattern is >= p";
    default: return "unknown chunk status";
  }
}

const char* toploc_error_string(int rc) {
  switch (rc) {
    case TOPLOC_OK: return "ok";
    case TOPLOC_ERR_INVALID_ARGUMENT: return "invalid argument";
    case TOPLOC_ERR_UNSUPPORTED: return "unsupported dtype, k or chunk size";
    case TOPLOC_ERR_WORKSPACE: return "workspace or staging buffer too small";
    case TOPLOC_ERR_CUDA: return "CUDA runtime error";
    case TOPLOC_ERR_ARCH: return "device is not compute capability 10.x";
    default: return "unknown error";
  }
}

int toploc_build_proofs(const void* d_act, const toploc_layout* lay, uint8_t* d_proofs, uint8_t* d_status,
                        int32_t* d_indices_opt, void* d_workspace, size_t workspace_bytes,
                        void* cuda_stream) {
  HostPlan plan;
  int rc = plan_layout(lay, &plan);
  if (rc != TOPLOC_OK) return rc;
  if (d_act == nullptr || d_proofs == nullptr || d_status == nullptr) return TOPLOC_ERR_INVALID_ARGUMENT;
  if (reinterpret_cast<uintptr_t>(d_proofs) % 2 != 0) return TOPLOC_ERR_INVALID_ARGUMENT;
  if ((rc = check_device()) != TOPLOC_OK) return rc;
  if (plan.num_chunks == 0) return TOPLOC_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const ChunkSpan* d_spans = nullptr;
  if ((rc = upload_spans(lay, plan, d_workspace, workspace_bytes, stream, &d_spans)) != TOPLOC_OK) return rc;
  const BatchParams bp = make_params(d_act, lay, plan, d_spans);
  BuildOut out;
  out.proofs = d_proofs;
  out.status = d_status;
  out.indices = d_indices_opt;
  const int mode = pick_mode(d_act, lay);
  if (lay->dtype == TOPLOC_DTYPE_BF16) launch_build<0>(mode, (unsigned)plan.num_chunks, stream, bp, out);
  else launch_build<1>(mode, (unsigned)plan.num_chunks, stream, bp, out);
  return cudaGetLastError() == cudaSuccess ? TOPLOC_OK : TOPLOC_ERR_CUDA;
}

int toploc_verify_proofs(const void* d_act, const toploc_layout* lay, const uint8_t* d_proofs,
                         const toploc_thresholds* thr, toploc_chunk_result* d_results,
                         const int32_t* d_gen_indices_opt, void* d_workspace, size_t workspace_bytes,
                         void* cuda_stream) {
  HostPlan plan;
  int rc = plan_layout(lay, &plan);
  if (rc != TOPLOC_OK) return rc;
  if (d_act == nullptr || d_proofs == nullptr || thr == nullptr || d_results == nullptr)
    return TOPLOC_ERR_INVALID_ARGUMENT;
  if (reinterpret_cast<uintptr_t>(d_proofs) % 2 != 0 || reinterpret_cast<uintptr_t>(d_results) % 8 != 0)
    return TOPLOC_ERR_INVALID_ARGUMENT;
  if (thr->t_exp < 0) return TOPLOC_ERR_INVALID_ARGUMENT;
  if ((rc = check_device()) != TOPLOC_OK) return rc;
  if (plan.num_chunks == 0) return TOPLOC_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const ChunkSpan* d_spans = nullptr;
  if ((rc = upload_spans(lay, plan, d_workspace, workspace_bytes, stream, &d_spans)) != TOPLOC_OK) return rc;
  const BatchParams bp = make_params(d_act, lay, plan, d_spans);
  VerifyIo io;
  io.proofs = d_proofs;
  io.results = d_results;
  io.gen_indices = d_gen_indices_opt;
  io.t_exp = thr->t_exp;
  io.sign_in_exponent = thr->sign_in_exponent;
  io.t_mean = thr->t_mean;
  io.t_median = thr->t_median;
  const int mode = pick_mode(d_act, lay);
  if (lay->dtype == TOPLOC_DTYPE_BF16) launch_verify<0>(mode, (unsigned)plan.num_chunks, stream, bp, io);
  else launch_verify<1>(mode, (unsigned)plan.num_chunks, stream, bp, io);
  return cudaGetLastError() == cudaSuccess ? TOPLOC_OK : TOPLOC_ERR_CUDA;
}

// Shared driver of the two host-memory entry points: groups of whole sequences
// go host -> staging -> kernel -> host, in stream order.
static int run_from_host(bool verify, const void* h_act, const toploc_layout* lay, uint8_t* h_proofs_out,
                         const uint8_t* h_proofs_in, uint8_t* h_status, const toploc_thresholds* thr,
                         toploc_chunk_result* h_results, void* d_staging, size_t staging_bytes,
                         void* cuda_stream) {
  HostPlan plan;
  int rc = plan_layout(lay, &plan);
  if (rc != TOPLOC_OK) return rc;
  if (h_act == nullptr || d_staging == nullptr) return TOPLOC_ERR_INVALID_ARGUMENT;
  if (reinterpret_cast<uintptr_t>(d_staging) % 256 != 0) return TOPLOC_ERR_INVALID_ARGUMENT;
  if (staging_bytes < toploc_staging_bytes(lay)) return TOPLOC_ERR_WORKSPACE;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const size_t esz = lay->dtype == TOPLOC_DTYPE_BF16 ? 2 : 4;
  const size_t pb = 2 + 2 * (size_t)lay->k;
  const size_t small_elem = verify ? sizeof(toploc_chunk_result) : 1;
  char* stage = static_cast<char*>(d_staging);
  int64_t* rebased = static_cast<int64_t*>(malloc(((size_t)lay->num_seqs + 1) * sizeof(int64_t)));
  if (rebased == nullptr) return TOPLOC_ERR_INVALID_ARGUMENT;
  long long chunk0 = 0;
  int s0 = 0;
  while (s0 < lay->num_seqs && rc == TOPLOC_OK) {
    // largest group of sequences starting at s0 that fits
    int s1 = s0 + 1;
    StagingPlan sp = carve_staging(lay, seq_begin(lay, s1) - seq_begin(lay, s0), chunks_between(lay, s0, s1),
                                   sizeof(toploc_chunk_result));
    while (s1 < lay->num_seqs) {
      StagingPlan bigger = carve_staging(lay, seq_begin(lay, s1 + 1) - seq_begin(lay, s0),
                                         chunks_between(lay, s0, s1 + 1), sizeof(toploc_chunk_result));
      if (bigger.total > staging_bytes) break;
      sp = bigger;
      ++s1;
    }
    const long long row_a = seq_begin(lay, s0), row_b = seq_begin(lay, s1);
    const long long chunks = chunks_between(lay, s0, s1);
    if (row_b > row_a && chunks > 0) {
      toploc_layout sub = *lay;
      sub.num_seqs = s1 - s0;
      if (lay->seq_offsets) {
        for (int s = s0; s <= s1; ++s) rebased[s - s0] = lay->seq_offsets[s] - row_a;
        sub.seq_offsets = rebased;
      }
      const size_t act_bytes = (size_t)(row_b - row_a) * (size_t)lay->row_stride * esz;
      const char* src = static_cast<const char*>(h_act) + (size_t)row_a * (size_t)lay->row_stride * esz;
      if (cudaMemcpyAsync(stage + sp.act_off, src, act_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        rc = TOPLOC_ERR_CUDA;
      if (rc == TOPLOC_OK && !verify) {
        rc = toploc_build_proofs(stage + sp.act_off, &sub, reinterpret_cast<uint8_t*>(stage + sp.proofs_off),
                                 reinterpret_cast<uint8_t*>(stage + sp.small_off), nullptr,
                                 stage + sp.spans_off, sp.total - sp.spans_off, stream);
        if (rc == TOPLOC_OK &&
            (cudaMemcpyAsync(h_proofs_out + (size_t)chunk0 * pb, stage + sp.proofs_off, (size_t)chunks * pb,
                             cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
             cudaMemcpyAsync(h_status + chunk0, stage + sp.small_off, (size_t)chunks, cudaMemcpyDeviceToHost,
                             stream) != cudaSuccess))
          rc = TOPLOC_ERR_CUDA;
      } else if (rc == TOPLOC_OK) {
        if (cudaMemcpyAsync(stage + sp.proofs_off, h_proofs_in + (size_t)chunk0 * pb, (size_t)chunks * pb,
                            cudaMemcpyHostToDevice, stream) != cudaSuccess)
          rc = TOPLOC_ERR_CUDA;
        if (rc == TOPLOC_OK)
          rc = toploc_verify_proofs(stage + sp.act_off, &sub, reinterpret_cast<uint8_t*>(stage + sp.proofs_off),
                                    thr, reinterpret_cast<toploc_chunk_result*>(stage + sp.small_off), nullptr,
                                    stage + sp.spans_off, sp.total - sp.spans_off, stream);
        if (rc == TOPLOC_OK &&
            cudaMemcpyAsync(h_results + chunk0, stage + sp.small_off, (size_t)chunks * small_elem,
                            cudaMemcpyDeviceToHost, stream) != cudaSuccess)
          rc = TOPLOC_ERR_CUDA;
      }
      // the ragged row table of this group is read from `rebased` before the call returns,
      // and staged copies of pageable memory are complete on return: safe to reuse both
    }
    chunk0 += chunks;
    s0 = s1;
  }
  free(rebased);
  if (cudaStreamSynchronize(stream) != cudaSuccess && rc == TOPLOC_OK) rc = TOPLOC_ERR_CUDA;
  return rc;
}

int toploc_build_proofs_host(const void* h_act, const toploc_layout* lay, uint8_t* h_proofs, uint8_t* h_status,
                             void* d_staging, size_t staging_bytes, void* cuda_stream) {
  if (h_proofs == nullptr || h_status == nullptr) return TOPLOC_ERR_INVALID_ARGUMENT;
  return run_from_host(false, h_act, lay, h_proofs, nullptr, h_status, nullptr, nullptr, d_staging,
                       staging_bytes, cuda_stream);
}

int toploc_verify_proofs_host(const void* h_act, const toploc_layout* lay, const uint8_t* h_proofs,
                              const toploc_thresholds* thr, toploc_chunk_result* h_results, void* d_staging,
                              size_t staging_bytes, void* cuda_stream) {
  if (h_proofs == nullptr || thr == nullptr || h_results == nullptr) return TOPLOC_ERR_INVALID_ARGUMENT;
  return run_from_host(true, h_act, lay, nullptr, h_proofs, nullptr, thr, h_results, d_staging, staging_bytes,
                       cuda_stream);
}

}  // extern "C"
