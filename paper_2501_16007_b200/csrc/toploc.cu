// TopLoc proof hot path for sm_100a.
//
// Proof generation, two kernels per call:
//   select        one warp (a 32-thread block) per chunk streams the chunk from
//                 HBM exactly once and keeps the exact top-k on chip (Algorithm 1,
//                 topk()), then runs the injective-modulus search (Algorithm 6).
//                 The k (index, pattern) pairs go to scratch memory.
//   interpolate   one warp per chunk does the arithmetic over Z_p: Newton
//                 interpolation and packing (Algorithm 3).  fp32 chunks that
//                 commit whole patterns use a second interpolation kernel over
//                 Z_q, q = 2^32 - 5.
// Validation, one kernel per call:
//   verify        the same selection (Algorithm 2, topk()), after which the same
//                 warp evaluates the committed polynomial at its k points
//                 (Algorithm 5), compares bit fields, and writes statistics and
//                 verdict.  Nothing goes through scratch memory.
// Around these:
//   merge         a chunk too long for one warp (a prompt as one chunk) is
//                 selected in segments by the select kernel; the merge kernel
//                 joins the segments' winners and runs the tail of its call.
//   stream        incremental proof generation: one new row per sequence and
//                 decode step updates a running selection kept in device memory.
//
// The path is a selection over data read once plus integer modular arithmetic:
// HBM bandwidth is the roofline, there is no dense contraction and therefore no
// tensor-core work.  The selection keeps its loads in flight as asynchronous
// copies into a small shared-memory ring per warp (many independent warps per
// SM, none waits on another) and spends about one instruction per seven
// elements on the elements that lose.
#include "toploc.h"
#include "toploc_device.cuh"

#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>

namespace {

using namespace toploc_device;

constexpr int kMaxK = TOPLOC_MAX_K;                 // polynomial proofs: largest k
constexpr int kSmallMaxK = SelectShared::kMaxK;     // up to here the smaller per-warp scratch serves

// ---------------------------------------------------------------------------
// constants of the method
// ---------------------------------------------------------------------------
constexpr uint32_t kPrime = 65521u;      // field modulus: largest prime below 2^16
constexpr uint32_t kPrime32 = 4294967291u;  // 32-bit field (fp32 chunks committing whole patterns): 2^32 - 5
constexpr uint32_t kModHigh = 65536u;    // Algorithm 6 scans 65536 down to 2^15 + 1
constexpr uint32_t kModLow = 32769u;

// Programmatic dependent launch.  A kernel that is followed in its stream by the interpolation
// kernel lets that grid be scheduled early (its blocks need an SM almost to themselves, so they
// only land where this grid has drained); the interpolation kernel builds its table of inverses
// and then waits here until the whole grid before it has finished and its writes are visible.
// Without a dependent launch behind it (or before it) both are no-ops.
__device__ __forceinline__ void allow_dependent_launch() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void wait_for_previous_grid() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

constexpr int kInterpWarps = 32;         // interpolation kernel: warps per block
#ifndef TOPLOC_INTERP_CHUNKS
#define TOPLOC_INTERP_CHUNKS 2
#endif
constexpr int kInterpChunks = TOPLOC_INTERP_CHUNKS;  // interpolation kernel: chunks a warp works on at once
// k above 256: sixteen slots per lane need more registers than a 1024-thread block has, so those
// chunks go to 512-thread blocks, one chunk per warp at a time.
constexpr int kInterpWarpsBig = 16;
static_assert((65536 + kInterpWarps * 2 * kInterpChunks * kSmallMaxK) * 2 <= 227 * 1024 &&
                  (65536 + kInterpWarpsBig * 2 * kMaxK) * 2 <= 227 * 1024,
              "table of inverses + per-warp rows must fit the shared memory of one block");

struct ChunkSpan {   // one per chunk of a ragged batch, built on the host
  long long row0;
  int rows;
  int pad;
};

// Long chunks (a prompt processed as one chunk) are selected in segments of
// whole rows, one warp per segment, and the segments' winners are merged.
struct ChunkSegments {  // one per chunk of a batch that holds a long chunk, built on the host
  long long row0;       // first row of the chunk
  int first_seg;        // its segments are first_seg .. first_seg + n_segs - 1
  int n_segs;
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
  int coef_bytes;              // 2: coefficients in Z_p; 4: fp32 chunks over Z_q, q = 2^32 - 5
  int padded;                  // validation only: fp32 chunks against Z_p proofs, commitments padded to 32 bits
};

__device__ __forceinline__ size_t proof_stride(const BatchParams& bp) { return 2 + (size_t)bp.coef_bytes * bp.k; }
__device__ __forceinline__ int proof_words(const BatchParams& bp) { return 1 + (bp.coef_bytes / 2) * bp.k; }

// What the select kernel leaves behind for the interpolation kernel (or hands to the caller).
struct Selection {
  uint32_t* idx;       // [num_chunks, k] selected flat indices
  uint16_t* bits;      // [num_chunks, k] their 16-bit patterns
  uint32_t* bits32;    // 32-bit field: [num_chunks, k] their whole patterns instead
  uint8_t* status;     // [num_chunks] TOPLOC_CHUNK_*; the caller's d_status during proof generation
  uint8_t* proofs;     // proof generation only: receives the modulus (or zeros)
  int32_t* indices;    // optional: indices in rank order
};

// Inputs of the merge kernel: the per-segment selections (indices local to the segment).
struct MergeParams {
  const ChunkSegments* chunks;
  const ChunkSpan* segs;
  const uint32_t* seg_idx;      // [num_segs, k]
  const uint16_t* seg_bits;     // [num_segs, k] (unused by fp32 chunks, whose patterns are read again)
  const uint8_t* seg_status;    // [num_segs]
  unsigned long long* words;    // [num_segs, k] scratch: the candidates of a chunk as ranking words
};

struct VerifyIo {
  const uint8_t* proofs;
  toploc_chunk_result* results;
  const int32_t* gen_indices;  // optional
  toploc_thresholds thr;              // thresholds of the call ...
  const toploc_thresholds* thr_each;  // ... or, when not null, one entry per chunk (device memory)
};

// The thresholds chunk `chunk` is judged by.
__device__ __forceinline__ toploc_thresholds thresholds_of(const VerifyIo& io, long long chunk) {
  return io.thr_each ? io.thr_each[chunk] : io.thr;
}

// Algorithm 2's verdict: reject iff a statistic exceeds its threshold (strictly), or nothing matched.
__device__ __forceinline__ bool rejects(const toploc_thresholds& t, const toploc_chunk_result& res) {
  if (res.n_match == 0) return true;  // nothing matched: nothing to accept on
  return ((long long)res.exp_mismatch > (long long)t.t_exp) || (res.mant_mean > t.t_mean) ||
         (res.mant_median > t.t_median);
}

// ---------------------------------------------------------------------------
// arithmetic in Z_p (all operands < p < 2^16, so a * b + c fits 32 bits)
// ---------------------------------------------------------------------------
__host__ __device__ constexpr uint32_t mul_mod(uint32_t a, uint32_t b) { return (a * b) % kPrime; }
__device__ __forceinline__ uint32_t mad_mod(uint32_t a, uint32_t b, uint32_t c) { return (a * b + c) % kPrime; }
// a - b in Z_p, given neg_b = p - b (in (0, p]).
__device__ __forceinline__ uint32_t diff_mod(uint32_t a, uint32_t neg_b) {
  const uint32_t d = a + neg_b;   // in (0, 2p)
  return min(d, d - kPrime);      // d - p wraps to a huge value when d < p
}

__host__ __device__ constexpr uint32_t pow_mod(uint32_t a, uint32_t e) {
  uint32_t r = 1;
  while (e) {
    if (e & 1u) r = mul_mod(r, a);
    a = mul_mod(a, a);
    e >>= 1;
  }
  return r;
}

// Smallest generator of the multiplicative group of Z_p (p - 1 = 2^4 3^2 5 7 13).
constexpr uint32_t find_generator() {
  for (uint32_t g = 2; g < kPrime; ++g) {
    bool ok = true;
    for (uint32_t q : {2u, 3u, 5u, 7u, 13u})
      if (pow_mod(g, (kPrime - 1) / q) == 1u) ok = false;
    if (ok) return g;
  }
  return 0;
}
constexpr uint32_t kGenerator = find_generator();
constexpr uint32_t kGeneratorInv = pow_mod(kGenerator, kPrime - 2);
static_assert(kGenerator != 0 && mul_mod(kGenerator, kGeneratorInv) == 1u, "generator of Z_p^*");

// Algorithm 6: largest m in [2^15 + 1, 2^16] for which the selected indices
// stay distinct as (index mod m) mod p -- the second reduction because the
// x-coordinates live in Z_p and m may exceed p (in the 32-bit field m < q and
// Algorithm 6 applies as printed).  Returns 0 if there is none.
// idx[e] is the flat index of point 32 e + lane.  The selection in shared
// memory is consumed: the tile ring and the candidate buffer become the
// 65536-bit set of residues seen.  Run by one warp (the only one of its block
// that is still at work).
template <class SH>
__device__ uint32_t find_injective_modulus(SH& sh, int k, const uint32_t (&idx)[SH::kMaxK / kThreads],
                                           bool wide_field) {
  constexpr int kOwned = SH::kMaxK / kThreads;
  const int lane = threadIdx.x & 31;
  uint32_t res[kOwned];
#pragma unroll
  for (int e = 0; e < kOwned; ++e) res[e] = 0;
  warp_barrier();  // every lane has taken its candidates out of sh.cand
  uint32_t* seen = reinterpret_cast<uint32_t*>(sh.ring);  // ring and cand are adjacent: 11 KB
  for (int i = lane; i < 2048; i += kThreads) seen[i] = 0;
  warp_barrier();
  uint32_t found = 0;
#pragma unroll 1
  for (uint32_t m = kModHigh; m >= kModLow; --m) {
    uint32_t dup = 0;
#pragma unroll
    for (int e = 0; e < kOwned; ++e) {
      int j = lane + e * kThreads;
      if (j < k) {
        uint32_t r = idx[e] % m;
        if (!wide_field && r >= kPrime) r -= kPrime;  // every residue is below q = 2^32 - 5 as it is
        res[e] = r;
        uint32_t bit = 1u << (r & 31u);
        dup |= atomicOr(&seen[r >> 5], bit) & bit;
      }
    }
    const bool clash = __any_sync(0xFFFFFFFFu, dup != 0);  // also orders the set's updates before its clearing
#pragma unroll
    for (int e = 0; e < kOwned; ++e) {
      int j = lane + e * kThreads;
      if (j < k) seen[res[e] >> 5] = 0;
    }
    warp_barrier();
    if (!clash) {
      found = m;
      break;
    }
  }
  return found;
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
// select kernel: topk() of Algorithms 1 and 2, one chunk per block; for proof
// generation (sel.proofs != nullptr) also findInjectiveModulus() of Algorithm 1.
// ---------------------------------------------------------------------------
template <int DT, class SH>
__device__ __forceinline__ void publish_selection(SH& sh, const BatchParams& bp, long long chunk,
                                                  const Selection& sel);

// one-warp blocks per SM the launch bound asks for (shared memory allows one or two more)
template <class SH>
constexpr int select_min_blocks() { return SH::kMaxK > 256 ? 13 : TOPLOC_SELECT_MIN_BLOCKS; }

template <int DT, int MODE, class SH>
__global__ void __launch_bounds__(kThreads, select_min_blocks<SH>()) toploc_select_kernel(BatchParams bp, Selection sel) {
  __shared__ SH sh;
  const int tid = threadIdx.x;
  const long long chunk = blockIdx.x;
  const int k = bp.k;
  uint16_t* proof = sel.proofs ? reinterpret_cast<uint16_t*>(sel.proofs + chunk * proof_stride(bp)) : nullptr;
  int32_t* indices = sel.indices ? sel.indices + chunk * k : nullptr;
  allow_dependent_launch();

  const ChunkPlace pl = locate_chunk<DT>(bp, chunk);
  const long long n_elems = (long long)pl.rows * bp.hidden;
  if (n_elems < k) {
    if (proof)
      for (int i = tid; i < proof_words(bp); i += kThreads) proof[i] = 0;
    if (indices)
      for (int i = tid; i < k; i += kThreads) indices[i] = 0;
    if (tid == 0) sel.status[chunk] = TOPLOC_CHUNK_K_EXCEEDS_CHUNK;
    return;
  }
  ChunkSource<DT, MODE> src;
  src.base = pl.base;
  src.row_stride = bp.row_stride;
  src.hidden = bp.hidden;
  src.vecs_per_row = bp.hidden / ChunkSource<DT, MODE>::kVec;
  select_topk<DT, MODE>(sh, src, (int)n_elems, k);
  publish_selection<DT>(sh, bp, chunk, sel);
}

// The chunk's selection (sh.cand[0..k)) goes to the interpolation kernel: indices
// and patterns to scratch, rank order where the caller asked for indices, and
// for proof generation the modulus (Algorithm 6) and the chunk's status.
template <int DT, class SH>
__device__ __forceinline__ void publish_selection(SH& sh, const BatchParams& bp, long long chunk,
                                                  const Selection& sel) {
  const int tid = threadIdx.x;
  const int k = bp.k;
  uint16_t* proof = sel.proofs ? reinterpret_cast<uint16_t*>(sel.proofs + chunk * proof_stride(bp)) : nullptr;
  const bool wide = DT == 1 && bp.coef_bytes == 4;
  int32_t* indices = sel.indices ? sel.indices + chunk * k : nullptr;
  uint32_t unrepresentable = 0;
  for (int j = tid; j < k; j += kThreads) {
    const unsigned long long cj = sh.cand[j];
    const uint32_t key = (uint32_t)(cj >> (kIdxBits + 1));
    const uint32_t sign = (uint32_t)cj & 1u;
    const uint32_t flat = kIdxMask - ((uint32_t)(cj >> 1) & kIdxMask);
    sel.idx[chunk * k + j] = flat;
    if (wide) {
      const uint32_t pattern = (sign << 31) | key;
      unrepresentable |= pattern >= kPrime32;
      sel.bits32[chunk * k + j] = pattern;
    } else {
      const uint32_t bits = (sign << 15) | (DT == 0 ? key : (key >> 16));
      unrepresentable |= bits >= kPrime;
      sel.bits[chunk * k + j] = (uint16_t)bits;
    }
    if (indices) {
      int rank = 0;  // position = number of better candidates
      for (int i = 0; i < k; ++i) rank += sh.cand[i] > cj;
      indices[rank] = (int32_t)flat;
    }
  }
  if (proof == nullptr) {
    if (tid == 0) sel.status[chunk] = TOPLOC_CHUNK_OK;
    return;
  }
  const bool nonfinite = __any_sync(0xFFFFFFFFu, unrepresentable != 0);
  uint32_t picked[SH::kMaxK / kThreads];
#pragma unroll
  for (int e = 0; e < SH::kMaxK / kThreads; ++e) {
    const int j = tid + e * kThreads;
    picked[e] = j < k ? kIdxMask - ((uint32_t)(sh.cand[j] >> 1) & kIdxMask) : 0u;
  }
  const uint32_t m = find_injective_modulus(sh, k, picked, wide);
  if (m == 0) {
    for (int i = tid; i < proof_words(bp); i += kThreads) proof[i] = 0;
    if (tid == 0) sel.status[chunk] = TOPLOC_CHUNK_NO_INJECTIVE_MODULUS;
    return;
  }
  if (tid == 0) {
    proof[0] = (uint16_t)(m & 0xFFFFu);  // 65536 is stored as 0
    sel.status[chunk] = nonfinite ? TOPLOC_CHUNK_NONFINITE_COMMITTED : TOPLOC_CHUNK_OK;
  }
}

// ---------------------------------------------------------------------------
// arithmetic over Z_p, one warp per chunk.  Entry j of a chunk's k points
// belongs to lane j % 32, slot j / 32 of that lane.
// ---------------------------------------------------------------------------

// Algorithm 3 for NCH chunks of one warp at a time (their dependency chains are
// independent, which keeps the issue slots filled).  inv[] is the table of
// inverses in Z_p; xa is this warp's scratch (NCH rows of ROW words: x_i in the
// lower half of word i, the Newton coefficient a_i in the upper half).  A chunk
// that is not live is carried along with zeros and not written.
//
// The Newton coefficients are the divided differences of Algorithm 3, reached
// without a division per pair of points: with P_{i-1} the interpolant of the
// first i points and N_i(x) = prod_{l < i} (x - x_l),
//   a_i = (y_i - P_{i-1}(x_i)) / N_i(x_i).
// Every point j carries t_j = y_j - P_{i-1}(x_j) and n_j = N_i(x_j); step i takes
// a_i = t_i / n_i from point i (ONE look-up in the table of inverses, at an
// address the whole warp shares, so it is a broadcast and not a gather) and
// every later point does  t_j <- t_j - a_i n_j,  n_j <- n_j (x_j - x_i).  Point j
// lives in lane j % 32, slot j / 32; only a_i and x_i travel between lanes.
// (One division per pair, t_j <- (t_j - a_i) / (x_j - x_i), costs the same
// arithmetic but k^2 / 2 gathers from the table per chunk; their bank conflicts
// made shared memory the bottleneck: 0.47 ms per launch on the 70B-shaped batch
// against 0.39 ms this way, which is bound by the integer-multiply pipe.)
// The Newton form is then multiplied out from the inside,
//   P <- a_{k-1};  P <- P * (x - x_i) + a_i  for i = k-2 .. 0.
template <int SLOTS, int NCH, int ROW>
__device__ __forceinline__ void interpolate_chunks(const uint16_t* inv, uint32_t* xa, int k, const Selection& sel,
                                                   const long long (&chunk)[NCH], const bool (&live)[NCH]) {
  const int lane = threadIdx.x & 31;
  constexpr uint32_t kFull = 0xFFFFFFFFu;
  const size_t proof_bytes = 2 + 2 * (size_t)k;
  // The last quarter of the slots keeps plain divided differences instead of (t, n): for them a
  // step is t_j <- (t_j - a_i) / (x_j - x_i), one modular multiplication and one gather from the
  // table of inverses per pair, and a point that becomes the pivot hands out a_i = t_i as it is.
  // Both forms yield the same a_i, so they mix freely; this share of gathers is what the
  // shared-memory pipe takes while the integer-multiply pipe is busy with the other slots
  // (generate minus select on the 70B-shaped batch: 0.50-0.51 ms against 0.54-0.55 ms with no
  // gathers at all, 0.45-0.53 ms with half the slots gathering; all under the power cap).
  constexpr int A_FROM = (SLOTS == 4 || SLOTS == 8) ? SLOTS * 3 / 4 : SLOTS;  // (sixteen slots: too much code to mix)
  uint32_t x[NCH][SLOTS], t[NCH][SLOTS], n[NCH][SLOTS];
#pragma unroll
  for (int c = 0; c < NCH; ++c) {
    uint32_t m = 65536u;
    if (live[c]) {
      m = reinterpret_cast<const uint16_t*>(sel.proofs + chunk[c] * proof_bytes)[0];
      if (m == 0) m = 65536u;
    }
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) {
      const int j = s * 32 + lane;
      x[c][s] = 0;
      t[c][s] = 0;
      n[c][s] = 1;
      if (j < k && live[c]) {
        uint32_t r = sel.idx[chunk[c] * k + j] % m;  // i_m = i mod m, then into Z_p
        if (r >= kPrime) r -= kPrime;
        uint32_t y = sel.bits[chunk[c] * k + j];     // Algorithm 3 starts from y mod M
        if (y >= kPrime) y -= kPrime;
        x[c][s] = r;
        t[c][s] = y;
      }
    }
  }
  // Steps i = 32 b + ii: the points of slot b in lanes above ii and every point of the later
  // slots take part (no per-slot tests inside the loop).
#pragma unroll
  for (int b = 0; b < SLOTS; ++b) {
    const int steps = min(32, k - 32 * b);  // the last point only yields its coefficient
#pragma unroll 1
    for (int ii = 0; ii < steps; ++ii) {
      const int i = 32 * b + ii;
      uint32_t neg_a[NCH], neg_x[NCH];
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        const uint32_t ni = __shfl_sync(kFull, n[c][b], ii);
        const uint32_t ti = __shfl_sync(kFull, t[c][b], ii);
        const uint32_t xi = __shfl_sync(kFull, x[c][b], ii);
        const uint32_t a = b < A_FROM ? mul_mod(ti, inv[ni]) : ti;  // n_i != 0: the x are distinct (Algorithm 6)
        if (lane == 0) xa[c * ROW + i] = xi | (a << 16);
        neg_a[c] = kPrime - a;
        neg_x[c] = kPrime - xi;
      }
      const bool later = lane > ii;
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        // a point at or before i computes values that are dropped
        if (b < A_FROM) {
          const uint32_t tb = mad_mod(neg_a[c], n[c][b], t[c][b]);
          const uint32_t nb = mul_mod(n[c][b], diff_mod(x[c][b], neg_x[c]));
          t[c][b] = later ? tb : t[c][b];
          n[c][b] = later ? nb : n[c][b];
        } else {
          const uint32_t tb = mul_mod(diff_mod(t[c][b], neg_a[c]), inv[diff_mod(x[c][b], neg_x[c])]);
          t[c][b] = later ? tb : t[c][b];
        }
      }
#pragma unroll
      for (int s = b + 1; s < SLOTS; ++s) {
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
          if (s < A_FROM) {
            t[c][s] = mad_mod(neg_a[c], n[c][s], t[c][s]);
            n[c][s] = mul_mod(n[c][s], diff_mod(x[c][s], neg_x[c]));
          } else {
            t[c][s] = mul_mod(diff_mod(t[c][s], neg_a[c]), inv[diff_mod(x[c][s], neg_x[c])]);
          }
        }
      }
    }
  }
  __syncwarp();
  // The Newton form multiplied out from the inside; after the step for x_i the polynomial has
  // degree D = k - 1 - i.  Coefficient d lives in lane d % 32, slot d / 32: slots above D / 32
  // hold zeros and are skipped, and the shift by one degree is a rotation of every live slot by
  // one lane (lane 0 of a slot takes lane 31 of the slot below, lane 0 of slot 0 takes a_i).
  uint32_t co[NCH][SLOTS];
#pragma unroll
  for (int c = 0; c < NCH; ++c) {
#pragma unroll
    for (int b = 0; b < SLOTS; ++b) co[c][b] = 0;
    if (lane == 0) co[c][0] = xa[c * ROW + k - 1] >> 16;
  }
  const int from = (lane + 31) & 31;
#pragma unroll
  for (int top = 0; top < SLOTS; ++top) {  // the slot that holds the leading coefficient
    const int d_first = max(32 * top, 1), d_last = min(32 * top + 31, k - 1);
#pragma unroll 1
    for (int D = d_first; D <= d_last; ++D) {
      const int i = k - 1 - D;
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        const uint32_t pair = xa[c * ROW + i];
        const uint32_t neg_x = kPrime - (pair & 0xFFFFu);  // p for x_i = 0, which multiplies like 0
        uint32_t below[SLOTS];  // coefficient d - 1, as seen from the owner of coefficient d
#pragma unroll
        for (int b = 0; b <= top; ++b) below[b] = __shfl_sync(kFull, co[c][b], from);
        // coefficient d takes  c[d-1] + (-x_i) c[d]
#pragma unroll
        for (int b = top; b >= 1; --b) co[c][b] = mad_mod(co[c][b], neg_x, lane == 0 ? below[b - 1] : below[b]);
        co[c][0] = mad_mod(co[c][0], neg_x, lane == 0 ? (pair >> 16) : below[0]);
      }
    }
  }
  // proof bytes 2 + 2d, 3 + 2d: coefficient of degree d, little-endian
#pragma unroll
  for (int c = 0; c < NCH; ++c) {
    if (!live[c]) continue;
    uint16_t* proof = reinterpret_cast<uint16_t*>(sel.proofs + chunk[c] * proof_bytes);
#pragma unroll
    for (int b = 0; b < SLOTS; ++b) {
      const int d = b * 32 + lane;
      if (d < k) proof[1 + d] = (uint16_t)co[c][b];
    }
  }
  __syncwarp();
}

// InterpolateModPolynomial() and encode() of Algorithm 1 for every chunk the
// select kernel finished.  Each block first fills a table of all inverses in
// Z_p (walking the powers of a generator forwards and backwards), then every
// warp takes chunks in turn, kInterpChunks at a time.
// WARPS x 32 threads per block, ROW = the largest k of the instantiation: 32 warps and 256 for
// k <= 256 (two chunks per warp at a time up to k = 128), 16 warps and 512 above.
template <int WARPS, int ROW>
__global__ void __launch_bounds__(WARPS * 32, 1)
toploc_interpolate_kernel(Selection sel, int k, long long num_chunks) {
  constexpr int NCH = ROW > 256 ? 1 : kInterpChunks;  // chunks a warp works on at once
  extern __shared__ __align__(16) uint16_t dyn_smem[];
  uint16_t* inv = dyn_smem;                               // 65536 entries
  uint16_t* scratch = dyn_smem + 65536;                   // NCH rows of ROW words per warp
  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  {
    // thread t owns a run of consecutive exponents of the generator
    constexpr uint32_t kRun = 65536u / (WARPS * 32);
    const uint32_t e0 = (uint32_t)tid * kRun;
    uint32_t a = pow_mod(kGenerator, e0);
    uint32_t b = pow_mod(kGeneratorInv, e0);
    if (tid == 0) inv[0] = 0;
#pragma unroll 4
    for (uint32_t i = 0; i < kRun; ++i) {
      if (e0 + i < kPrime - 1) inv[a] = (uint16_t)b;
      a = mul_mod(a, kGenerator);
      b = mul_mod(b, kGeneratorInv);
    }
  }
  __syncthreads();
  wait_for_previous_grid();  // the selections and moduli are in place
  uint32_t* xa = reinterpret_cast<uint32_t*>(scratch) + warp * NCH * ROW;
  const long long groups = (num_chunks + NCH - 1) / NCH;
  // group g goes to block g % gridDim.x, so a small batch spreads over the blocks before it fills their warps
  for (long long g = blockIdx.x + (long long)gridDim.x * warp; g < groups; g += (long long)gridDim.x * WARPS) {
    long long chunk[NCH];
    bool live[NCH];
    bool any = false;
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      chunk[c] = g * NCH + c;
      live[c] = false;
      if (chunk[c] < num_chunks) {
        const uint8_t st = sel.status[chunk[c]];
        live[c] = st != TOPLOC_CHUNK_NO_INJECTIVE_MODULUS && st != TOPLOC_CHUNK_K_EXCEEDS_CHUNK;
      }
      any |= live[c];
    }
    if (!any) continue;
    if constexpr (ROW > 256) {
      interpolate_chunks<ROW / 32, 1, ROW>(inv, xa, k, sel, chunk, live);
    } else {
      if (k <= 32) interpolate_chunks<1, NCH, ROW>(inv, xa, k, sel, chunk, live);
      else if (k <= 64) interpolate_chunks<2, NCH, ROW>(inv, xa, k, sel, chunk, live);
      else if (k <= 128) interpolate_chunks<4, NCH, ROW>(inv, xa, k, sel, chunk, live);
      else {
        // eight slots per lane: one chunk at a time keeps the state in registers
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
          const long long one_chunk[1] = {chunk[c]};
          const bool one_live[1] = {live[c]};
          if (live[c]) interpolate_chunks<8, 1, ROW>(inv, xa, k, sel, one_chunk, one_live);
        }
      }
    }
  }
}

// decode(), Horner evaluation (Algorithm 5), extractBits(), the error
// accumulation and the verdict of Algorithm 2 for one chunk, by the warp that
// selected it.  res arrives initialised and with the decoded modulus.
template <int SLOTS, class SH>
__device__ __forceinline__ void evaluate_warp(SH& sh, int k, long long chunk, const uint32_t (&idx)[SLOTS],
                                              const uint32_t (&bits)[SLOTS], const VerifyIo& io,
                                              toploc_chunk_result res) {
  const int lane = threadIdx.x;
  const uint16_t* proof = reinterpret_cast<const uint16_t*>(io.proofs + chunk * (2 + 2 * (size_t)k));
  // the selection has left shared memory (it is in idx / bits), so the ring is free
  uint32_t* coef = reinterpret_cast<uint32_t*>(sh.ring);  // SH::kMaxK words
  uint32_t* gen = coef + SH::kMaxK;                       // SH::kMaxK words
  uint32_t* hist = sh.top_hist;                           // a 7-bit mantissa difference is at most 127
  const toploc_thresholds thr = thresholds_of(io, chunk);
  warp_barrier();
  for (int d = lane; d < k; d += 32) coef[d] = proof[1 + d];
  if (io.gen_indices)
    for (int j = lane; j < k; j += 32) gen[j] = (uint32_t)io.gen_indices[chunk * k + j];
  for (int b = lane; b < 128; b += 32) hist[b] = 0;
  warp_barrier();

  const uint32_t m = res.modulus;
  uint32_t x[SLOTS], acc[SLOTS];
#pragma unroll
  for (int s = 0; s < SLOTS; ++s) {
    uint32_t r = idx[s] % m;
    if (r >= kPrime) r -= kPrime;
    x[s] = r;
    acc[s] = coef[k - 1];  // Horner, highest degree first
  }
#pragma unroll 4
  for (int d = k - 2; d >= 0; --d) {
    const uint32_t cd = coef[d];
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) acc[s] = mad_mod(acc[s], x[s], cd);
  }
  uint32_t err_e = 0, diff_sum = 0, common = 0;
#pragma unroll
  for (int s = 0; s < SLOTS; ++s) {
    if (s * 32 + lane >= k) continue;
    const uint32_t seen = bits[s];
    uint32_t e_p = acc[s] >> 7, e_v = seen >> 7;  // sign + 8 exponent bits
    if (!thr.sign_in_exponent) {
      e_p &= 0xFFu;
      e_v &= 0xFFu;
    }
    if (e_p == e_v) {
      int diff = (int)(acc[s] & 0x7Fu) - (int)(seen & 0x7Fu);
      diff = diff < 0 ? -diff : diff;
      atomicAdd(&hist[diff], 1u);
      diff_sum += (uint32_t)diff;
    } else {
      ++err_e;
    }
    if (io.gen_indices) {
      uint32_t hit = 0;
      for (int i = 0; i < k; ++i) hit |= gen[i] == idx[s];
      common += hit;
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    err_e += __shfl_xor_sync(0xFFFFFFFFu, err_e, off);
    diff_sum += __shfl_xor_sync(0xFFFFFFFFu, diff_sum, off);
    common += __shfl_xor_sync(0xFFFFFFFFu, common, off);
  }
  warp_barrier();
  // median from the histogram: sorted positions (n - 1) / 2 and n / 2; lane l owns bins 4l .. 4l + 3
  const uint32_t n = (uint32_t)k - err_e;
  uint32_t local[4], sum = 0;
#pragma unroll
  for (int b = 0; b < 4; ++b) {
    local[b] = hist[lane * 4 + b];
    sum += local[b];
  }
  uint32_t incl = sum;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const uint32_t other = __shfl_up_sync(0xFFFFFFFFu, incl, off);
    if (lane >= off) incl += other;
  }
  int lo_val = -1, hi_val = -1;
  if (n > 0) {
    const uint32_t lo_pos = (n - 1) / 2, hi_pos = n / 2;
    uint32_t below = incl - sum;
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const uint32_t upto = below + local[b];
      if (below <= lo_pos && lo_pos < upto) lo_val = lane * 4 + b;
      if (below <= hi_pos && hi_pos < upto) hi_val = lane * 4 + b;
      below = upto;
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    lo_val = max(lo_val, __shfl_xor_sync(0xFFFFFFFFu, lo_val, off));
    hi_val = max(hi_val, __shfl_xor_sync(0xFFFFFFFFu, hi_val, off));
  }
  if (lane == 0) {
    res.exp_mismatch = err_e;
    res.n_match = n;
    res.mant_diff_sum = diff_sum;
    if (io.gen_indices) res.topk_mismatch = k - (int)common;
    if (n > 0) {
      res.mant_mean = (double)diff_sum / (double)n;
      res.mant_median = ((double)lo_val + (double)hi_val) * 0.5;
    }
    res.accept = rejects(thr, res) ? 0 : 1;
    io.results[chunk] = res;
  }
}

// ---------------------------------------------------------------------------
// The 32-bit field: fp32 chunks that commit whole patterns work in Z_q,
// q = 2^32 - 5 (products are 64 bits wide and 2^32 = 5 folds them back).  A
// table of inverses is out of reach, so Algorithm 3 is arranged around ONE
// inversion per chunk.
// ---------------------------------------------------------------------------

// hi * 2^32 + lo reduced into [0, q): 2^32 == 5, so the value is 5 hi + lo; that sum has at most
// three bits above the 32nd, which fold the same way; a last wrap of 2^32 adds 5 to a small rest.
__device__ __forceinline__ uint32_t fold_q(uint32_t hi, uint32_t lo) {
  uint32_t s, above, r, wrapped;
  asm("{\n\t"
      ".reg .u32 l5, h5;\n\t"
      "mul.lo.u32 l5, %2, 5;\n\t"
      "mul.hi.u32 h5, %2, 5;\n\t"
      "add.cc.u32 %0, %3, l5;\n\t"
      "addc.u32 %1, h5, 0;\n\t"
      "}"
      : "=r"(s), "=r"(above)
      : "r"(hi), "r"(lo));
  asm("mad.lo.cc.u32 %0, %2, 5, %3;\n\t"
      "addc.u32 %1, 0, 0;"
      : "=r"(r), "=r"(wrapped)
      : "r"(above), "r"(s));
  r += 5u * wrapped;              // above <= 5: after a wrap the rest is below 25
  return min(r, r - kPrime32);    // r - q wraps to a huge value when r < q
}
__device__ __forceinline__ uint32_t mul_q(uint32_t a, uint32_t b) { return fold_q(__umulhi(a, b), a * b); }
__device__ __forceinline__ uint32_t mad_q(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t lo, hi;
  asm("mad.lo.cc.u32 %0, %2, %3, %4;\n\t"
      "madc.hi.u32 %1, %2, %3, 0;"
      : "=r"(lo), "=r"(hi)
      : "r"(a), "r"(b), "r"(c));
  return fold_q(hi, lo);
}
__device__ __forceinline__ uint32_t sub_q(uint32_t a, uint32_t b) { return a >= b ? a - b : a + (kPrime32 - b); }

// a^(q - 2): the inverse of a != 0 in Z_q (0 for a = 0).  The inverse is unique,
// so this agrees with the extended Euclid of Algorithm 4.
__device__ __forceinline__ uint32_t inv_q(uint32_t a) {
  uint32_t r = a;
#pragma unroll 1
  for (int bit = 30; bit >= 0; --bit) {
    r = mul_q(r, r);
    if (((kPrime32 - 2u) >> bit) & 1u) r = mul_q(r, a);
  }
  return r;
}

// Algorithm 3 (InterpolateModPolynomial) over Z_q for one chunk, by one warp.
// Point j lives in lane j % 32, slot j / 32.  The Newton coefficient of point i is
//   a_i = (y_i - P_{i-1}(x_i)) / N_i(x_i),   N_i(x) = prod_{l < i} (x - x_l),
// where P_{i-1} interpolates the first i points.  Every point j carries
// n_j = N_i(x_j) and, instead of t_j = y_j - P_{i-1}(x_j), the multiple
// T_j = s_i t_j with s_i = n_0 n_1 ... n_{i-1} (the pivots' n so far), because
//   t_j <- t_j - (t_i / n_i) n_j      becomes      T_j <- n_i T_j - T_i n_j
// without any division; then a_i = T_i / s_{i+1}.  The divisors are prefix
// products of the pivots' n_i, so ONE inversion of the last one and a suffix
// product per point give them all:  1 / s_{i+1} = (1 / s_k) n_{i+1} ... n_{k-1}.
// The Newton form is then multiplied out from the inside,
//   P <- P * (x - x_i) + a_i  for i = k-2 .. 0,
// with coefficient d in lane d % 32, slot d / 32: slots above the current degree hold zeros and
// are skipped, the shift by one degree is a rotation of every live slot by one lane.
// row_x / row_t / row_n: this warp's scratch rows in shared memory (x_i; T_i, later a_i; n_i).
template <int SLOTS>
__device__ __forceinline__ void interpolate_warp_q(int k, const uint32_t (&x)[SLOTS], const uint32_t (&y)[SLOTS],
                                                   uint16_t* row_x, uint32_t* row_t, uint32_t* row_n, uint16_t* proof) {
  const int lane = threadIdx.x & 31;
  constexpr uint32_t kFull = 0xFFFFFFFFu;
  uint32_t T[SLOTS], N[SLOTS];
#pragma unroll
  for (int s = 0; s < SLOTS; ++s) {
    T[s] = y[s];
    N[s] = 1u;
  }
  uint32_t scale = 1u;  // s_i, the same in every lane
#pragma unroll
  for (int b = 0; b < SLOTS; ++b) {
    const int steps = min(32, k - 32 * b);  // the last point only hands out its T and n
#pragma unroll 1
    for (int ii = 0; ii < steps; ++ii) {
      const uint32_t ni = __shfl_sync(kFull, N[b], ii);
      const uint32_t ti = __shfl_sync(kFull, T[b], ii);
      const uint32_t xi = __shfl_sync(kFull, x[b], ii);
      scale = mul_q(scale, ni);
      if (lane == 0) {
        row_x[32 * b + ii] = (uint16_t)xi;  // x = index mod m is below 2^16
        row_t[32 * b + ii] = ti;
        row_n[32 * b + ii] = ni;
      }
      const bool later = lane > ii;
      const uint32_t tb = sub_q(mul_q(ni, T[b]), mul_q(ti, N[b]));
      const uint32_t nb = mul_q(N[b], sub_q(x[b], xi));
      T[b] = later ? tb : T[b];
      N[b] = later ? nb : N[b];
#pragma unroll
      for (int s = b + 1; s < SLOTS; ++s) {
        T[s] = sub_q(mul_q(ni, T[s]), mul_q(ti, N[s]));
        N[s] = mul_q(N[s], sub_q(x[s], xi));
      }
    }
  }
  __syncwarp();
  // a_i = T_i / s_{i+1}: lane l owns i = l * SLOTS .. l * SLOTS + SLOTS - 1
  {
    const uint32_t inv_last = inv_q(scale);  // 1 / s_k
    uint32_t own[SLOTS], after[SLOTS];       // n_i, and the product of the n beyond i inside this lane
#pragma unroll
    for (int e = 0; e < SLOTS; ++e) {
      const int i = lane * SLOTS + e;
      own[e] = i < k ? row_n[i] : 1u;
    }
    after[SLOTS - 1] = 1u;
#pragma unroll
    for (int e = SLOTS - 2; e >= 0; --e) after[e] = mul_q(after[e + 1], own[e + 1]);
    uint32_t from_here = mul_q(after[0], own[0]);  // product over this lane's i, then over the lanes above too
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const uint32_t other = __shfl_down_sync(kFull, from_here, off);
      if (lane + off < 32) from_here = mul_q(from_here, other);
    }
    uint32_t beyond = __shfl_down_sync(kFull, from_here, 1);  // the lanes above this one
    if (lane == 31) beyond = 1u;
    const uint32_t base = mul_q(inv_last, beyond);
#pragma unroll
    for (int e = 0; e < SLOTS; ++e) {
      const int i = lane * SLOTS + e;
      if (i < k) row_t[i] = mul_q(row_t[i], mul_q(base, after[e]));
    }
  }
  __syncwarp();
  uint32_t co[SLOTS];
#pragma unroll
  for (int b = 0; b < SLOTS; ++b) co[b] = 0u;
  if (lane == 0) co[0] = row_t[k - 1];
  const int from = (lane + 31) & 31;
#pragma unroll
  for (int top = 0; top < SLOTS; ++top) {  // the slot that holds the leading coefficient
    const int d_first = max(32 * top, 1), d_last = min(32 * top + 31, k - 1);
#pragma unroll 1
    for (int D = d_first; D <= d_last; ++D) {
      const int i = k - 1 - D;
      const uint32_t neg_x = sub_q(0u, (uint32_t)row_x[i]);
      const uint32_t a_i = row_t[i];
      uint32_t below[SLOTS];  // coefficient d - 1, as seen from the owner of coefficient d
#pragma unroll
      for (int b = 0; b <= top; ++b) below[b] = __shfl_sync(kFull, co[b], from);
      // coefficient d takes  c[d-1] + (-x_i) c[d]
#pragma unroll
      for (int b = top; b >= 1; --b) co[b] = mad_q(co[b], neg_x, lane == 0 ? below[b - 1] : below[b]);
      co[0] = mad_q(co[0], neg_x, lane == 0 ? a_i : below[0]);
    }
  }
  // proof bytes 2 + 4d .. 5 + 4d: coefficient of degree d, little-endian (the proof is 2-byte aligned)
#pragma unroll
  for (int b = 0; b < SLOTS; ++b) {
    const int d = b * 32 + lane;
    if (d < k) {
      proof[1 + 2 * d] = (uint16_t)(co[b] & 0xFFFFu);
      proof[2 + 2 * d] = (uint16_t)(co[b] >> 16);
    }
  }
}

constexpr int kInterpQWarps = 8;  // 32-bit field interpolation: warps (chunks) per block

// InterpolateModPolynomial() and encode() of Algorithm 1 over Z_q for every
// chunk the select (or merge) kernel finished, one warp per chunk.
template <int SLOTS>
__device__ __forceinline__ void interpolate_chunk_q(const Selection& sel, int k, long long chunk, uint32_t* rows,
                                                    uint16_t* row_x) {
  const int lane = threadIdx.x & 31;
  uint16_t* proof = reinterpret_cast<uint16_t*>(sel.proofs + chunk * (2 + 4 * (size_t)k));
  uint32_t m = proof[0];
  if (m == 0) m = 65536u;
  uint32_t x[SLOTS], y[SLOTS];
#pragma unroll
  for (int s = 0; s < SLOTS; ++s) {
    const int j = s * 32 + lane;
    x[s] = 0;
    y[s] = 0;
    if (j < k) {
      x[s] = sel.idx[chunk * k + j] % m;  // i_m = i mod m (below 2^16 < q)
      const uint32_t pattern = sel.bits32[chunk * k + j];
      y[s] = pattern >= kPrime32 ? pattern - kPrime32 : pattern;  // "dd <- y mod M"
    }
  }
  interpolate_warp_q<SLOTS>(k, x, y, row_x, rows, rows + kMaxK, proof);
}

__global__ void __launch_bounds__(kInterpQWarps * 32)
toploc_interpolate_q_kernel(Selection sel, int k, long long num_chunks) {
  __shared__ uint32_t rows[kInterpQWarps][2 * kMaxK];
  __shared__ uint16_t rows_x[kInterpQWarps][kMaxK];
  const int warp = threadIdx.x >> 5;
  const long long chunk = (long long)blockIdx.x * kInterpQWarps + warp;
  if (chunk >= num_chunks) return;
  const uint8_t st = sel.status[chunk];
  if (st == TOPLOC_CHUNK_NO_INJECTIVE_MODULUS || st == TOPLOC_CHUNK_K_EXCEEDS_CHUNK) return;
  if (k <= 32) interpolate_chunk_q<1>(sel, k, chunk, rows[warp], rows_x[warp]);
  else if (k <= 64) interpolate_chunk_q<2>(sel, k, chunk, rows[warp], rows_x[warp]);
  else if (k <= 128) interpolate_chunk_q<4>(sel, k, chunk, rows[warp], rows_x[warp]);
  else if (k <= 256) interpolate_chunk_q<8>(sel, k, chunk, rows[warp], rows_x[warp]);
  else interpolate_chunk_q<kMaxK / 32>(sel, k, chunk, rows[warp], rows_x[warp]);
}

// Algorithm 2 after the selection, over Z_q, for one chunk whose selected
// indices and whole fp32 patterns are in registers: Horner evaluation
// (Algorithm 5), extractBits() (bit 31 sign, bits 30..23 exponent, bits 22..0
// mantissa), error accumulation, verdict.  The median of up to k 23-bit
// differences is found by rank counting (no histogram fits).
// PADDED: the proof is a 16-bit field proof (a bf16 generator's); the polynomial is evaluated
// over Z_p and the committed 16-bit pattern padded with 16 zero bits before the comparison
// (Section 5.6, fp32 validator of a bf16 model).
template <int SLOTS, bool PADDED, class SH>
__device__ __forceinline__ void evaluate_warp_q(SH& sh, int k, long long chunk, const uint32_t (&idx)[SLOTS],
                                                const uint32_t (&pattern)[SLOTS], const VerifyIo& io,
                                                toploc_chunk_result res) {
  const int lane = threadIdx.x;
  const uint16_t* proof =
      reinterpret_cast<const uint16_t*>(io.proofs + chunk * (2 + (PADDED ? 2 : 4) * (size_t)k));
  // the selection has left shared memory, so the ring is free: three rows of kMaxK words
  uint32_t* coef = reinterpret_cast<uint32_t*>(sh.ring);
  uint32_t* gen = coef + SH::kMaxK;
  uint32_t* diffs = gen + SH::kMaxK;
  constexpr uint32_t kNoMatch = 0xFFFFFFFFu;  // larger than any 23-bit difference
  const toploc_thresholds thr = thresholds_of(io, chunk);
  warp_barrier();
  for (int d = lane; d < k; d += 32)
    coef[d] = PADDED ? (uint32_t)proof[1 + d] : ((uint32_t)proof[1 + 2 * d] | ((uint32_t)proof[2 + 2 * d] << 16));
  if (io.gen_indices)
    for (int j = lane; j < k; j += 32) gen[j] = (uint32_t)io.gen_indices[chunk * k + j];
  warp_barrier();

  const uint32_t m = res.modulus;
  uint32_t x[SLOTS], acc[SLOTS];
#pragma unroll
  for (int s = 0; s < SLOTS; ++s) {
    x[s] = idx[s] % m;
    if (PADDED && x[s] >= kPrime) x[s] -= kPrime;
    acc[s] = coef[k - 1];  // Horner, highest degree first
  }
#pragma unroll 2
  for (int d = k - 2; d >= 0; --d) {
    const uint32_t cd = coef[d];
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) acc[s] = PADDED ? mad_mod(acc[s], x[s], cd) : mad_q(acc[s], x[s], cd);
  }
  if (PADDED) {
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) acc[s] <<= 16;  // the committed 16-bit pattern, 16 zero bits below it
  }
  uint32_t err_e = 0, diff_sum = 0, common = 0;
#pragma unroll
  for (int s = 0; s < SLOTS; ++s) {
    const int j = s * 32 + lane;
    if (j >= k) continue;
    const uint32_t seen = pattern[s];
    uint32_t e_p = acc[s] >> 23, e_v = seen >> 23;  // sign + 8 exponent bits
    if (!thr.sign_in_exponent) {
      e_p &= 0xFFu;
      e_v &= 0xFFu;
    }
    uint32_t diff = kNoMatch;
    if (e_p == e_v) {
      const uint32_t m_p = acc[s] & 0x7FFFFFu, m_v = seen & 0x7FFFFFu;
      diff = m_p > m_v ? m_p - m_v : m_v - m_p;
      diff_sum += diff;  // at most 256 differences below 2^23
    } else {
      ++err_e;
    }
    diffs[j] = diff;
    if (io.gen_indices) {
      uint32_t hit = 0;
      for (int i = 0; i < k; ++i) hit |= gen[i] == idx[s];
      common += hit;
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    err_e += __shfl_xor_sync(0xFFFFFFFFu, err_e, off);
    diff_sum += __shfl_xor_sync(0xFFFFFFFFu, diff_sum, off);
    common += __shfl_xor_sync(0xFFFFFFFFu, common, off);
  }
  warp_barrier();
  // median: the differences at sorted positions (n - 1) / 2 and n / 2, a difference's position being
  // the number of differences that precede it (smaller, or equal and earlier)
  const uint32_t n = (uint32_t)k - err_e;
  int lo_val = -1, hi_val = -1;
  if (n > 0) {
    const uint32_t lo_pos = (n - 1) / 2, hi_pos = n / 2;
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) {
      const int j = s * 32 + lane;
      if (j >= k) continue;
      const uint32_t mine = diffs[j];
      if (mine == kNoMatch) continue;
      uint32_t before = 0;
      for (int i = 0; i < k; ++i) {
        const uint32_t other = diffs[i];
        before += (other < mine) || (other == mine && i < j);
      }
      if (before == lo_pos) lo_val = (int)mine;
      if (before == hi_pos) hi_val = (int)mine;
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    lo_val = max(lo_val, __shfl_xor_sync(0xFFFFFFFFu, lo_val, off));
    hi_val = max(hi_val, __shfl_xor_sync(0xFFFFFFFFu, hi_val, off));
  }
  if (lane == 0) {
    res.exp_mismatch = err_e;
    res.n_match = n;
    res.mant_diff_sum = diff_sum;
    if (io.gen_indices) res.topk_mismatch = k - (int)common;
    if (n > 0) {
      res.mant_mean = (double)diff_sum / (double)n;
      res.mant_median = ((double)lo_val + (double)hi_val) * 0.5;
    }
    res.accept = rejects(thr, res) ? 0 : 1;
    io.results[chunk] = res;
  }
}

template <int DT, int SLOTS, class SH>
__device__ __forceinline__ void verify_chunk(SH& sh, int k, bool wide, bool padded, long long chunk,
                                             const VerifyIo& io, const toploc_chunk_result& res) {
  const int lane = threadIdx.x;
  uint32_t idx[SLOTS], bits[SLOTS];
#pragma unroll
  for (int s = 0; s < SLOTS; ++s) {
    const int j = s * 32 + lane;
    idx[s] = 0;
    bits[s] = 0;
    if (j < k) {
      const unsigned long long cj = sh.cand[j];
      const uint32_t key = (uint32_t)(cj >> (kIdxBits + 1));
      const uint32_t sign = (uint32_t)cj & 1u;
      idx[s] = kIdxMask - ((uint32_t)(cj >> 1) & kIdxMask);
      bits[s] = (DT == 1 && wide) ? ((sign << 31) | key) : ((sign << 15) | (DT == 0 ? key : (key >> 16)));
    }
  }
  if (DT == 1 && wide && padded) evaluate_warp_q<SLOTS, true>(sh, k, chunk, idx, bits, io, res);
  else if (DT == 1 && wide) evaluate_warp_q<SLOTS, false>(sh, k, chunk, idx, bits, io, res);
  else evaluate_warp<SLOTS>(sh, k, chunk, idx, bits, io, res);
}

// decode() of Algorithm 2 for one chunk, by one warp: fills res with zeros and
// the decoded modulus.  A malformed proof (modulus outside [2^15 + 1, 2^16] or a
// coefficient >= p, >= q for 4-byte coefficients) is reported without looking at the activations: its result
// is written and false returned.
__device__ __forceinline__ bool decode_proof(const VerifyIo& io, long long chunk, int k, int coef_bytes,
                                             toploc_chunk_result* res) {
  const int lane = threadIdx.x;
  res->exp_mismatch = 0;
  res->n_match = 0;
  res->mant_diff_sum = 0;
  res->topk_mismatch = -1;
  res->mant_mean = 0.0;
  res->mant_median = 0.0;
  res->accept = 0;
  res->status = TOPLOC_CHUNK_OK;
  res->pad[0] = res->pad[1] = 0;
  const uint16_t* proof = reinterpret_cast<const uint16_t*>(io.proofs + chunk * (2 + (size_t)coef_bytes * k));
  uint32_t m = proof[0];
  if (m == 0) m = 65536u;
  res->modulus = m;
  uint32_t bad = (m < kModLow || m > kModHigh);
  if (coef_bytes == 2) {
    for (int d = lane; d < k; d += kThreads) bad |= proof[1 + d] >= kPrime;
  } else {
    for (int d = lane; d < k; d += kThreads)
      bad |= ((uint32_t)proof[1 + 2 * d] | ((uint32_t)proof[2 + 2 * d] << 16)) >= kPrime32;
  }
  if (__any_sync(0xFFFFFFFFu, bad != 0)) {
    res->status = TOPLOC_CHUNK_BAD_PROOF;
    if (lane == 0) io.results[chunk] = *res;
    return false;
  }
  return true;
}

// ---------------------------------------------------------------------------
// verify kernel: Algorithm 2 for one chunk per block (one warp): decode(),
// topk() while the chunk streams in, then Horner evaluation, comparison and
// verdict by the same warp.  Validation needs no scratch memory beyond the row
// table of a ragged batch.
// ---------------------------------------------------------------------------
template <int DT, int MODE, class SH>
__global__ void __launch_bounds__(kThreads, select_min_blocks<SH>()) toploc_verify_kernel(BatchParams bp, VerifyIo io) {
  __shared__ SH sh;
  const int tid = threadIdx.x;
  const long long chunk = blockIdx.x;
  const int k = bp.k;

  toploc_chunk_result res;
  if (!decode_proof(io, chunk, k, bp.coef_bytes, &res)) return;
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

  const bool padded = bp.padded != 0;
  const bool wide = bp.coef_bytes == 4 || padded;  // whole patterns are compared
  if constexpr (SH::kMaxK > 256) {
    verify_chunk<DT, SH::kMaxSlots>(sh, k, wide, padded, chunk, io, res);  // launched for k above 256 only
  } else {
    if (k <= 32) verify_chunk<DT, 1>(sh, k, wide, padded, chunk, io, res);
    else if (k <= 64) verify_chunk<DT, 2>(sh, k, wide, padded, chunk, io, res);
    else if (k <= 128) verify_chunk<DT, 4>(sh, k, wide, padded, chunk, io, res);
    else verify_chunk<DT, 8>(sh, k, wide, padded, chunk, io, res);
  }
}

// ---------------------------------------------------------------------------
// merge kernel: the top-k of a chunk from the top-k of its segments, one block
// per chunk (its first warp then runs the same tails as the select and verify
// kernels).  Every
// candidate becomes one 64-bit word whose unsigned order is the ranking order
// over the whole chunk: key << 33 | (2^32 - 1 - flat index) << 1 | sign.  The
// k-th largest word is found digit by digit (MSB-first radix select, eight
// 8-bit passes over the chunk's words in scratch memory); the words that reach
// it are the chunk's selection.  A chunk of one segment passes through.
// TAIL: 0 hand the selection out, 1 proof generation (also the modulus),
// 2 validation.
// ---------------------------------------------------------------------------
template <int DT, int TAIL, int SLOTS, class SH>
__device__ __forceinline__ void finish_merged(SH& sh, const BatchParams& bp, long long chunk,
                                              const Selection& sel, const VerifyIo& io,
                                              const toploc_chunk_result& res) {
  const int lane = threadIdx.x;
  const int k = bp.k;
  const bool padded = DT == 1 && TAIL == 2 && bp.padded != 0;
  const bool wide = DT == 1 && (bp.coef_bytes == 4 || padded);
  uint32_t idx[SH::kMaxK / kThreads], bits[SLOTS];
  uint32_t unrepresentable = 0;
#pragma unroll
  for (int e = 0; e < SH::kMaxK / kThreads; ++e) idx[e] = 0;
#pragma unroll
  for (int e = 0; e < SLOTS; ++e) {
    const int j = e * 32 + lane;
    bits[e] = 0;
    if (j < k) {
      const unsigned long long w = sh.cand[j];
      const uint32_t key = (uint32_t)(w >> 33);
      const uint32_t sign = (uint32_t)w & 1u;
      idx[e] = 0xFFFFFFFFu - (uint32_t)(w >> 1);
      bits[e] = wide ? ((sign << 31) | key) : ((sign << 15) | (DT == 0 ? key : (key >> 16)));
      unrepresentable |= bits[e] >= (wide ? kPrime32 : kPrime);
      if (TAIL != 2) {
        sel.idx[chunk * k + j] = idx[e];
        if (wide) sel.bits32[chunk * k + j] = bits[e];
        else sel.bits[chunk * k + j] = (uint16_t)bits[e];
        if (sel.indices) {
          int rank = 0;  // position = number of better candidates
          for (int i = 0; i < k; ++i) rank += sh.cand[i] > w;
          sel.indices[chunk * k + rank] = (int32_t)idx[e];
        }
      }
    }
  }
  if (TAIL == 0) {
    if (lane == 0) sel.status[chunk] = TOPLOC_CHUNK_OK;
  } else if (TAIL == 1) {
    uint16_t* proof = reinterpret_cast<uint16_t*>(sel.proofs + chunk * proof_stride(bp));
    const bool nonfinite = __any_sync(0xFFFFFFFFu, unrepresentable != 0);
    const uint32_t m = find_injective_modulus(sh, k, idx, wide);
    if (m == 0) {
      for (int i = lane; i < proof_words(bp); i += kThreads) proof[i] = 0;
      if (lane == 0) sel.status[chunk] = TOPLOC_CHUNK_NO_INJECTIVE_MODULUS;
      return;
    }
    if (lane == 0) {
      proof[0] = (uint16_t)(m & 0xFFFFu);  // 65536 is stored as 0
      sel.status[chunk] = nonfinite ? TOPLOC_CHUNK_NONFINITE_COMMITTED : TOPLOC_CHUNK_OK;
    }
  } else {
    uint32_t own[SLOTS];
#pragma unroll
    for (int e = 0; e < SLOTS; ++e) own[e] = idx[e];
    if (padded) evaluate_warp_q<SLOTS, true>(sh, k, chunk, own, bits, io, res);
    else if (wide) evaluate_warp_q<SLOTS, false>(sh, k, chunk, own, bits, io, res);
    else evaluate_warp<SLOTS>(sh, k, chunk, own, bits, io, res);
  }
}

constexpr int kMergeThreads = 256;  // merge kernel: the passes over a chunk's words use the whole block

template <int DT, int TAIL>
__global__ void __launch_bounds__(kMergeThreads)
toploc_merge_kernel(BatchParams bp, MergeParams mp, Selection sel, VerifyIo io) {
  __shared__ SelectSharedBig sh;  // (one block per chunk: the larger scratch costs nothing here)
  __shared__ int kept;     // words taken so far
  __shared__ int proceed;  // decode() found the proof well-formed
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const bool first_warp = tid < 32;  // the warp that goes on to the tail
  const long long chunk = blockIdx.x;
  const int k = bp.k;
  toploc_chunk_result res;
  if (TAIL == 2) {
    if (first_warp) {
      const bool ok = decode_proof(io, chunk, k, bp.coef_bytes, &res);
      if (lane == 0) proceed = ok;
    }
    __syncthreads();
    if (!proceed) return;
  }

  const ChunkSegments cs = mp.chunks[chunk];
  if (mp.seg_status[cs.first_seg] != TOPLOC_CHUNK_OK) {
    // fewer than k elements: such a chunk is one segment, which said so
    if (!first_warp) return;
    if (TAIL == 2) {
      res.status = TOPLOC_CHUNK_K_EXCEEDS_CHUNK;
      if (lane == 0) io.results[chunk] = res;
      return;
    }
    if (TAIL == 1) {
      uint16_t* proof = reinterpret_cast<uint16_t*>(sel.proofs + chunk * proof_stride(bp));
      for (int i = lane; i < proof_words(bp); i += kThreads) proof[i] = 0;
    }
    if (sel.indices)
      for (int i = lane; i < k; i += kThreads) sel.indices[chunk * k + i] = 0;
    if (lane == 0) sel.status[chunk] = TOPLOC_CHUNK_K_EXCEEDS_CHUNK;
    return;
  }

  const int n = cs.n_segs * k;
  unsigned long long* words = mp.words + (size_t)cs.first_seg * k;
  for (int c = tid; c < n; c += kMergeThreads) {
    const int seg = c / k;
    const size_t at = (size_t)(cs.first_seg + seg) * k + (size_t)(c - seg * k);
    const long long seg_row0 = mp.segs[cs.first_seg + seg].row0;
    const uint32_t local = mp.seg_idx[at];
    const uint32_t flat = (uint32_t)((seg_row0 - cs.row0) * bp.hidden) + local;
    uint32_t key, sign;
    if (DT == 0) {
      const uint32_t pattern = mp.seg_bits[at];
      key = pattern & 0x7FFFu;
      sign = pattern >> 15;
    } else {
      // the segment kept only part of the pattern: read the element again
      const long long row = seg_row0 + local / (uint32_t)bp.hidden;
      const uint32_t col = local % (uint32_t)bp.hidden;
      const uint32_t pattern = static_cast<const uint32_t*>(bp.act)[row * bp.row_stride + col];
      key = pattern & 0x7FFFFFFFu;
      sign = pattern >> 31;
    }
    words[c] = ((unsigned long long)key << 33) | ((unsigned long long)(0xFFFFFFFFu - flat) << 1) | sign;
  }
  if (tid == 0) kept = 0;
  __syncthreads();

  unsigned long long kth = 0;  // the k-th largest word; all of them if the chunk is one segment
  if (n > k) {
    unsigned long long prefix = 0;
    int want = k;
    // a bf16 key has 15 bits: the two leading digits of its words are zero
#pragma unroll 1
    for (int pass = (DT == 0 ? 2 : 0); pass < 8; ++pass) {
      const int shift = 56 - 8 * pass;
      for (int b = tid; b < 256; b += kMergeThreads) sh.top_hist[b] = 0;
      __syncthreads();
      for (int c = tid; c < n; c += kMergeThreads) {
        const unsigned long long w = words[c];
        if (pass == 0 || (w >> (shift + 8)) == prefix) atomicAdd(&sh.top_hist[(uint32_t)(w >> shift) & 255u], 1u);
      }
      __syncthreads();
      if (first_warp) find_from_top<8>(sh, sh.top_hist, want);
      __syncthreads();
      prefix = (prefix << 8) | sh.digit;
      want = sh.want;
    }
    kth = prefix;
  }
  for (int c = tid; c < n; c += kMergeThreads) {
    const unsigned long long w = words[c];
    if (w >= kth) sh.cand[atomicAdd(&kept, 1)] = w;  // words are distinct: exactly k are taken, in any order
  }
  __syncthreads();
  if (!first_warp) return;

  if (k <= 32) finish_merged<DT, TAIL, 1>(sh, bp, chunk, sel, io, res);
  else if (k <= 64) finish_merged<DT, TAIL, 2>(sh, bp, chunk, sel, io, res);
  else if (k <= 128) finish_merged<DT, TAIL, 4>(sh, bp, chunk, sel, io, res);
  else if (k <= 256) finish_merged<DT, TAIL, 8>(sh, bp, chunk, sel, io, res);
  else finish_merged<DT, TAIL, kMaxK / 32>(sh, bp, chunk, sel, io, res);
}

// ---------------------------------------------------------------------------
// Incremental proof generation (the provider's side during decoding, Section
// 5.5: a proof per 32 new tokens): the rows of a chunk arrive one token at a
// time, while they are still warm in L2, and each sequence keeps its running
// top-k between the steps.  Streaming a chunk in index order and keeping the
// best k so far (ties to the lower index) yields the chunk's top-k, so the
// result equals toploc_build_proofs over the assembled chunk.
// ---------------------------------------------------------------------------
// One new row per sequence: token t of the running chunk.  One warp per sequence.
template <int DT, int MODE>
__global__ void __launch_bounds__(kThreads)
toploc_stream_append_kernel(const char* rows, long long row_stride, int hidden, int k, int token,
                            unsigned char* state) {
  constexpr int VEC = ChunkSource<DT, MODE>::kVec;
  constexpr int kElem = DT == 0 ? 2 : 4;
  __shared__ SelectSharedBig sh;
  const long long seq = blockIdx.x;
  unsigned char* mine = state + seq * stream_state_stride(k);
  WarpState st = running_selection_open<DT>(sh, mine, k);
  // the row stands at flat indices token * hidden ..: a source whose vector token * (hidden / VEC) is the row's first
  ChunkSource<DT, MODE> src;
  src.base = rows + seq * row_stride * kElem - (long long)token * hidden * kElem;
  src.row_stride = hidden;
  src.hidden = hidden;
  src.vecs_per_row = hidden / VEC;
  const int per_row = hidden / VEC;
  st = running_selection_take<DT, MODE>(sh, st, src, token * per_row, (token + 1) * per_row, k);
  running_selection_close<DT>(sh, st, mine, k);
}

// The running selections become the chunks' selections: what the select kernel
// leaves behind, for the interpolation kernel to finish.
template <int DT>
__global__ void __launch_bounds__(kThreads) toploc_stream_finish_kernel(BatchParams bp, Selection sel,
                                                                        const unsigned char* state) {
  __shared__ SelectSharedBig sh;
  const int lane = threadIdx.x;
  const long long seq = blockIdx.x;
  const int k = bp.k;
  const StreamHeader* head = reinterpret_cast<const StreamHeader*>(state + seq * stream_state_stride(k));
  const unsigned long long* held = reinterpret_cast<const unsigned long long*>(head + 1);
  if ((int)head->count < k) {
    uint16_t* proof = reinterpret_cast<uint16_t*>(sel.proofs + seq * proof_stride(bp));
    for (int i = lane; i < proof_words(bp); i += kThreads) proof[i] = 0;
    if (sel.indices)
      for (int i = lane; i < k; i += kThreads) sel.indices[seq * k + i] = 0;
    if (lane == 0) sel.status[seq] = TOPLOC_CHUNK_K_EXCEEDS_CHUNK;
    return;
  }
  for (int e = lane; e < k; e += kThreads) sh.cand[e] = held[e];
  warp_barrier();
  publish_selection<DT>(sh, bp, seq, sel);
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
struct HostPlan {
  long long num_chunks;
  long long max_seq_rows;
  long long num_segs;  // segments over all chunks; equals num_chunks unless some chunk is long
  int chunks_per_seq;  // uniform only
  bool ragged;
  bool split;          // some chunk is selected in more than one segment
};

// A chunk of more than kLongChunkElems elements is selected in segments of whole
// rows (about kSegmentElems elements each, at most kMaxSegmentsPerChunk unless
// the 24-bit index field of a candidate forces more) whose winners are merged.
constexpr long long kLongChunkElems = 1ll << 19;
constexpr long long kSegmentElems = 1ll << 18;
constexpr long long kMaxSegmentsPerChunk = 64;
constexpr long long kMaxSegmentElems = 1ll << kIdxBits;

// Segments of a chunk of `rows` rows (1: the chunk is selected directly).
// Segment g covers rows [rows * g / n, rows * (g + 1) / n).
long long segments_of(long long rows, long long hidden) {
  const long long n = rows * hidden;
  if (n <= kLongChunkElems) return 1;
  long long segs = (n + kSegmentElems - 1) / kSegmentElems;
  if (segs > kMaxSegmentsPerChunk) segs = kMaxSegmentsPerChunk;
  const long long rows_fit = kMaxSegmentElems / hidden;  // rows whose indices fit the candidate's field
  const long long forced = (rows + rows_fit - 1) / rows_fit;
  if (segs < forced) segs = forced;
  if (segs > rows) segs = rows;
  return segs;
}

// Chunks and segments of a sequence of len rows: len / L full chunks and perhaps a shorter last one.
void count_sequence(const toploc_layout* lay, long long len, long long* chunks, long long* segs) {
  const long long full = len / lay->chunk_len, rest = len % lay->chunk_len;
  *chunks += full + (rest ? 1 : 0);
  if (full) *segs += full * segments_of(lay->chunk_len, lay->hidden);
  if (rest) *segs += segments_of(rest, lay->hidden);
}

int plan_layout(const toploc_layout* lay, HostPlan* plan) {
  if (lay == nullptr) return TOPLOC_ERR_INVALID_ARGUMENT;
  if (lay->dtype != TOPLOC_DTYPE_BF16 && lay->dtype != TOPLOC_DTYPE_FP32) return TOPLOC_ERR_UNSUPPORTED;
  if (lay->hidden <= 0 || lay->chunk_len <= 0 || lay->num_seqs <= 0) return TOPLOC_ERR_INVALID_ARGUMENT;
  if (lay->field != TOPLOC_FIELD_16 && lay->field != TOPLOC_FIELD_32 && lay->field != TOPLOC_FIELD_16_PADDED)
    return TOPLOC_ERR_INVALID_ARGUMENT;
  if (lay->field != TOPLOC_FIELD_16 && lay->dtype != TOPLOC_DTYPE_FP32) return TOPLOC_ERR_UNSUPPORTED;
  if (lay->k < 1) return TOPLOC_ERR_INVALID_ARGUMENT;
  if (lay->k > TOPLOC_MAX_K) return TOPLOC_ERR_UNSUPPORTED;
  if (lay->row_stride < lay->hidden) return TOPLOC_ERR_INVALID_ARGUMENT;
  if (lay->hidden > kMaxSegmentElems) return TOPLOC_ERR_UNSUPPORTED;  // a row must fit one segment
  plan->ragged = lay->seq_offsets != nullptr;
  plan->chunks_per_seq = 0;
  long long n = 0, longest = 0, segs = 0;
  // only chunks that exist count against the size limit
  auto largest_chunk_fits = [&](long long len) {
    const long long rows = len < lay->chunk_len ? len : lay->chunk_len;
    return rows * lay->hidden <= (long long)TOPLOC_MAX_CHUNK_ELEMS;
  };
  if (plan->ragged) {
    if (lay->seq_offsets[0] < 0) return TOPLOC_ERR_INVALID_ARGUMENT;
    for (int s = 0; s < lay->num_seqs; ++s) {
      long long len = lay->seq_offsets[s + 1] - lay->seq_offsets[s];
      if (len < 0) return TOPLOC_ERR_INVALID_ARGUMENT;
      if (!largest_chunk_fits(len)) return TOPLOC_ERR_UNSUPPORTED;
      count_sequence(lay, len, &n, &segs);
      if (len > longest) longest = len;
    }
  } else {
    if (lay->tokens_per_seq <= 0) return TOPLOC_ERR_INVALID_ARGUMENT;
    long long cps = (lay->tokens_per_seq + lay->chunk_len - 1) / lay->chunk_len;
    if (cps > 0x7FFFFFFFll) return TOPLOC_ERR_UNSUPPORTED;
    plan->chunks_per_seq = (int)cps;
    if (!largest_chunk_fits(lay->tokens_per_seq)) return TOPLOC_ERR_UNSUPPORTED;
    count_sequence(lay, lay->tokens_per_seq, &n, &segs);
    n *= lay->num_seqs;
    segs *= lay->num_seqs;
    longest = lay->tokens_per_seq;
  }
  if (n > 0x7FFFFFFFll || segs > 0x7FFFFFFFll) return TOPLOC_ERR_UNSUPPORTED;
  plan->num_chunks = n;
  plan->num_segs = segs;
  plan->split = segs != n;
  plan->max_seq_rows = longest;
  return TOPLOC_OK;
}

struct DeviceInfo {
  bool known;
  int major;
  int sms;
  bool interp_smem_set;
  void* builtin_scratch;  // device address of g_builtin_scratch on this device, once looked up
};

// Scratch for toploc_build_proofs_builtin_scratch: lives in the library's own
// device image, so every GPU that loads the library holds these bytes until
// the process exits.  In host code this name is only a handle; the address a
// kernel can use comes from cudaGetSymbolAddress (see builtin_scratch_address).
constexpr size_t kBuiltinScratchBytes = TOPLOC_BUILTIN_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_builtin_scratch[kBuiltinScratchBytes];

// table of inverses + the warps' rows (x_i and a_i as one 32-bit word per point)
size_t interp_smem_bytes(bool big) {
  const size_t row_words = big ? (size_t)kInterpWarpsBig * kMaxK : (size_t)kInterpWarps * kInterpChunks * kSmallMaxK;
  return (65536 + 2 * row_words) * sizeof(uint16_t);
}

// Per-device facts, looked up on a device's first call.  Host threads may call
// the library concurrently: the table is filled under a lock.
std::mutex g_device_table_lock;

int device_info(DeviceInfo** out) {
  static DeviceInfo table[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return TOPLOC_ERR_CUDA;
  if (dev < 0 || dev >= 64) return TOPLOC_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> guard(g_device_table_lock);
  DeviceInfo& d = table[dev];
  if (!d.known) {
    if (cudaDeviceGetAttribute(&d.major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
      return TOPLOC_ERR_CUDA;
    d.known = true;
  }
  if (d.major != 10) return TOPLOC_ERR_ARCH;
  if (!d.interp_smem_set) {
    if (cudaFuncSetAttribute(toploc_interpolate_kernel<kInterpWarps, kSmallMaxK>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)interp_smem_bytes(false)) != cudaSuccess ||
        cudaFuncSetAttribute(toploc_interpolate_kernel<kInterpWarpsBig, kMaxK>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)interp_smem_bytes(true)) != cudaSuccess)
      return TOPLOC_ERR_CUDA;
    d.interp_smem_set = true;
  }
  *out = &d;
  return TOPLOC_OK;
}

// Device address of the built-in scratch on the current device (looked up once per device).
int builtin_scratch_address(DeviceInfo* d, void** out) {
  std::lock_guard<std::mutex> guard(g_device_table_lock);
  if (d->builtin_scratch == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_builtin_scratch) != cudaSuccess || ptr == nullptr) return TOPLOC_ERR_CUDA;
    d->builtin_scratch = ptr;
  }
  *out = d->builtin_scratch;
  return TOPLOC_OK;
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

size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Pointers the kernels read or write with loads of their element size: an address that is not
// a multiple of it would fault on the device, so it is refused on the host.
bool misaligned(const void* p, size_t a) { return reinterpret_cast<uintptr_t>(p) % a != 0; }
size_t element_bytes(const toploc_layout* lay) { return lay->dtype == TOPLOC_DTYPE_BF16 ? 2 : 4; }

size_t coef_bytes_of(const toploc_layout* lay) { return lay->field == TOPLOC_FIELD_32 ? 4 : 2; }
size_t proof_bytes_of(const toploc_layout* lay) { return 2 + coef_bytes_of(lay) * (size_t)lay->k; }

// Scratch of one call: ragged row table, then the selection; with long chunks
// (segs != chunks) the row table describes segments and is followed by the
// chunk table, the segments' selections and the merge's words.
struct WorkspacePlan {
  size_t spans_off, chunk_table_off, seg_idx_off, seg_bits_off, seg_status_off, words_off;
  size_t idx_off, bits_off, status_off, total;
};

// pattern_bytes: 2, or 4 for fp32 chunks committed over the 32-bit field.
WorkspacePlan plan_workspace(bool ragged, long long chunks, int k, long long segs, size_t pattern_bytes) {
  WorkspacePlan w;
  const bool split = segs != chunks;
  size_t off = 0;
  w.spans_off = off;
  off += (ragged || split) ? round_up((size_t)segs * sizeof(ChunkSpan), 256) : 0;
  w.chunk_table_off = off;
  off += split ? round_up((size_t)chunks * sizeof(ChunkSegments), 256) : 0;
  w.seg_idx_off = off;
  off += split ? round_up((size_t)segs * k * sizeof(uint32_t), 256) : 0;
  w.seg_bits_off = off;
  off += split ? round_up((size_t)segs * k * pattern_bytes, 256) : 0;
  w.seg_status_off = off;
  off += split ? round_up((size_t)segs, 256) : 0;
  w.words_off = off;
  off += split ? round_up((size_t)segs * k * sizeof(unsigned long long), 256) : 0;
  w.idx_off = off;
  off += round_up((size_t)chunks * k * sizeof(uint32_t), 256);
  w.bits_off = off;
  off += round_up((size_t)chunks * k * pattern_bytes, 256);
  w.status_off = off;
  off += round_up((size_t)chunks, 256);
  w.total = off;
  return w;
}

long long seq_begin(const toploc_layout* lay, int s) {
  return lay->seq_offsets ? lay->seq_offsets[s] : (long long)s * lay->tokens_per_seq;
}

// Fills the device row table (one span per segment; a chunk that is not long
// is its own segment) and, for a batch with long chunks, the chunk table.
int upload_spans(const toploc_layout* lay, const HostPlan& plan, void* d_spans, void* d_chunk_table,
                 cudaStream_t stream) {
  const size_t span_bytes = (size_t)plan.num_segs * sizeof(ChunkSpan);
  const size_t table_bytes = plan.split ? (size_t)plan.num_chunks * sizeof(ChunkSegments) : 0;
  ChunkSpan* spans = static_cast<ChunkSpan*>(malloc(span_bytes));
  ChunkSegments* table = plan.split ? static_cast<ChunkSegments*>(malloc(table_bytes)) : nullptr;
  if (spans == nullptr || (plan.split && table == nullptr)) {
    free(spans);
    free(table);
    return TOPLOC_ERR_HOST_MEMORY;
  }
  long long c = 0, g = 0;
  for (int s = 0; s < lay->num_seqs; ++s) {
    const long long end = seq_begin(lay, s + 1);
    for (long long r = seq_begin(lay, s); r < end; r += lay->chunk_len) {
      const long long left = end - r;
      const long long rows = left < lay->chunk_len ? left : lay->chunk_len;
      const long long n_segs = segments_of(rows, lay->hidden);
      if (table) {
        table[c].row0 = r;
        table[c].first_seg = (int)g;
        table[c].n_segs = (int)n_segs;
      }
      for (long long i = 0; i < n_segs; ++i) {
        const long long a = rows * i / n_segs, b = rows * (i + 1) / n_segs;
        spans[g].row0 = r + a;
        spans[g].rows = (int)(b - a);
        spans[g].pad = 0;
        ++g;
      }
      ++c;
    }
  }
  // pageable sources: the runtime has staged the bytes by the time these return
  cudaError_t err = cudaMemcpyAsync(d_spans, spans, span_bytes, cudaMemcpyHostToDevice, stream);
  if (err == cudaSuccess && table)
    err = cudaMemcpyAsync(d_chunk_table, table, table_bytes, cudaMemcpyHostToDevice, stream);
  free(spans);
  free(table);
  return err == cudaSuccess ? TOPLOC_OK : TOPLOC_ERR_CUDA;
}

// k above 256 takes the kernels built around the larger per-warp scratch.
template <int DT, class SH>
void launch_select_sized(int mode, unsigned grid, cudaStream_t stream, const BatchParams& bp, const Selection& sel) {
  if (mode == 0) toploc_select_kernel<DT, 0, SH><<<grid, kThreads, 0, stream>>>(bp, sel);
  else if (mode == 1) toploc_select_kernel<DT, 1, SH><<<grid, kThreads, 0, stream>>>(bp, sel);
  else toploc_select_kernel<DT, 2, SH><<<grid, kThreads, 0, stream>>>(bp, sel);
}

template <int DT>
void launch_select(int mode, unsigned grid, cudaStream_t stream, const BatchParams& bp, const Selection& sel) {
  if (bp.k > kSmallMaxK) launch_select_sized<DT, SelectSharedBig>(mode, grid, stream, bp, sel);
  else launch_select_sized<DT, SelectShared>(mode, grid, stream, bp, sel);
}

template <int DT, class SH>
void launch_verify_sized(int mode, unsigned grid, cudaStream_t stream, const BatchParams& bp, const VerifyIo& io) {
  if (mode == 0) toploc_verify_kernel<DT, 0, SH><<<grid, kThreads, 0, stream>>>(bp, io);
  else if (mode == 1) toploc_verify_kernel<DT, 1, SH><<<grid, kThreads, 0, stream>>>(bp, io);
  else toploc_verify_kernel<DT, 2, SH><<<grid, kThreads, 0, stream>>>(bp, io);
}

template <int DT>
void launch_verify(int mode, unsigned grid, cudaStream_t stream, const BatchParams& bp, const VerifyIo& io) {
  if (bp.k > kSmallMaxK) launch_verify_sized<DT, SelectSharedBig>(mode, grid, stream, bp, io);
  else launch_verify_sized<DT, SelectShared>(mode, grid, stream, bp, io);
}

template <int DT>
void launch_merge(int tail, unsigned grid, cudaStream_t stream, const BatchParams& bp, const MergeParams& mp,
                  const Selection& sel, const VerifyIo& io) {
  if (tail == 0) toploc_merge_kernel<DT, 0><<<grid, kMergeThreads, 0, stream>>>(bp, mp, sel, io);
  else if (tail == 1) toploc_merge_kernel<DT, 1><<<grid, kMergeThreads, 0, stream>>>(bp, mp, sel, io);
  else toploc_merge_kernel<DT, 2><<<grid, kMergeThreads, 0, stream>>>(bp, mp, sel, io);
}

// A batch as the kernels see it.
struct PreparedBatch {
  BatchParams bp;       // chunks; in a batch with long chunks: segments (one warp each)
  MergeParams mp;       // batches with long chunks only
  Selection segs;       // where the segment selections go (batches with long chunks only)
  WorkspacePlan wp;
  char* ws;
  unsigned grid;        // blocks of the select / verify kernel
};

// Checks the scratch and describes the batch to the kernels; the row table of a
// ragged batch or of one with long chunks is uploaded.
int prepare_batch(const void* d_act, const toploc_layout* lay, void* d_workspace, size_t workspace_bytes,
                  cudaStream_t stream, const HostPlan* plan, DeviceInfo** dev, PreparedBatch* pb) {
  int rc = device_info(dev);
  if (rc != TOPLOC_OK) return rc;
  const WorkspacePlan wp = plan_workspace(plan->ragged, plan->num_chunks, lay->k, plan->num_segs, coef_bytes_of(lay));
  if (d_workspace == nullptr || workspace_bytes < wp.total) return TOPLOC_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(d_workspace) % 16 != 0) return TOPLOC_ERR_INVALID_ARGUMENT;
  char* ws = static_cast<char*>(d_workspace);
  pb->wp = wp;
  pb->ws = ws;
  pb->grid = (unsigned)plan->num_segs;
  BatchParams* bp = &pb->bp;
  bp->act = d_act;
  bp->row_stride = lay->row_stride;
  bp->tokens_per_seq = lay->tokens_per_seq;
  bp->spans = nullptr;
  bp->hidden = lay->hidden;
  bp->chunk_len = lay->chunk_len;
  bp->k = lay->k;
  bp->chunks_per_seq = plan->chunks_per_seq;
  bp->coef_bytes = (int)coef_bytes_of(lay);
  bp->padded = lay->field == TOPLOC_FIELD_16_PADDED;
  if (plan->ragged || plan->split) {
    if ((rc = upload_spans(lay, *plan, ws + wp.spans_off, ws + wp.chunk_table_off, stream)) != TOPLOC_OK) return rc;
    bp->spans = reinterpret_cast<const ChunkSpan*>(ws + wp.spans_off);
  }
  if (plan->split) {
    pb->segs.idx = reinterpret_cast<uint32_t*>(ws + wp.seg_idx_off);
    pb->segs.bits = reinterpret_cast<uint16_t*>(ws + wp.seg_bits_off);
    pb->segs.bits32 = reinterpret_cast<uint32_t*>(ws + wp.seg_bits_off);
    pb->segs.status = reinterpret_cast<uint8_t*>(ws + wp.seg_status_off);
    pb->segs.proofs = nullptr;
    pb->segs.indices = nullptr;
    pb->mp.chunks = reinterpret_cast<const ChunkSegments*>(ws + wp.chunk_table_off);
    pb->mp.segs = bp->spans;
    pb->mp.seg_idx = pb->segs.idx;
    pb->mp.seg_bits = pb->segs.bits;
    pb->mp.seg_status = pb->segs.status;
    pb->mp.words = reinterpret_cast<unsigned long long*>(ws + wp.words_off);
  }
  return TOPLOC_OK;
}

// Front half of proof generation and of toploc_select_topk: scratch carving and
// the select kernel (for a batch with long chunks: per segment, then the merge).
int run_select(const void* d_act, const toploc_layout* lay, void* d_workspace, size_t workspace_bytes,
               cudaStream_t stream, uint8_t* d_status_or_null, uint8_t* d_proofs_or_null,
               int32_t* d_indices_opt, HostPlan* plan, Selection* sel, DeviceInfo** dev,
               uint32_t* d_sel_idx_or_null = nullptr, uint16_t* d_sel_bits_or_null = nullptr) {
  PreparedBatch pb;
  int rc = prepare_batch(d_act, lay, d_workspace, workspace_bytes, stream, plan, dev, &pb);
  if (rc != TOPLOC_OK) return rc;
  sel->idx = d_sel_idx_or_null ? d_sel_idx_or_null : reinterpret_cast<uint32_t*>(pb.ws + pb.wp.idx_off);
  sel->bits = d_sel_bits_or_null ? d_sel_bits_or_null : reinterpret_cast<uint16_t*>(pb.ws + pb.wp.bits_off);
  sel->bits32 = reinterpret_cast<uint32_t*>(pb.ws + pb.wp.bits_off);  // written instead of bits by the 32-bit field
  sel->status = d_status_or_null ? d_status_or_null : reinterpret_cast<uint8_t*>(pb.ws + pb.wp.status_off);
  sel->proofs = d_proofs_or_null;
  sel->indices = d_indices_opt;
  const int mode = pick_mode(d_act, lay);
  const bool bf16 = lay->dtype == TOPLOC_DTYPE_BF16;
  if (!plan->split) {
    if (bf16) launch_select<0>(mode, pb.grid, stream, pb.bp, *sel);
    else launch_select<1>(mode, pb.grid, stream, pb.bp, *sel);
  } else {
    if (bf16) launch_select<0>(mode, pb.grid, stream, pb.bp, pb.segs);
    else launch_select<1>(mode, pb.grid, stream, pb.bp, pb.segs);
    const VerifyIo none = {};
    const int tail = d_proofs_or_null ? 1 : 0;
    if (bf16) launch_merge<0>(tail, (unsigned)plan->num_chunks, stream, pb.bp, pb.mp, *sel, none);
    else launch_merge<1>(tail, (unsigned)plan->num_chunks, stream, pb.bp, pb.mp, *sel, none);
  }
  return cudaGetLastError() == cudaSuccess ? TOPLOC_OK : TOPLOC_ERR_CUDA;
}

// Carves the staging buffer of the *_host entry points for a group of
// sequences: activations, per-chunk outputs, proofs, scratch.
struct StagingPlan {
  size_t act_off, small_off, proofs_off, work_off, work_bytes, total;
};

StagingPlan carve_staging(const toploc_layout* lay, long long rows, long long chunks, long long segs) {
  const size_t esz = lay->dtype == TOPLOC_DTYPE_BF16 ? 2 : 4;
  StagingPlan sp;
  sp.act_off = 0;
  size_t off = round_up((size_t)rows * (size_t)lay->row_stride * esz, 256);
  sp.small_off = off;
  off += round_up((size_t)chunks * sizeof(toploc_chunk_result), 256);
  sp.proofs_off = off;
  off += round_up((size_t)chunks * proof_bytes_of(lay), 256);
  sp.work_off = off;
  sp.work_bytes = plan_workspace(true, chunks, lay->k, segs, coef_bytes_of(lay)).total;
  off += sp.work_bytes;
  sp.total = off;
  return sp;
}

// Chunks and segments of sequences s0 .. s1 - 1.
void count_between(const toploc_layout* lay, int s0, int s1, long long* chunks, long long* segs) {
  *chunks = 0;
  *segs = 0;
  for (int s = s0; s < s1; ++s) count_sequence(lay, seq_begin(lay, s + 1) - seq_begin(lay, s), chunks, segs);
}

StagingPlan carve_staging_for(const toploc_layout* lay, int s0, int s1) {
  long long chunks, segs;
  count_between(lay, s0, s1, &chunks, &segs);
  return carve_staging(lay, seq_begin(lay, s1) - seq_begin(lay, s0), chunks, segs);
}

// What the incremental entry points accept: one chunk per sequence, short enough
// for the 24-bit index field of a candidate.
int plan_stream(const toploc_layout* lay) {
  if (lay == nullptr) return TOPLOC_ERR_INVALID_ARGUMENT;
  if (lay->dtype != TOPLOC_DTYPE_BF16 && lay->dtype != TOPLOC_DTYPE_FP32) return TOPLOC_ERR_UNSUPPORTED;
  if (lay->hidden <= 0 || lay->chunk_len <= 0 || lay->num_seqs <= 0 || lay->k < 1 || lay->row_stride < lay->hidden)
    return TOPLOC_ERR_INVALID_ARGUMENT;
  if (lay->field != TOPLOC_FIELD_16 && lay->field != TOPLOC_FIELD_32) return TOPLOC_ERR_INVALID_ARGUMENT;
  if (lay->field == TOPLOC_FIELD_32 && lay->dtype != TOPLOC_DTYPE_FP32) return TOPLOC_ERR_UNSUPPORTED;
  if (lay->k > TOPLOC_MAX_K) return TOPLOC_ERR_UNSUPPORTED;
  if ((long long)lay->hidden * lay->chunk_len > kMaxSegmentElems) return TOPLOC_ERR_UNSUPPORTED;
  return TOPLOC_OK;
}

template <int DT>
void launch_stream_append(int mode, const toploc_layout* lay, const void* d_rows, int token, void* d_state,
                                 cudaStream_t stream) {
  const char* rows = static_cast<const char*>(d_rows);
  unsigned char* state = static_cast<unsigned char*>(d_state);
  const unsigned grid = (unsigned)lay->num_seqs;
  if (mode == 0)
    toploc_stream_append_kernel<DT, 0><<<grid, kThreads, 0, stream>>>(rows, lay->row_stride, lay->hidden, lay->k,
                                                                      token, state);
  else
    toploc_stream_append_kernel<DT, 2><<<grid, kThreads, 0, stream>>>(rows, lay->row_stride, lay->hidden, lay->k,
                                                                      token, state);
}

// Algorithm 3 and encode() for the chunks whose selection and modulus are in place.
void launch_interpolation(const toploc_layout* lay, const DeviceInfo* dev, const Selection& sel, long long num_chunks,
                          cudaStream_t stream) {
  if (lay->field == TOPLOC_FIELD_32) {
    const long long q_blocks = (num_chunks + kInterpQWarps - 1) / kInterpQWarps;
    toploc_interpolate_q_kernel<<<(unsigned)q_blocks, kInterpQWarps * 32, 0, stream>>>(sel, lay->k, num_chunks);
    return;
  }
  // one block per SM; a small batch gets a block for every four of its groups (each block first
  // builds its table of inverses, so not one per group)
  const bool big = lay->k > kSmallMaxK;
  const long long groups = big ? num_chunks : (num_chunks + kInterpChunks - 1) / kInterpChunks;
  long long blocks = (groups + 3) / 4;
  if (blocks > dev->sms) blocks = dev->sms;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)blocks);
  cfg.blockDim = dim3((big ? kInterpWarpsBig : kInterpWarps) * 32);
  cfg.dynamicSmemBytes = interp_smem_bytes(big);
  cfg.stream = stream;
  cudaLaunchAttribute early[1];
  early[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // see wait_for_previous_grid()
  early[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = early;
  cfg.numAttrs = 1;
  if (big) cudaLaunchKernelEx(&cfg, toploc_interpolate_kernel<kInterpWarpsBig, kMaxK>, sel, lay->k, num_chunks);
  else cudaLaunchKernelEx(&cfg, toploc_interpolate_kernel<kInterpWarps, kSmallMaxK>, sel, lay->k, num_chunks);
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

size_t toploc_layout_proof_bytes(const toploc_layout* lay) {
  HostPlan plan;
  return plan_layout(lay, &plan) == TOPLOC_OK ? proof_bytes_of(lay) : 0;
}

size_t toploc_workspace_bytes(const toploc_layout* lay) {
  HostPlan plan;
  if (plan_layout(lay, &plan) != TOPLOC_OK) return 0;
  return plan_workspace(plan.ragged, plan.num_chunks, lay->k, plan.num_segs, coef_bytes_of(lay)).total;
}

size_t toploc_staging_bytes(const toploc_layout* lay) {
  HostPlan plan;
  if (plan_layout(lay, &plan) != TOPLOC_OK) return 0;
  long long chunks = 0, segs = 0;
  count_sequence(lay, plan.max_seq_rows, &chunks, &segs);
  return carve_staging(lay, plan.max_seq_rows, chunks, segs).total;
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
    case TOPLOC_ERR_HOST_MEMORY: return "out of host memory";
    case TOPLOC_ERR_BUILTIN_SCRATCH:
      return "batch needs more scratch than the library's built-in buffer holds (TOPLOC_BUILTIN_SCRATCH_BYTES)";
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
  if (misaligned(d_proofs, 2) || misaligned(d_act, element_bytes(lay)) || misaligned(d_indices_opt, 4))
    return TOPLOC_ERR_INVALID_ARGUMENT;
  if (lay->field == TOPLOC_FIELD_16_PADDED) return TOPLOC_ERR_UNSUPPORTED;  // a way to validate, not to commit
  if (plan.num_chunks == 0) return TOPLOC_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  Selection sel;
  DeviceInfo* dev = nullptr;
  rc = run_select(d_act, lay, d_workspace, workspace_bytes, stream, d_status, d_proofs, d_indices_opt, &plan,
                  &sel, &dev);
  if (rc != TOPLOC_OK) return rc;
  launch_interpolation(lay, dev, sel, plan.num_chunks, stream);
  return cudaGetLastError() == cudaSuccess ? TOPLOC_OK : TOPLOC_ERR_CUDA;
}

// Validation with the thresholds of the call (thr, host memory) or one entry per chunk
// (d_thr_each, device memory); exactly one of the two is given.
static int verify_proofs_with(const void* d_act, const toploc_layout* lay, const uint8_t* d_proofs,
                              const toploc_thresholds* thr, const toploc_thresholds* d_thr_each,
                              toploc_chunk_result* d_results, const int32_t* d_gen_indices_opt,
                              void* d_workspace, size_t workspace_bytes, void* cuda_stream) {
  HostPlan plan;
  int rc = plan_layout(lay, &plan);
  if (rc != TOPLOC_OK) return rc;
  if (d_act == nullptr || d_proofs == nullptr || (thr == nullptr && d_thr_each == nullptr) || d_results == nullptr)
    return TOPLOC_ERR_INVALID_ARGUMENT;
  if (misaligned(d_proofs, 2) || misaligned(d_results, 8) || misaligned(d_act, element_bytes(lay)) ||
      misaligned(d_gen_indices_opt, 4) || misaligned(d_thr_each, 8))
    return TOPLOC_ERR_INVALID_ARGUMENT;
  if (thr != nullptr && thr->t_exp < 0) return TOPLOC_ERR_INVALID_ARGUMENT;
  if (plan.num_chunks == 0) return TOPLOC_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  DeviceInfo* dev = nullptr;
  PreparedBatch pb;
  rc = prepare_batch(d_act, lay, d_workspace, workspace_bytes, stream, &plan, &dev, &pb);
  if (rc != TOPLOC_OK) return rc;
  VerifyIo io;
  io.proofs = d_proofs;
  io.results = d_results;
  io.gen_indices = d_gen_indices_opt;
  io.thr = thr ? *thr : toploc_thresholds{};
  io.thr_each = d_thr_each;
  const int mode = pick_mode(d_act, lay);
  const bool bf16 = lay->dtype == TOPLOC_DTYPE_BF16;
  if (!plan.split) {
    if (bf16) launch_verify<0>(mode, pb.grid, stream, pb.bp, io);
    else launch_verify<1>(mode, pb.grid, stream, pb.bp, io);
  } else {
    // long chunks: select per segment, then merge and validate per chunk
    if (bf16) launch_select<0>(mode, pb.grid, stream, pb.bp, pb.segs);
    else launch_select<1>(mode, pb.grid, stream, pb.bp, pb.segs);
    const Selection none = {};
    if (bf16) launch_merge<0>(2, (unsigned)plan.num_chunks, stream, pb.bp, pb.mp, none, io);
    else launch_merge<1>(2, (unsigned)plan.num_chunks, stream, pb.bp, pb.mp, none, io);
  }
  return cudaGetLastError() == cudaSuccess ? TOPLOC_OK : TOPLOC_ERR_CUDA;
}

int toploc_verify_proofs(const void* d_act, const toploc_layout* lay, const uint8_t* d_proofs,
                         const toploc_thresholds* thr, toploc_chunk_result* d_results,
                         const int32_t* d_gen_indices_opt, void* d_workspace, size_t workspace_bytes,
                         void* cuda_stream) {
  if (thr == nullptr) return TOPLOC_ERR_INVALID_ARGUMENT;
  return verify_proofs_with(d_act, lay, d_proofs, thr, nullptr, d_results, d_gen_indices_opt, d_workspace,
                            workspace_bytes, cuda_stream);
}

int toploc_verify_proofs_per_chunk_thresholds(const void* d_act, const toploc_layout* lay, const uint8_t* d_proofs,
                                              const toploc_thresholds* d_thr_per_chunk,
                                              toploc_chunk_result* d_results, const int32_t* d_gen_indices_opt,
                                              void* d_workspace, size_t workspace_bytes, void* cuda_stream) {
  if (d_thr_per_chunk == nullptr) return TOPLOC_ERR_INVALID_ARGUMENT;
  return verify_proofs_with(d_act, lay, d_proofs, nullptr, d_thr_per_chunk, d_results, d_gen_indices_opt,
                            d_workspace, workspace_bytes, cuda_stream);
}

int toploc_default_thresholds(int32_t k, int32_t field, toploc_thresholds* thr) {
  if (thr == nullptr || k < 1) return TOPLOC_ERR_INVALID_ARGUMENT;
  if (field != TOPLOC_FIELD_16 && field != TOPLOC_FIELD_32 && field != TOPLOC_FIELD_16_PADDED)
    return TOPLOC_ERR_INVALID_ARGUMENT;
  // Section 5.2 states 38 / 10 / 8 (bf16) and 8 / 256 / 128 (fp32) at k = 128.  The exponent
  // threshold counts points and scales with k; mean and median are per-point statistics.
  const bool fp32_fields = field != TOPLOC_FIELD_16;
  thr->t_exp = (int32_t)(((long long)(fp32_fields ? 8 : 38) * k) / 128);
  thr->sign_in_exponent = 1;
  thr->t_mean = fp32_fields ? 256.0 : 10.0;
  thr->t_median = fp32_fields ? 128.0 : 8.0;
  return TOPLOC_OK;
}

int toploc_select_topk(const void* d_act, const toploc_layout* lay, uint32_t* d_sel_indices,
                       uint16_t* d_sel_patterns, uint8_t* d_status, int32_t* d_ranked_indices_opt,
                       void* d_workspace, size_t workspace_bytes, void* cuda_stream) {
  HostPlan plan;
  int rc = plan_layout(lay, &plan);
  if (rc != TOPLOC_OK) return rc;
  if (d_act == nullptr || d_sel_indices == nullptr || d_sel_patterns == nullptr || d_status == nullptr)
    return TOPLOC_ERR_INVALID_ARGUMENT;
  if (misaligned(d_sel_indices, 4) || misaligned(d_sel_patterns, 2) || misaligned(d_act, element_bytes(lay)) ||
      misaligned(d_ranked_indices_opt, 4))
    return TOPLOC_ERR_INVALID_ARGUMENT;
  if (lay->field != TOPLOC_FIELD_16) return TOPLOC_ERR_UNSUPPORTED;  // this entry point hands out 16-bit patterns
  if (plan.num_chunks == 0) return TOPLOC_OK;
  Selection sel;
  DeviceInfo* dev = nullptr;
  return run_select(d_act, lay, d_workspace, workspace_bytes, static_cast<cudaStream_t>(cuda_stream), d_status,
                    nullptr, d_ranked_indices_opt, &plan, &sel, &dev, d_sel_indices, d_sel_patterns);
}

int toploc_build_proofs_builtin_scratch(const void* d_act, const toploc_layout* lay, uint8_t* d_proofs,
                                        uint8_t* d_status, int32_t* d_indices_opt, void* cuda_stream) {
  HostPlan plan;
  int rc = plan_layout(lay, &plan);
  if (rc != TOPLOC_OK) return rc;
  if (plan.ragged || plan.split) return TOPLOC_ERR_UNSUPPORTED;  // the row table would have to be built on the heap
  if (plan_workspace(false, plan.num_chunks, lay->k, plan.num_segs, coef_bytes_of(lay)).total > kBuiltinScratchBytes)
    return TOPLOC_ERR_BUILTIN_SCRATCH;
  DeviceInfo* dev = nullptr;
  if ((rc = device_info(&dev)) != TOPLOC_OK) return rc;
  void* scratch = nullptr;
  if ((rc = builtin_scratch_address(dev, &scratch)) != TOPLOC_OK) return rc;
  // Nothing in the scratch has to start at zero: the select kernel writes every
  // selection and status entry that the interpolation kernel goes on to read.
  return toploc_build_proofs(d_act, lay, d_proofs, d_status, d_indices_opt, scratch, kBuiltinScratchBytes,
                             cuda_stream);
}

// ---- incremental proof generation -------------------------------------------

size_t toploc_stream_state_bytes(const toploc_layout* lay) {
  return plan_stream(lay) == TOPLOC_OK ? (size_t)lay->num_seqs * stream_state_stride(lay->k) : 0;
}

size_t toploc_stream_workspace_bytes(const toploc_layout* lay) {
  if (plan_stream(lay) != TOPLOC_OK) return 0;
  return plan_workspace(false, lay->num_seqs, lay->k, lay->num_seqs, coef_bytes_of(lay)).total;
}

int toploc_stream_begin(void* d_state, const toploc_layout* lay, void* cuda_stream) {
  int rc = plan_stream(lay);
  if (rc != TOPLOC_OK) return rc;
  if (d_state == nullptr || reinterpret_cast<uintptr_t>(d_state) % 16 != 0) return TOPLOC_ERR_INVALID_ARGUMENT;
  // empty running selections: nothing held, every element is a candidate
  return cudaMemsetAsync(d_state, 0, toploc_stream_state_bytes(lay), static_cast<cudaStream_t>(cuda_stream)) ==
                 cudaSuccess
             ? TOPLOC_OK
             : TOPLOC_ERR_CUDA;
}

int toploc_stream_append(const void* d_rows, const toploc_layout* lay, int32_t token_in_chunk, void* d_state,
                         void* cuda_stream) {
  int rc = plan_stream(lay);
  if (rc != TOPLOC_OK) return rc;
  if (d_rows == nullptr || d_state == nullptr) return TOPLOC_ERR_INVALID_ARGUMENT;
  if (token_in_chunk < 0 || token_in_chunk >= lay->chunk_len) return TOPLOC_ERR_INVALID_ARGUMENT;
  if (misaligned(d_state, 16) || misaligned(d_rows, element_bytes(lay))) return TOPLOC_ERR_INVALID_ARGUMENT;
  DeviceInfo* dev = nullptr;
  if ((rc = device_info(&dev)) != TOPLOC_OK) return rc;
  // rows that are 16-byte aligned are read as vectors, others element by element
  const int mode = pick_mode(d_rows, lay) == 2 ? 2 : 0;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (lay->dtype == TOPLOC_DTYPE_BF16) launch_stream_append<0>(mode, lay, d_rows, token_in_chunk, d_state, stream);
  else launch_stream_append<1>(mode, lay, d_rows, token_in_chunk, d_state, stream);
  return cudaGetLastError() == cudaSuccess ? TOPLOC_OK : TOPLOC_ERR_CUDA;
}

int toploc_stream_finish(const void* d_state, const toploc_layout* lay, uint8_t* d_proofs, uint8_t* d_status,
                         int32_t* d_indices_opt, void* d_workspace, size_t workspace_bytes, void* cuda_stream) {
  int rc = plan_stream(lay);
  if (rc != TOPLOC_OK) return rc;
  if (d_state == nullptr || d_proofs == nullptr || d_status == nullptr) return TOPLOC_ERR_INVALID_ARGUMENT;
  if (misaligned(d_proofs, 2) || misaligned(d_state, 16) || misaligned(d_indices_opt, 4))
    return TOPLOC_ERR_INVALID_ARGUMENT;
  const WorkspacePlan wp = plan_workspace(false, lay->num_seqs, lay->k, lay->num_seqs, coef_bytes_of(lay));
  if (d_workspace == nullptr || workspace_bytes < wp.total) return TOPLOC_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(d_workspace) % 16 != 0) return TOPLOC_ERR_INVALID_ARGUMENT;
  DeviceInfo* dev = nullptr;
  if ((rc = device_info(&dev)) != TOPLOC_OK) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(d_workspace);
  BatchParams bp = {};
  bp.hidden = lay->hidden;
  bp.chunk_len = lay->chunk_len;
  bp.k = lay->k;
  bp.coef_bytes = (int)coef_bytes_of(lay);
  Selection sel;
  sel.idx = reinterpret_cast<uint32_t*>(ws + wp.idx_off);
  sel.bits = reinterpret_cast<uint16_t*>(ws + wp.bits_off);
  sel.bits32 = reinterpret_cast<uint32_t*>(ws + wp.bits_off);
  sel.status = d_status;
  sel.proofs = d_proofs;
  sel.indices = d_indices_opt;
  const unsigned char* state = static_cast<const unsigned char*>(d_state);
  const long long n = lay->num_seqs;
  if (lay->dtype == TOPLOC_DTYPE_BF16) toploc_stream_finish_kernel<0><<<(unsigned)n, kThreads, 0, stream>>>(bp, sel, state);
  else toploc_stream_finish_kernel<1><<<(unsigned)n, kThreads, 0, stream>>>(bp, sel, state);
  if (cudaGetLastError() != cudaSuccess) return TOPLOC_ERR_CUDA;
  launch_interpolation(lay, dev, sel, n, stream);
  return cudaGetLastError() == cudaSuccess ? TOPLOC_OK : TOPLOC_ERR_CUDA;
}

// Shared driver of the two host-memory entry points: groups of whole sequences
// go host -> staging -> kernels -> host, in stream order.
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
  const size_t pb = proof_bytes_of(lay);
  char* stage = static_cast<char*>(d_staging);
  int64_t* rebased = static_cast<int64_t*>(malloc(((size_t)lay->num_seqs + 1) * sizeof(int64_t)));
  if (rebased == nullptr) return TOPLOC_ERR_HOST_MEMORY;
  long long chunk0 = 0;
  int s0 = 0;
  while (s0 < lay->num_seqs && rc == TOPLOC_OK) {
    // largest group of sequences starting at s0 that fits
    int s1 = s0 + 1;
    StagingPlan sp = carve_staging_for(lay, s0, s1);
    while (s1 < lay->num_seqs) {
      StagingPlan bigger = carve_staging_for(lay, s0, s1 + 1);
      if (bigger.total > staging_bytes) break;
      sp = bigger;
      ++s1;
    }
    const long long row_a = seq_begin(lay, s0), row_b = seq_begin(lay, s1);
    long long chunks, group_segs;
    count_between(lay, s0, s1, &chunks, &group_segs);
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
                                 stage + sp.work_off, sp.work_bytes, stream);
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
                                    stage + sp.work_off, sp.work_bytes, stream);
        if (rc == TOPLOC_OK &&
            cudaMemcpyAsync(h_results + chunk0, stage + sp.small_off,
                            (size_t)chunks * sizeof(toploc_chunk_result), cudaMemcpyDeviceToHost,
                            stream) != cudaSuccess)
          rc = TOPLOC_ERR_CUDA;
      }
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
