/*
 * toploc_device.cuh -- the selection step of TopLoc as device code, for kernels
 * that produce the activations themselves.
 *
 * Section 5.5 takes the proof inside the inference engine: a hook obtains the
 * top-k values of the last hidden layer while the model decodes, one proof per
 * 32 new tokens.  The cheapest place for that hook is the kernel that writes
 * the last hidden states (the final normalisation, the epilogue of the last
 * projection): its output tile is still in shared memory, so the proof never
 * reads the activations from HBM at all.  This header gives such a kernel the
 * pieces:
 *
 *   running_selection_open    one warp loads a sequence's running top-k (the
 *                             state toploc_stream_begin prepared) into a
 *                             SelectShared scratch in shared memory
 *   running_selection_offer   the same warp tests a tile of freshly produced
 *                             values (shared or global memory) against the
 *                             running threshold and keeps what may still
 *                             belong to the chunk's top-k
 *   running_selection_close   at most k candidates go back to the state
 *
 * and toploc_stream_finish (toploc.h) turns the states into proofs once the
 * chunk is complete.  Streaming a chunk in index order while keeping the best k
 * so far, ties to the lower flat index, is exactly topk(h, k) of Algorithm 1,
 * so the proofs equal those of toploc_build_proofs over the assembled chunk.
 * toploc_rmsnorm_append (toploc.h) is a producer built this way.
 *
 * The library's own kernels are built from the same code: everything in
 * namespace toploc_device below the public part is what toploc_select_kernel,
 * toploc_verify_kernel and toploc_stream_append_kernel run.
 *
 * Rules: one full warp (32 converged lanes) drives a selection; a SelectShared
 * object (13.4 KB of shared memory; SelectSharedBig, 16.5 KB, for k above 256) belongs to that warp
 * from open to close;
 * tiles are 16-byte aligned, hold a multiple of 8 bf16 (4 fp32) values and are
 * offered in ascending flat-index order (flat index = token_in_chunk * hidden +
 * channel, at most 2^24 per chunk); k <= TOPLOC_MAX_K.
 */
#ifndef TOPLOC_DEVICE_CUH_
#define TOPLOC_DEVICE_CUH_

#include <cuda_runtime.h>
#include <stdint.h>

#include "toploc.h"

namespace toploc_device {

// ---------------------------------------------------------------------------
// launch shape
// ---------------------------------------------------------------------------
#ifndef TOPLOC_SELECT_MIN_BLOCKS
#define TOPLOC_SELECT_MIN_BLOCKS 15      // select: one-warp blocks per SM (shared memory allows 15)
#endif
#ifndef TOPLOC_SELECT_STAGES
#define TOPLOC_SELECT_STAGES 3           // select: tiles in flight per warp
#endif
constexpr int kThreads = 32;             // select: one warp per chunk
constexpr int kUnroll = 4;               // select: 16-byte loads per lane and tile
constexpr int kStages = TOPLOC_SELECT_STAGES;
#ifndef TOPLOC_CAND_CAP
#define TOPLOC_CAND_CAP 640
#endif
#ifndef TOPLOC_HIT_TRIGGER
#define TOPLOC_HIT_TRIGGER 32
#endif
#ifndef TOPLOC_HIT_TRIGGER_DIV
#define TOPLOC_HIT_TRIGGER_DIV 4
#endif
#ifndef TOPLOC_HIT_CAP
#define TOPLOC_HIT_CAP 184
#endif
#ifndef TOPLOC_HIT_CAP_BIG
#define TOPLOC_HIT_CAP_BIG 188
#endif
#ifndef TOPLOC_DRAIN_AHEAD
#define TOPLOC_DRAIN_AHEAD 1
#endif
constexpr int kDrainAhead = TOPLOC_DRAIN_AHEAD;    // select: rounds of parked vectors fetched at once (more than
                                                   // one: 2 % slower on the 70B-shaped batch, no change on small chunks)
constexpr int kHitTrigger = TOPLOC_HIT_TRIGGER;    // select: drain once this many are parked (more for large k)
constexpr int kIdxBits = 24;             // flat index field of a candidate
constexpr uint32_t kIdxMask = (1u << kIdxBits) - 1u;

// A candidate is one 64-bit word whose unsigned order is the ranking order:
// magnitude key (bit pattern without sign) descending, then flat index
// ascending.  Layout: key << 25 | (kIdxMask - index) << 1 | sign.
__device__ __forceinline__ unsigned long long make_candidate(uint32_t key, uint32_t flat, uint32_t sign) {
  return ((unsigned long long)key << (kIdxBits + 1)) | ((unsigned long long)(kIdxMask - flat) << 1) | sign;
}

// Shared memory of one selecting warp.  CAP: candidate buffer entries (8 bytes each); KMAX: the
// largest k it serves.  Two sizes are in use: SelectShared (k <= 256, 13.4 KB: sixteen warps per
// SM) and SelectSharedBig (k <= TOPLOC_MAX_K = 512, 16.5 KB: thirteen).
template <int CAP, int KMAX, int HITCAP>
struct __align__(16) SelectSharedT {
  static constexpr int kCap = CAP;
  static constexpr int kMaxK = KMAX;
  static constexpr int kHitCap = HITCAP;  // vectors that can be parked between drains
  static constexpr int kLooseKeep = CAP - 8 * kThreads;  // a mid-stream compaction may leave this many:
                                                         // a round appends at most 8 per lane
  static_assert(HITCAP >= kHitTrigger - 1 + kThreads * kUnroll, "a tile's hits must fit below the drain trigger");
  static constexpr int kMaxSlots = KMAX / 32;  // tail: entries a lane owns at most
  static_assert(CAP * 8 >= 8 * KMAX * 2, "the candidate buffer holds the maxima of the first vectors");
  static_assert(CAP >= KMAX + kThreads * 8, "a round of appends must fit after a compaction");
  static_assert(sizeof(uint4) * kStages * kUnroll * kThreads + 8 * CAP >= 8192,
                "ring + candidates double as the 65536-bit residue set");
  static_assert(sizeof(uint4) * kStages * kUnroll * kThreads >= 12 * KMAX, "the ring holds three rows of KMAX words");
  uint4 ring[kStages * kUnroll * kThreads];  // tiles on their way from HBM (asynchronous copies)
  unsigned long long cand[CAP];       // candidates held; ring + cand later serve as the residue set
  uint32_t hit_idx[HITCAP];           // vectors that passed the streaming filter, not yet unpacked
                                      // (index within the chunk; they are fetched again when unpacked)
  uint32_t top_hist[256];             // held candidates by the upper 8 bits of their 15-bit key; a
                                      // compaction borrows it for its digit histograms
  uint32_t low_hist[128];             // those whose upper bits equal top_bin, by the lower 7 bits
  uint32_t top_bin;                   // which upper-bits value low_hist describes (kNoBin: none)
  uint32_t digit;
  uint32_t bin;
  int want;
};
using SelectShared = SelectSharedT<TOPLOC_CAND_CAP, 256, TOPLOC_HIT_CAP>;
using SelectSharedBig = SelectSharedT<1024, TOPLOC_MAX_K, TOPLOC_HIT_CAP_BIG>;
// Shared memory is handed out in units of 256 bytes plus 1 KB per block, 228 KB per SM: these sizes
// are what keeps sixteen (thirteen) one-warp blocks resident.
static_assert(sizeof(SelectShared) <= 13568 && sizeof(SelectSharedBig) <= 16640, "resident blocks per SM");
static_assert(TOPLOC_MAX_K == 512, "SelectSharedBig is sized for k up to 512");
constexpr uint32_t kNoBin = 0xFFFFFFFFu;

// What the warp knows about its chunk so far.  Every lane holds the same
// values: appends are agreed on by ballot, so the counters need no atomics.
struct WarpState {
  uint32_t thr;  // an element is a candidate iff its key is >= thr
  int count;     // candidates held in sh.cand
  int nhits;     // vectors parked in sh.hit_idx
};

// The block is one warp, so a warp barrier orders its shared memory.
__device__ __forceinline__ void warp_barrier() { __syncwarp(); }

// The 15-bit key the running threshold is kept in: a bf16 key as it is, the
// upper half of an fp32 key.
template <int DT>
__device__ __forceinline__ uint32_t coarse_key(unsigned long long cand) {
  const uint32_t key = (uint32_t)(cand >> (kIdxBits + 1));
  return DT == 0 ? key : (key >> 16);
}

__device__ __forceinline__ uint4 load_streaming(const uint4* p) {
  uint4 v;
  asm("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
      : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
      : "l"(p));
  return v;
}

// 16 bytes global -> shared without passing through registers; completion is
// tracked per thread in commit groups (a thread only ever reads what it copied).
__device__ __forceinline__ void copy_async_16(uint32_t smem_dst, const void* gmem_src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void copy_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void copy_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// ---------------------------------------------------------------------------
// Where a chunk's elements live.  MODE 0: rows are contiguous (row_stride ==
// hidden) and 16-byte aligned, the chunk is one flat array of vectors.
// MODE 1: 16-byte aligned rows with padding between them.  MODE 2: anything
// else, one element at a time.  MODE 3: a flat array of 16-byte vectors behind a
// generic pointer -- a tile in shared memory (or global memory) that a producing
// kernel offers to a running selection.  DT 0 = bf16, 1 = fp32.
// ---------------------------------------------------------------------------
template <int DT, int MODE>
struct ChunkSource {
  static constexpr int kVec = (MODE == 2) ? 1 : (DT == 0 ? 8 : 4);
  static constexpr int kElemBytes = (DT == 0) ? 2 : 4;
  const char* base;
  long long row_stride;
  int hidden;
  int vecs_per_row;

  // address of vector v (not MODE 2)
  __device__ __forceinline__ const void* address(int v) const {
    if (MODE == 0 || MODE == 3) return reinterpret_cast<const uint4*>(base) + v;
    int t = v / vecs_per_row;
    int c = v - t * vecs_per_row;
    return base + ((long long)t * row_stride + (long long)c * kVec) * kElemBytes;
  }

  __device__ __forceinline__ uint4 load(int v) const {
    if (MODE == 3) {
      return *reinterpret_cast<const uint4*>(address(v));
    } else if (MODE != 2) {
      return load_streaming(reinterpret_cast<const uint4*>(address(v)));
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

// Does any element of the vector have key >= thr?  bf16: both 15-bit keys of a
// word sit in separate 16-bit lanes, and adding (0x8000 - thr) to a lane sets
// its top bit exactly when key >= thr (no carry leaves a lane).
__device__ __forceinline__ uint32_t bf16_lane_add(uint32_t thr) { return (0x8000u - thr) * 0x00010001u; }

// Per 16-bit lane the larger magnitude of two bf16 values (the sign bit of the result is not
// meaningful); a NaN in either gives the all-ones magnitude, which every threshold lets through
// to the exact unpacking.
__device__ __forceinline__ uint32_t max_magnitude_bf16x2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("max.NaN.xorsign.abs.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}

// The same for two fp32 values.
__device__ __forceinline__ uint32_t max_magnitude_f32(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("max.NaN.xorsign.abs.f32 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}

template <int DT, int VEC>
__device__ __forceinline__ bool vector_reaches(const uint4& w, uint32_t thr, uint32_t add) {
  if (VEC == 1) {
    return (DT == 0 ? (w.x & 0x7FFFu) : (w.x & 0x7FFFFFFFu)) >= thr;
  } else if (DT == 0) {
    // largest magnitude of each 16-bit lane over the four words (three packed maxima, no sign
    // masking of the inputs), then the add-and-test-top-bit comparison once
    const uint32_t m = max_magnitude_bf16x2(max_magnitude_bf16x2(w.x, w.y), max_magnitude_bf16x2(w.z, w.w));
    return (((m & 0x7FFF7FFFu) + add) & 0x80008000u) != 0;
  } else {
    const uint32_t m = max_magnitude_f32(max_magnitude_f32(w.x, w.y), max_magnitude_f32(w.z, w.w));
    return (m & 0x7FFFFFFFu) >= thr;
  }
}

// The warp walks a histogram from its highest bin down and finds the bin in
// which the want-th entry (counted from the top) falls; lane l owns bins
// PER_LANE * l .. PER_LANE * l + PER_LANE - 1.  Writes sh.digit (the bin, or
// kNoBin when the histogram holds fewer than want entries), sh.bin (its
// population) and sh.want (the rank wanted inside it).
template <int PER_LANE, class SH>
__device__ __forceinline__ void find_from_top(SH& sh, const uint32_t* hist, int want) {
  const int lane = threadIdx.x & 31;
  warp_barrier();  // histogram updates are in; results of an earlier call have been read
  uint32_t local[PER_LANE];
  uint32_t sum = 0;
#pragma unroll
  for (int b = 0; b < PER_LANE; ++b) {
    local[b] = hist[lane * PER_LANE + b];
    sum += local[b];
  }
  uint32_t incl = sum;  // becomes the sum over lanes >= this one
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    uint32_t other = __shfl_down_sync(0xFFFFFFFFu, incl, off);
    if (lane + off < 32) incl += other;
  }
  const uint32_t total = __shfl_sync(0xFFFFFFFFu, incl, 0);
  if (lane == 0 && total < (uint32_t)want) sh.digit = kNoBin;
  const uint32_t above = incl - sum;  // entries in higher lanes
  if (above < (uint32_t)want && incl >= (uint32_t)want) {
    uint32_t acc = above;
#pragma unroll
    for (int b = PER_LANE - 1; b >= 0; --b) {
      if (acc < (uint32_t)want && acc + local[b] >= (uint32_t)want) {
        sh.digit = (uint32_t)(lane * PER_LANE + b);
        sh.bin = local[b];
        sh.want = want - (int)acc;
      }
      acc += local[b];
    }
  }
  warp_barrier();
}

// Raises the threshold from the two key histograms, without touching the
// candidates: the k-th largest 15-bit key among the held candidates is found
// by walking top_hist, then low_hist, from the top.  For bf16 that key is
// exact, and since at least k held candidates reach it and every later element
// has a higher flat index, later elements must beat it strictly.  For fp32 the
// 15 bits are only the upper half of the key, so later elements need only
// reach it.
template <int DT, class SH>
__device__ __noinline__ uint32_t raise_threshold(SH& sh, int k, uint32_t thr, int count) {
  const int lane = threadIdx.x & 31;
  if (count < k) return thr;
  find_from_top<8>(sh, sh.top_hist, k);
  const uint32_t top = sh.digit;
  const int want = sh.want;
  if (top != sh.top_bin) {
    // the boundary moved into another upper-bits bin: describe that one
    warp_barrier();
    for (int b = lane; b < 128; b += kThreads) sh.low_hist[b] = 0;
    if (lane == 0) sh.top_bin = top;
    warp_barrier();
    for (int e = lane; e < count; e += kThreads) {
      const uint32_t key = coarse_key<DT>(sh.cand[e]);
      if ((key >> 7) == top) atomicAdd(&sh.low_hist[key & 127u], 1u);
    }
  }
  find_from_top<4>(sh, sh.low_hist, want);
  const uint32_t key = (top << 7) | sh.digit;
  const uint32_t raised = DT == 0 ? key + 1u : key << 16;
  return max(thr, raised);
}

// Keeps the best candidates (radix select on the 56 meaningful bits, most
// significant digit first) and sets the threshold to "strictly better than
// the k-th".  Ties on the key are only broken by index when it matters: once
// the key digits are settled the scan stops if the boundary bin can be kept
// whole -- because exactly k candidates remain, or, for a compaction in
// mid-stream (exact == false), because a round of appends still fits behind
// what remains; only the last compaction of a chunk must leave exactly k.
// Returns the new state.
template <int DT, class SH>
__device__ __noinline__ WarpState compact_candidates(SH& sh, int k, WarpState st, bool exact) {
  const int lane = threadIdx.x & 31;
  const int n = st.count;
  if (n <= k) return st;
  unsigned long long prefix = 0ull, mask = 0ull;
  int want = k;
  // bf16 keys have 15 bits: candidate bits 40..55 are zero, two digit passes fewer
#pragma unroll 1
  for (int shift = (DT == 0 ? 32 : 48); shift >= 0; shift -= 8) {
    warp_barrier();
    for (int b = lane; b < 256; b += kThreads) sh.top_hist[b] = 0;
    warp_barrier();
    for (int e = lane; e < n; e += kThreads) {
      const unsigned long long c = sh.cand[e];
      if ((c & mask) == prefix) atomicAdd(&sh.top_hist[(uint32_t)(c >> shift) & 255u], 1u);
    }
    find_from_top<8>(sh, sh.top_hist, want);  // largest digit with enough candidates at or above it
    prefix |= (unsigned long long)sh.digit << shift;
    mask |= 255ull << shift;
    want = sh.want;
    const int kept = k - want + (int)sh.bin;
    // lower bits of the pivot stay 0: the boundary bin is kept whole
    if (shift <= 24 && (kept == k || (!exact && kept <= SH::kLooseKeep))) break;
  }
  const unsigned long long pivot = prefix;  // everything >= pivot is kept
  // in place, in order: a slot is overwritten only after it has been read
  int out = 0;
  warp_barrier();
  for (int base = 0; base < n; base += kThreads) {
    const int e = base + lane;
    const unsigned long long c = e < n ? sh.cand[e] : 0ull;
    const bool keep = e < n && c >= pivot;
    const uint32_t votes = __ballot_sync(0xFFFFFFFFu, keep);
    const int pos = out + __popc(votes & ((1u << lane) - 1u));
    warp_barrier();
    if (keep) sh.cand[pos] = c;
    out += __popc(votes);
  }
  // Distinct candidates leave at most kLooseKeep here (exactly k when exact).  Equal candidates -- a
  // caller of the incremental entry points offering a flat index twice -- could leave more at the
  // cut; the buffer's arithmetic relies on the bound, so it is enforced.
  out = min(out, exact ? k : SH::kLooseKeep);
  // the key histograms describe the survivors only
  for (int b = lane; b < 256; b += kThreads) sh.top_hist[b] = 0;
  if (lane == 0) sh.top_bin = kNoBin;
  warp_barrier();
  for (int e = lane; e < out; e += kThreads) atomicAdd(&sh.top_hist[coarse_key<DT>(sh.cand[e]) >> 7], 1u);
  warp_barrier();
  st.count = out;
  st.thr = max(st.thr, (uint32_t)(pivot >> (kIdxBits + 1)) + 1u);
  return st;
}

// The cheap way to make room in mid-stream: the key histograms already know the k-th largest
// 15-bit key among the held candidates, so everything below it is dropped in one pass and the
// histograms are trimmed to match.  What remains is k plus the rest of the boundary key's bin --
// a handful on ordinary data; the caller falls back on compact_candidates when that is still too
// many (long runs of equal magnitudes).
template <int DT, class SH>
__device__ __noinline__ WarpState shed_below_kth(SH& sh, int k, WarpState st) {
  const int lane = threadIdx.x & 31;
  const int n = st.count;
  if (n <= k) return st;
  st.thr = raise_threshold<DT>(sh, k, st.thr, n);  // leaves top_bin and digit describing the k-th key
  const uint32_t top = sh.top_bin, low = sh.digit;
  const uint32_t kth = (top << 7) | low;
  int out = 0;
  warp_barrier();
  for (int base = 0; base < n; base += kThreads) {
    const int e = base + lane;
    const unsigned long long c = e < n ? sh.cand[e] : 0ull;
    const bool keep = e < n && coarse_key<DT>(c) >= kth;
    const uint32_t votes = __ballot_sync(0xFFFFFFFFu, keep);
    const int pos = out + __popc(votes & ((1u << lane) - 1u));
    warp_barrier();
    if (keep) sh.cand[pos] = c;
    out += __popc(votes);
  }
  uint32_t in_top = 0;
  for (int b = lane; b < 128; b += kThreads) {
    if ((uint32_t)b < low) sh.low_hist[b] = 0;
    else in_top += sh.low_hist[b];
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) in_top += __shfl_xor_sync(0xFFFFFFFFu, in_top, off);
  for (int b = lane; b < 256; b += kThreads) {
    if ((uint32_t)b < top) sh.top_hist[b] = 0;
    else if ((uint32_t)b == top) sh.top_hist[b] = in_top;
  }
  warp_barrier();
  st.count = out;
  return st;
}

// Bit e of the result is set iff element e of the vector has key >= thr.
template <int DT, int VEC>
__device__ __forceinline__ uint32_t passing_mask(const uint4& w, uint32_t thr) {
  if (VEC == 1) {
    return ((DT == 0 ? (w.x & 0x7FFFu) : (w.x & 0x7FFFFFFFu)) >= thr) ? 1u : 0u;
  } else if (DT == 0) {
    const uint32_t add = bf16_lane_add(thr);
    const uint32_t words[4] = {w.x, w.y, w.z, w.w};
    uint32_t m = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t t = (words[i] & 0x7FFF7FFFu) + add;  // top bit of each half: key >= thr
      m |= ((t >> 15) & 1u) << (2 * i);
      m |= (t >> 31) << (2 * i + 1);
    }
    return m;
  } else {
    return ((w.x & 0x7FFFFFFFu) >= thr ? 1u : 0u) | ((w.y & 0x7FFFFFFFu) >= thr ? 2u : 0u) |
           ((w.z & 0x7FFFFFFFu) >= thr ? 4u : 0u) | ((w.w & 0x7FFFFFFFu) >= thr ? 8u : 0u);
  }
}

// Element e (a run-time position) of a vector as (key, sign), by selects.
template <int DT, int VEC>
__device__ __forceinline__ void pick_element(const uint4& w, uint32_t e, uint32_t* key, uint32_t* sign) {
  if (VEC == 1) {
    *key = DT == 0 ? (w.x & 0x7FFFu) : (w.x & 0x7FFFFFFFu);
    *sign = DT == 0 ? (w.x >> 15) & 1u : (w.x >> 31);
  } else {
    const uint32_t wi = DT == 0 ? (e >> 1) : e;
    const uint32_t word = (wi & 2u) ? ((wi & 1u) ? w.w : w.z) : ((wi & 1u) ? w.y : w.x);
    if (DT == 0) {
      const uint32_t half = (word >> ((e & 1u) * 16u)) & 0xFFFFu;
      *key = half & 0x7FFFu;
      *sign = half >> 15;
    } else {
      *key = word & 0x7FFFFFFFu;
      *sign = word >> 31;
    }
  }
}

// Appends the elements of one vector per lane that reach the threshold.  Each
// lane counts its passing elements, a warp prefix sum hands out the slots (the
// counter is warp-uniform, no atomic), then every lane stores its own few.
// Makes room first (a mid-stream compaction) if the round would not fit.
template <int DT, int VEC, class SH>
__device__ __forceinline__ void append_round(SH& sh, int k, WarpState& st, const uint4& w, bool valid,
                                             uint32_t flat0) {
  const int lane = threadIdx.x & 31;
  uint32_t mask = 0;
  int incl = 0, total = 0;
#pragma unroll 1
  for (int attempt = 0; attempt < 2; ++attempt) {
    mask = valid ? passing_mask<DT, VEC>(w, st.thr) : 0u;
    incl = __popc(mask);
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int other = __shfl_up_sync(0xFFFFFFFFu, incl, off);
      if (lane >= off) incl += other;
    }
    total = __shfl_sync(0xFFFFFFFFu, incl, 31);
    if (st.count + total <= SH::kCap) break;
    // Both leave at most SH::kLooseKeep (a round adds at most 32 * VEC) and may raise the threshold.
    st = shed_below_kth<DT>(sh, k, st);
    if (st.count > SH::kLooseKeep) st = compact_candidates<DT>(sh, k, st, false);
  }
  int pos = st.count + incl - __popc(mask);
  const uint32_t top_bin = sh.top_bin;
  while (mask) {
    const uint32_t e = (uint32_t)__ffs((int)mask) - 1u;
    mask &= mask - 1u;
    uint32_t key, sign;
    pick_element<DT, VEC>(w, e, &key, &sign);
    const unsigned long long c = make_candidate(key, flat0 + e, sign);
    sh.cand[pos++] = c;
    const uint32_t ck = coarse_key<DT>(c);
    atomicAdd(&sh.top_hist[ck >> 7], 1u);
    if ((ck >> 7) == top_bin) atomicAdd(&sh.low_hist[ck & 127u], 1u);
  }
  __syncwarp();
  st.count += total;
}

// Processes vectors [vb, ve) one vector per lane at a time, raising the
// threshold after every round.
template <int DT, int MODE, class SH>
__device__ __noinline__ WarpState select_carefully(SH& sh, const ChunkSource<DT, MODE> src, int vb,
                                                   int ve, int k, WarpState st) {
  constexpr int VEC = ChunkSource<DT, MODE>::kVec;
  const int lane = threadIdx.x & 31;
  for (int s = vb; s < ve; s += kThreads) {
    const int v = s + lane;
    const bool valid = v < ve;
    uint4 w = make_uint4(0, 0, 0, 0);
    if (valid) w = src.load(v);
    append_round<DT, VEC>(sh, k, st, w, valid, (uint32_t)v * VEC);
    // early rounds move the threshold a lot, later ones little: raise after every round at
    // first, then after every other one (and after the last)
    const int round = (s - vb) / kThreads;
    if (round < 6 || (round & 1) || s + kThreads >= ve) st.thr = raise_threshold<DT>(sh, k, st.thr, st.count);
  }
  return st;
}

// Unpacks the parked hit vectors into candidates (against the current,
// possibly higher, threshold), one vector per lane and round, then raises the
// threshold.  Only the vector's index was parked: the 16 bytes are fetched
// again (they were read moments ago, so this rarely reaches DRAM).
template <int DT, int MODE, class SH>
__device__ __noinline__ WarpState drain_hits(SH& sh, const ChunkSource<DT, MODE> src, int k,
                                             WarpState st) {
  constexpr int VEC = ChunkSource<DT, MODE>::kVec;
  const int lane = threadIdx.x & 31;
  warp_barrier();  // the parked indices are visible
  // The fetches of kDrainAhead rounds are issued together (a fetch waits behind the SM's own
  // streaming requests for thousands of cycles).
  for (int base = 0; base < st.nhits; base += kDrainAhead * kThreads) {
    uint4 w[kDrainAhead];
    uint32_t v[kDrainAhead];
#pragma unroll
    for (int r = 0; r < kDrainAhead; ++r) {
      const int h = base + r * kThreads + lane;
      w[r] = make_uint4(0, 0, 0, 0);
      v[r] = 0;
      if (h < st.nhits) {
        v[r] = sh.hit_idx[h];
        w[r] = src.load((int)v[r]);
      }
    }
#pragma unroll
    for (int r = 0; r < kDrainAhead; ++r) {
      const int h = base + r * kThreads + lane;
      if (base + r * kThreads < st.nhits) append_round<DT, VEC>(sh, k, st, w[r], h < st.nhits, v[r] * VEC);
    }
  }
  st.nhits = 0;
  st.thr = raise_threshold<DT>(sh, k, st.thr, st.count);
  return st;
}

// Parked vectors are unpacked once this many of them wait.  A larger k admits more of them and
// every drain ends with a look at the key histograms, so the trigger grows with k as far as the
// parking space allows (one tile can park kThreads * kUnroll more).
template <class SH>
__device__ __forceinline__ int drain_trigger(int k) {
  return min(max(kHitTrigger, k / TOPLOC_HIT_TRIGGER_DIV), SH::kHitCap - kThreads * kUnroll + 1);
}

// Largest key in one vector, as the 15-bit key the threshold is kept in.
template <int DT, int VEC>
__device__ __forceinline__ uint32_t vector_max_coarse_key(const uint4& w) {
  if (VEC == 1) {
    return DT == 0 ? (w.x & 0x7FFFu) : ((w.x & 0x7FFFFFFFu) >> 16);
  } else if (DT == 0) {
    const uint32_t m = __vmaxu2(__vmaxu2(w.x & 0x7FFF7FFFu, w.y & 0x7FFF7FFFu),
                                __vmaxu2(w.z & 0x7FFF7FFFu, w.w & 0x7FFF7FFFu));
    return max(m & 0xFFFFu, m >> 16);
  } else {
    return max(max(w.x & 0x7FFFFFFFu, w.y & 0x7FFFFFFFu), max(w.z & 0x7FFFFFFFu, w.w & 0x7FFFFFFFu)) >> 16;
  }
}

// A sound first threshold from the chunk's first n_first vectors (n_first >= k):
// the k-th largest of their per-vector maxima.  Each maximum is a different
// element, so at least k elements of the chunk reach it and the k-th largest
// element cannot lie below it.  Uses the candidate buffer to hold the maxima
// and leaves the histograms empty again.
template <int DT, int MODE, class SH>
__device__ __noinline__ uint32_t sound_first_threshold(SH& sh, const ChunkSource<DT, MODE> src,
                                                       int n_first, int k, int ring_vecs) {
  constexpr int VEC = ChunkSource<DT, MODE>::kVec;
  const int lane = threadIdx.x & 31;
  uint16_t* maxima = reinterpret_cast<uint16_t*>(sh.cand);
  warp_barrier();
  // The first ring_vecs vectors are on their way into the ring already (vector v in slot v,
  // copied by the lane that reads it here): the vectors beyond them are loaded first, then the
  // ring's are taken from shared memory once they have landed -- one round trip to memory for
  // the whole look-ahead of the common case instead of one per four vectors of a lane.
  if (ring_vecs > n_first) ring_vecs = n_first;
#pragma unroll 4
  for (int v = ring_vecs + lane; v < n_first; v += kThreads) {
    const uint32_t key = vector_max_coarse_key<DT, VEC>(src.load(v));
    maxima[v] = (uint16_t)key;
    atomicAdd(&sh.top_hist[key >> 7], 1u);
  }
  if (ring_vecs > 0) copy_async_wait<0>();
  for (int v = lane; v < ring_vecs; v += kThreads) {
    const uint32_t key = vector_max_coarse_key<DT, VEC>(sh.ring[v]);
    maxima[v] = (uint16_t)key;
    atomicAdd(&sh.top_hist[key >> 7], 1u);
  }
  find_from_top<8>(sh, sh.top_hist, k);
  const uint32_t top = sh.digit;
  const int want = sh.want;
  for (int b = lane; b < 128; b += kThreads) sh.low_hist[b] = 0;
  warp_barrier();
  for (int v = lane; v < n_first; v += kThreads) {
    const uint32_t key = maxima[v];
    if ((key >> 7) == top) atomicAdd(&sh.low_hist[key & 127u], 1u);
  }
  find_from_top<4>(sh, sh.low_hist, want);
  const uint32_t key = (top << 7) | sh.digit;
  warp_barrier();
  for (int b = lane; b < 256; b += kThreads) sh.top_hist[b] = 0;
  warp_barrier();
  return DT == 0 ? key : key << 16;
}

// Exact top-k of one chunk by one warp: on return sh.cand[0..k) holds the k
// selected candidates (in no particular order).  n_elems >= k is the caller's
// business.
//
// The chunk is streamed in index order.  A warm-up over the first vectors
// establishes a threshold; after that a lane only tests whether a 16-byte
// vector holds anything at or above the threshold and, if so, the vector is
// parked in shared memory.  Parked vectors are unpacked by the whole warp at
// once, so the rare slow work is done with every lane busy.  Nothing here
// waits on another warp: a chunk's serial steps only delay that chunk, while
// the other warps of the SM keep their own loads in flight.
template <int DT, int MODE, class SH>
__device__ void select_topk(SH& sh, const ChunkSource<DT, MODE>& src, int n_elems, int k) {
  constexpr int VEC = ChunkSource<DT, MODE>::kVec;
  constexpr int kTileVecs = kThreads * kUnroll;
  const int lane = threadIdx.x & 31;
  const uint32_t below = (1u << lane) - 1u;
  const int n_vecs = n_elems / VEC;

  for (int b = lane; b < 256; b += kThreads) sh.top_hist[b] = 0;
  if (lane == 0) sh.top_bin = kNoBin;
  WarpState st;
  st.thr = 0;  // accept everything until k candidates exist
  st.count = 0;
  st.nhits = 0;

  // Before streaming, a threshold that only a minority of vectors reach.  Large
  // aligned chunks get it from a look at the maxima of their first vectors
  // (which are then streamed like everything else); otherwise the first vectors
  // are selected from directly.
  const int trigger = drain_trigger<SH>(k);
  const int first = (32 / VEC) * max(k, 128);
  const bool look_ahead = (MODE != 2) && n_vecs >= first;
  const int warm = look_ahead ? 0 : min(n_vecs, first);
  const int n_tiles = (n_vecs - warm) / kTileVecs;
  const int full_end = warm + n_tiles * kTileVecs;

  // Streaming tiles travel through a ring of kStages tiles in shared memory,
  // filled by asynchronous 16-byte copies: the loads of the next tiles are in
  // flight, at no cost in registers, while this tile is filtered and while the
  // warp drains or compacts.  Slot (stage, u, lane) is private to its lane.
  // The first tiles are requested before the warm-up starts.
  static_assert(MODE != 3, "whole chunks are streamed from global memory");
  constexpr bool kRing = (MODE != 2);
  const uint32_t ring_lane = (uint32_t)__cvta_generic_to_shared(&sh.ring[lane]);
  constexpr uint32_t kStageBytes = kUnroll * kThreads * sizeof(uint4);
  // stage is a compile-time constant at every call site (the tile loop is unrolled by kStages)
  auto request_tile = [&](int tile, int stage) {
    if (kRing && tile < n_tiles) {
      const uint32_t dst = ring_lane + (uint32_t)stage * kStageBytes;
      if (MODE == 0) {
        const char* g = src.base + ((size_t)(warm + tile * kTileVecs + lane)) * sizeof(uint4);
#pragma unroll
        for (int u = 0; u < kUnroll; ++u)
          copy_async_16(dst + (uint32_t)(u * kThreads * sizeof(uint4)), g + u * kThreads * sizeof(uint4));
      } else {
        const int v = warm + tile * kTileVecs + lane;
#pragma unroll
        for (int u = 0; u < kUnroll; ++u)
          copy_async_16(dst + (uint32_t)(u * kThreads * sizeof(uint4)), src.address(v + u * kThreads));
      }
    }
    if (kRing) copy_async_commit();
  };
#pragma unroll
  for (int t = 0; t < kStages; ++t) request_tile(t, t);
  warp_barrier();

  if (look_ahead) st.thr = sound_first_threshold<DT, MODE>(sh, src, first, k, kRing ? min(n_tiles, kStages) * kTileVecs : 0);
  else st = select_carefully<DT, MODE>(sh, src, 0, warm, k, st);

  for (int tile0 = 0; tile0 < n_tiles; tile0 += kStages) {
#pragma unroll
    for (int stage = 0; stage < kStages; ++stage) {
      const int tile = tile0 + stage;
      if (tile >= n_tiles) break;
      const int v0 = warm + tile * kTileVecs;
      uint4 w[kUnroll];
      if (kRing) {
        copy_async_wait<kStages - 1>();  // this lane's copies of `tile` have landed
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) w[u] = sh.ring[(stage * kUnroll + u) * kThreads + lane];
        // Refill the stage as soon as the tile is in registers instead of after its tests.  The
        // instructions below read one register of every load, so they issue only once all of
        // them have returned; the copies are issued after them and cannot overwrite a slot
        // that is still being read.
        uint32_t landed = 0;
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) asm volatile("or.b32 %0, %0, %1;" : "+r"(landed) : "r"(w[u].x));
        request_tile(tile + kStages, stage);
      } else {
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) w[u] = src.load(v0 + u * kThreads + lane);
      }
      const uint32_t add = bf16_lane_add(st.thr);
      // the tests of a tile's vectors are independent of each other: all of them first,
      // then the votes, then one warp-uniform branch for the (less common) tile with a hit
      bool hit[kUnroll];
      uint32_t votes[kUnroll];
      uint32_t any_votes = 0;
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) hit[u] = vector_reaches<DT, VEC>(w[u], st.thr, add);
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        votes[u] = __ballot_sync(0xFFFFFFFFu, hit[u]);
        any_votes |= votes[u];
      }
      if (any_votes) {
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
          if (hit[u]) {
            const int pos = st.nhits + __popc(votes[u] & below);
            sh.hit_idx[pos] = (uint32_t)(v0 + u * kThreads + lane);
          }
          st.nhits += __popc(votes[u]);
        }
      }
      if (!kRing) request_tile(tile + kStages, stage);  // (keeps the commit-group count in step; no copies)
      // a tile parks at most kTileVecs vectors, so the buffer cannot overflow
      if (st.nhits >= trigger) st = drain_hits<DT, MODE>(sh, src, k, st);
    }
  }
  if (kRing) copy_async_wait<0>();
  st = drain_hits<DT, MODE>(sh, src, k, st);
  st = select_carefully<DT, MODE>(sh, src, full_end, n_vecs, k, st);
  compact_candidates<DT>(sh, k, st, true);  // exactly k remain
  warp_barrier();
}

struct StreamHeader {  // per sequence, followed by kMaxK-independent room for k candidates
  uint32_t count;      // candidates held (at most k between steps)
  uint32_t thr;        // an element is a candidate iff its key is >= thr
  uint32_t pad[2];
};

__host__ __device__ inline size_t stream_state_stride(int k) { return sizeof(StreamHeader) + 8 * (size_t)k; }

// Vectors [vb, ve) against a threshold that is already meaningful: the filter of the select kernel's
// streaming loop (test, park the vectors that reach the threshold, unpack them by the warp), with
// plain loads instead of the ring.
template <int DT, int MODE, class SH>
__device__ __forceinline__ WarpState filter_vectors(SH& sh, const ChunkSource<DT, MODE>& src, int vb, int ve,
                                                    int k, WarpState st) {
  constexpr int VEC = ChunkSource<DT, MODE>::kVec;
  const int lane = threadIdx.x & 31;
  const uint32_t below = (1u << lane) - 1u;
  const int trigger = drain_trigger<SH>(k);
  for (int v0 = vb; v0 < ve; v0 += kThreads * kUnroll) {
    uint4 w[kUnroll];
    bool hit[kUnroll];
    uint32_t votes[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int v = v0 + u * kThreads + lane;
      w[u] = v < ve ? src.load(v) : make_uint4(0, 0, 0, 0);
    }
    const uint32_t add = bf16_lane_add(st.thr);
    uint32_t any_votes = 0;
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      hit[u] = (v0 + u * kThreads + lane < ve) && vector_reaches<DT, VEC>(w[u], st.thr, add);
      votes[u] = __ballot_sync(0xFFFFFFFFu, hit[u]);
      any_votes |= votes[u];
    }
    if (any_votes) {
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        if (hit[u]) sh.hit_idx[st.nhits + __popc(votes[u] & below)] = (uint32_t)(v0 + u * kThreads + lane);
        st.nhits += __popc(votes[u]);
      }
      if (st.nhits >= trigger) st = drain_hits<DT, MODE>(sh, src, k, st);
    }
  }
  return drain_hits<DT, MODE>(sh, src, k, st);
}


// ---------------------------------------------------------------------------
// Running selections from inside a producing kernel (see the top of this file).
// DT: 0 = bf16 values, 1 = fp32 values.  `state` points at ONE sequence's state:
// d_state + sequence * running_selection_bytes(k).
// ---------------------------------------------------------------------------
__host__ __device__ inline size_t running_selection_bytes(int k) { return stream_state_stride(k); }

template <int DT, class SH>
__device__ __forceinline__ WarpState running_selection_open(SH& sh, const unsigned char* state, int k) {
  const int lane = threadIdx.x & 31;
  const StreamHeader* head = reinterpret_cast<const StreamHeader*>(state);
  const unsigned long long* held = reinterpret_cast<const unsigned long long*>(head + 1);
  WarpState st;
  st.count = min((int)head->count, k);  // a state holds at most k candidates
  st.thr = head->thr;
  st.nhits = 0;
  for (int b = lane; b < 256; b += kThreads) sh.top_hist[b] = 0;
  if (lane == 0) sh.top_bin = kNoBin;
  warp_barrier();
  for (int e = lane; e < st.count; e += kThreads) {
    const unsigned long long c = held[e];
    sh.cand[e] = c;
    atomicAdd(&sh.top_hist[coarse_key<DT>(c) >> 7], 1u);
  }
  warp_barrier();
  return st;
}

// Vectors [vb, ve) of a source against the running selection: once k candidates are held the
// threshold does the work; before that every element is a candidate.
template <int DT, int MODE, class SH>
__device__ __forceinline__ WarpState running_selection_take(SH& sh, WarpState st,
                                                            const ChunkSource<DT, MODE>& src, int vb, int ve, int k) {
  if (st.count >= k) return filter_vectors<DT, MODE>(sh, src, vb, ve, k, st);
  return select_carefully<DT, MODE>(sh, src, vb, ve, k, st);
}

// tile: n_elems values whose first one has flat index flat_base within the chunk.
template <int DT, class SH>
__device__ __forceinline__ WarpState running_selection_offer(SH& sh, WarpState st, const void* tile,
                                                             int n_elems, uint32_t flat_base, int k) {
  constexpr int VEC = ChunkSource<DT, 3>::kVec;
  constexpr int kElem = ChunkSource<DT, 3>::kElemBytes;
  ChunkSource<DT, 3> src;
  // vector v of the source is the chunk's elements v * VEC ..: the tile's first vector is flat_base / VEC
  src.base = static_cast<const char*>(tile) - (long long)flat_base * kElem;
  src.row_stride = 0;
  src.hidden = 0;
  src.vecs_per_row = 0;
  const int vb = (int)(flat_base / VEC);
  return running_selection_take<DT, 3>(sh, st, src, vb, vb + n_elems / VEC, k);
}

template <int DT, class SH>
__device__ __forceinline__ void running_selection_close(SH& sh, WarpState st, unsigned char* state, int k) {
  const int lane = threadIdx.x & 31;
  StreamHeader* head = reinterpret_cast<StreamHeader*>(state);
  unsigned long long* held = reinterpret_cast<unsigned long long*>(head + 1);
  st = compact_candidates<DT>(sh, k, st, true);  // at most k are carried to the next step
  // (Candidates are distinct as long as every flat index is offered once.  A caller that offers
  // an index twice can leave equal candidates at the cut; the state still never takes more than k.)
  st.count = min(st.count, k);
  warp_barrier();
  for (int e = lane; e < st.count; e += kThreads) held[e] = sh.cand[e];
  if (lane == 0) {
    head->count = (uint32_t)st.count;
    head->thr = st.thr;
  }
}

}  // namespace toploc_device

#endif  // TOPLOC_DEVICE_CUH_
