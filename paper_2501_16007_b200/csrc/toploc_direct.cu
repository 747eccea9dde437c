// toploc_direct.cu -- direct commitments for sm_100a: the top-k indices and values of a
// chunk stored as they are (Section 4: 6 bytes per point), for k up to 4096 (the range of
// the exponent-error table in Section 3), and their validation (Algorithm 2 with the
// polynomial evaluation replaced by an index look-up).
//
// Kernels, by the shape of the call:
//   k <= 256 (k <= 512 where the next pair does not apply), chunks of at most 2^19 elements:
//     toploc_direct_commit_warp_kernel / toploc_direct_verify_warp_kernel -- one warp per chunk,
//     the selection of the proof path (toploc_device::select_topk);
//   k > 256, 16-byte aligned rows, chunks of at most 2^18 elements:
//     toploc_direct_commit_half_kernel / toploc_direct_verify_half_kernel -- one 512-thread block
//     per chunk, two per SM; the chunk is streamed once (select_unordered with the bytes of its
//     first pass); chunks whose candidates outgrow the buffer go to toploc_direct_*_rescue_kernel;
//   everything else:
//     toploc_direct_commit_kernel / toploc_direct_verify_kernel<dtype, vector> -- one 1024-thread
//     block per chunk: select_unordered with a second streaming pass (aligned rows, at most 2^19
//     elements), else one of the two selections below.
//
// The two older selections of the 1024-thread kernels:
//   one pass (vector layouts, k <= 2048): the chunk is streamed once; elements that reach a
//   running threshold are kept as candidates in shared memory, in index order, and counted in a
//   histogram of their upper 11 key bits, from which the threshold is raised as candidates
//   arrive; the exact k-th key is then found among the candidates (select_in_one_pass);
//   two passes (everything else, and chunks whose candidates outgrow their buffer): a radix
//   select on the magnitude key with the whole first digit -- 15 bits, i.e. every bf16 key --
//   histogrammed in shared memory.  A first part of the chunk is counted in full; the k-th
//   largest key of that part is a sound lower bound for the chunk's k-th largest key, so the
//   rest of the chunk only counts elements that reach it.  fp32 keys take two more 8-bit digits
//   over the elements that match the digits found so far.  A last pass in index order takes
//   every key above the k-th largest and the first elements equal to it (ties go to the lower
//   index) and places them, by a block-wide prefix sum, in ascending index order.  The chunk is
//   read from HBM by the first pass; the second finds it in L2 (one block per SM: 148 chunks
//   in flight).
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "nearest_ratio.cuh"
#include "toploc.h"
#include "toploc_device.cuh"

namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kTopBits = 15;                 // width of the first digit
constexpr int kBins = 1 << kTopBits;
constexpr int kUnroll = 4;                   // 16-byte loads in flight per thread
constexpr int kMaxChunkElems = 1 << 24;
constexpr int kListOffset = 256;             // verify: words of the histogram kept for the mantissa differences
constexpr size_t kRingBytes = (size_t)kUnroll * kThreads * 16;

struct DirectParams {
  const void* act;
  long long row_stride;      // elements
  long long tokens_per_seq;
  int hidden;
  int chunk_len;
  int k;
  int chunks_per_seq;
};

struct DirectVerify {
  const uint8_t* commits;
  toploc_chunk_result* results;
  uint32_t* exp_dev;         // optional [num_chunks, 9]
  toploc_thresholds thr;              // thresholds of the call ...
  const toploc_thresholds* thr_each;  // ... or, when not null, one entry per chunk (device memory)
};

// Dynamic shared memory of a block: the copy ring, this struct, and kSpareBytes that continue
// its last member (the one-pass selection keeps its candidates in hist and the spare together).
// Scalars of the two-pass selection without barriers (select_unordered), in shared memory.
struct LooseControl {
  unsigned long long warp_sums[2][32];
  uint32_t picked_bin;
  uint32_t picked_remaining;
  uint32_t cand_count;       // candidates handed out so far (may run past the buffer: then overflow is set)
  uint32_t thr;              // an element is a candidate iff its key is >= thr; only ever raised
  uint32_t last_raise;       // cand_count when thr was last raised
  uint32_t raise_lock;       // 1 while a warp is raising thr
  uint32_t overflow;
  uint32_t emitted;
};

struct DirectShared {
  unsigned long long warp_sums[2][kWarps];
  uint32_t picked_bin;
  uint32_t picked_remaining;
  uint32_t bad;
  uint32_t counters[4];      // exponent mismatches, matches, mantissa difference sum, common indices
  uint32_t dev[9];
  uint32_t pad[4];
  LooseControl loose;
  uint32_t hist[kBins];
};
constexpr size_t kSpareBytes = 34704;
constexpr size_t kSharedBytes = kRingBytes + sizeof(DirectShared) + kSpareBytes;
// One-pass selection (vector layouts, k <= kStreamMaxK): a histogram of the upper 11 key bits
// and up to cand_cap candidates (flat index, whole pattern) in index order.
constexpr int kCoarseBins = 2048;
__host__ __device__ constexpr int cand_cap(int dt) { return dt == 0 ? 25984 : 19584; }       // 6 / 8 bytes each
constexpr int kStreamMaxK = 2048;   // beyond it the candidates of a 2^18-element chunk no longer fit
static_assert(kSharedBytes <= 227 * 1024 && sizeof(DirectShared) % 16 == 0 && kSpareBytes % 16 == 0, "shared memory budget");
static_assert(offsetof(DirectShared, hist) + sizeof(uint32_t) * kBins == sizeof(DirectShared), "hist is the last member");
static_assert((size_t)kCoarseBins * 4 + (size_t)cand_cap(0) * 6 <= (size_t)kBins * 4 + kSpareBytes &&
                  (size_t)kCoarseBins * 4 + (size_t)cand_cap(1) * 8 <= (size_t)kBins * 4 + kSpareBytes,
              "candidates fit");
static_assert(12 * TOPLOC_MAX_K_DIRECT <= kRingBytes, "the verify lists fit the idle ring");
// The free-running one-pass selection parks, per warp, the vectors that passed the quick test
// until there are enough of them to unpack with every lane busy; its candidates are unordered.
constexpr int kParkCap = 64 + kUnroll * 32;   // a batch parks at most kUnroll vectors per lane
constexpr int kParkTrigger = 64;              // at most: a round of unpacking takes two vectors per lane
constexpr size_t kParkBytes = (size_t)kWarps * kParkCap * 4;
__host__ __device__ constexpr int loose_cap(int dt) {
  return (int)(((size_t)kBins * 4 + kSpareBytes - (size_t)kCoarseBins * 4 - kParkBytes) / (dt == 0 ? 6 : 8)) / 64 * 64;
}
constexpr int kLooseMaxElems = 1 << 19;       // its index-order bitmap must fit the ring
static_assert((size_t)kLooseMaxElems / 8 <= kRingBytes, "one bit per element of the chunk");
static_assert(loose_cap(0) >= 5 * 4096 && loose_cap(1) >= 4 * 4096, "room for the candidates of k = 4096");

// A group is VEC consecutive elements of one row (one 16-byte vector, or one element when
// the layout does not allow aligned vectors).
template <int DT, bool VECTOR>
struct Reader {
  static constexpr int ESZ = DT == 0 ? 2 : 4;
  static constexpr int VEC = VECTOR ? 16 / ESZ : 1;
  const char* base;
  long long row_stride_bytes;
  int groups_per_row;
  int n_groups;
  bool flat;

  __device__ __forceinline__ const char* address(int g) const {
    if (flat) return base + (long long)g * (VEC * ESZ);  // rows follow one another without a gap
    const int row = g / groups_per_row;
    const int col = g - row * groups_per_row;
    return base + row * row_stride_bytes + (long long)col * (VEC * ESZ);
  }

  // A batch is this thread's groups first + u * kThreads, u < kUnroll, below g_end.  Vector
  // layouts move a batch through the thread's own kUnroll 16-byte slots of the ring in shared
  // memory with asynchronous copies: request() starts the copies, take() waits for them and
  // moves the slots to registers, after which the next batch may be requested -- so a batch is
  // in flight while the previous one is worked on, barriers included.  Nothing waits on
  // another thread.  Other layouts load directly in take().
  template <int T = kThreads>
  __device__ __forceinline__ void request(uint4* ring, int first, int g_end) const {
    if constexpr (VECTOR) {
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int g = first + u * T;
        if (g < g_end) {
          const uint32_t dst = (uint32_t)__cvta_generic_to_shared(ring + u * T + threadIdx.x);
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(address(g)) : "memory");
        }
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
  }
  // The same, for the batch after one whose registers are w: each copy's destination is made
  // to depend on the register that was read from it, so the copy cannot overtake the read.
  template <int T = kThreads>
  __device__ __forceinline__ void request_after(uint4* ring, int first, int g_end, const uint32_t (&w)[kUnroll][4],
                                                int prev_first, int prev_end) const {
    if constexpr (VECTOR) {
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int g = first + u * T;
        if (g < g_end) {
          uint32_t dst = (uint32_t)__cvta_generic_to_shared(ring + u * T + threadIdx.x);
          if (prev_first + u * T < prev_end) {
            uint32_t zero;
            asm volatile("and.b32 %0, %1, 0;" : "=r"(zero) : "r"(w[u][3]));
            dst += zero;
          }
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(address(g)) : "memory");
        }
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
  }
  template <int T = kThreads>
  __device__ __forceinline__ void take(const uint4* ring, int first, int g_end, uint32_t (&w)[kUnroll][4]) const {
    if (VECTOR) asm volatile("cp.async.wait_group 0;" ::: "memory");
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int g = first + u * T;
      if (g < g_end) {
        if (VECTOR) {
          const uint4 v = ring[u * T + threadIdx.x];
          w[u][0] = v.x; w[u][1] = v.y; w[u][2] = v.z; w[u][3] = v.w;
        } else if (DT == 0) {
          w[u][0] = *reinterpret_cast<const uint16_t*>(address(g));
        } else {
          w[u][0] = *reinterpret_cast<const uint32_t*>(address(g));
        }
      }
    }
  }
  // whole pattern of element j of a loaded group, j known at run time (no indexed registers)
  __device__ __forceinline__ static uint32_t pattern_at(const uint32_t (&w)[4], uint32_t j) {
    if (!VECTOR) return w[0];
    if (DT == 0) {
      const uint32_t lo = (j & 2u) ? w[1] : w[0], hi = (j & 2u) ? w[3] : w[2];
      const uint32_t word = (j & 4u) ? hi : lo;
      return (j & 1u) ? word >> 16 : word & 0xFFFFu;
    }
    const uint32_t lo = (j & 1u) ? w[1] : w[0], hi = (j & 1u) ? w[3] : w[2];
    return (j & 2u) ? hi : lo;
  }
  // Bit j is set iff the key of element j is >= thr; thr may be one past the largest key
  // (no bit set).  bf16 vectors: per word, (keys + (2^15 - thr)) carries into bits 15 and 31
  // exactly for the keys that reach thr (keys have 15 bits, so nothing crosses the halves).
  __device__ __forceinline__ static uint32_t reach_mask(const uint32_t (&w)[4], uint32_t thr) {
    if (!VECTOR) return key(w[0]) >= thr ? 1u : 0u;
    if (DT == 0) {
      const uint32_t add = (0x8000u - thr) * 0x00010001u;
      const uint32_t m0 = ((w[0] & 0x7FFF7FFFu) + add) & 0x80008000u;
      const uint32_t m1 = ((w[1] & 0x7FFF7FFFu) + add) & 0x80008000u;
      const uint32_t m2 = ((w[2] & 0x7FFF7FFFu) + add) & 0x80008000u;
      const uint32_t m3 = ((w[3] & 0x7FFF7FFFu) + add) & 0x80008000u;
      const uint32_t m = (m0 >> 15) | (m1 >> 13) | (m2 >> 11) | (m3 >> 9);  // even elements at bits 0..6, odd at 16..22
      return (m | (m >> 15)) & 0xFFu;
    }
    return ((w[0] & 0x7FFFFFFFu) >= thr ? 1u : 0u) | ((w[1] & 0x7FFFFFFFu) >= thr ? 2u : 0u) |
           ((w[2] & 0x7FFFFFFFu) >= thr ? 4u : 0u) | ((w[3] & 0x7FFFFFFFu) >= thr ? 8u : 0u);
  }
  __device__ __forceinline__ static uint32_t key(uint32_t pat) { return DT == 0 ? pat & 0x7FFFu : pat & 0x7FFFFFFFu; }
  __device__ __forceinline__ static uint32_t committed(uint32_t pat) { return DT == 0 ? pat : pat >> 16; }
};

__host__ __device__ constexpr int key_bits(int dt) { return dt == 0 ? 15 : 31; }

// Exclusive prefix sum over the block of a 64-bit value (callers pack several small counters
// into it); *total receives the block's sum.  `slot` alternates between calls so that one
// barrier per call is enough.
__device__ __forceinline__ unsigned long long block_scan_exclusive(DirectShared& sh, unsigned long long v, int slot,
                                                                   unsigned long long* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned long long inc = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const unsigned long long o = __shfl_up_sync(0xFFFFFFFFu, inc, d);
    if (lane >= d) inc += o;
  }
  if (lane == 31) sh.warp_sums[slot][warp] = inc;
  __syncthreads();
  unsigned long long mine = sh.warp_sums[slot][lane];  // kWarps == 32: lane w holds warp w's sum
  unsigned long long winc = mine;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const unsigned long long o = __shfl_up_sync(0xFFFFFFFFu, winc, d);
    if (lane >= d) winc += o;
  }
  *total = __shfl_sync(0xFFFFFFFFu, winc, 31);
  const unsigned long long before_warp = __shfl_sync(0xFFFFFFFFu, winc - mine, warp);
  return before_warp + inc - v;
}
static_assert(kWarps == 32, "the second level of the block scan is one warp wide");
static_assert(kListOffset * 4 + 12 * TOPLOC_MAX_K_DIRECT <= kBins * 4, "the verify lists fit where the histogram was");
static_assert((kBins / kThreads & (kBins / kThreads - 1)) == 0, "bins per thread: a power of two");

// The bin, counted from the top, in which the want-th largest counted element lies
// (1 <= want <= number of counted elements): sh.picked_bin, and sh.picked_remaining = want
// minus the elements in higher bins.  All threads call; ends with a barrier.
__device__ __forceinline__ void find_bin_from_top(DirectShared& sh, int nbins, uint32_t want, int slot) {
  const int per = nbins >= kThreads ? nbins / kThreads : 1;
  const int top = nbins - 1 - (int)threadIdx.x * per;  // this thread owns bins top, top-1, ..., top-per+1
  uint32_t s = 0;
  if (top >= 0)  // each lane starts at another offset: its bins are `per` words apart from its neighbour's
    for (int b = 0; b < per; ++b) s += sh.hist[top - ((b + (int)threadIdx.x) & (per - 1))];
  unsigned long long total;
  const uint32_t before = (uint32_t)block_scan_exclusive(sh, s, slot, &total);
  if (top >= 0 && before < want && want <= before + s) {
    uint32_t c = before;
    for (int b = 0; b < per; ++b) {
      const uint32_t h = sh.hist[top - b];
      if (c + h >= want) {
        sh.picked_bin = (uint32_t)(top - b);
        sh.picked_remaining = want - c;
        break;
      }
      c += h;
    }
  }
  __syncthreads();
}

// Counts, over groups [g_begin, g_end), digit (key >> shift) & dmask of every element with
// lo_key <= key < hi_key.  A group is tested as a whole; only the elements that pass are
// looked at one by one.
template <int DT, bool VECTOR>
__device__ __forceinline__ void histogram_pass(DirectShared& sh, uint4* ring, const Reader<DT, VECTOR>& rd, int g_begin, int g_end,
                                               uint32_t lo_key, uint32_t hi_key, int shift, uint32_t dmask) {
  using R = Reader<DT, VECTOR>;
  constexpr uint32_t kLargestKey = DT == 0 ? 0x7FFFu : 0x7FFFFFFFu;
  rd.request(ring, g_begin + (int)threadIdx.x, g_end);
  for (int base = g_begin; base < g_end; base += kUnroll * kThreads) {
    const int g0 = base + (int)threadIdx.x;
    uint32_t w[kUnroll][4];
    rd.take(ring, g0, g_end, w);
    if (base + kUnroll * kThreads < g_end) rd.request_after(ring, g0 + kUnroll * kThreads, g_end, w, g0, g_end);
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int g = g0 + u * kThreads;
      if (g < g_end) {
        uint32_t m = R::reach_mask(w[u], lo_key);
        if (hi_key <= kLargestKey) m &= ~R::reach_mask(w[u], hi_key);
        while (m) {
          const uint32_t j = (uint32_t)__ffs((int)m) - 1u;
          m &= m - 1u;
          atomicAdd(&sh.hist[(R::key(R::pattern_at(w[u], j)) >> shift) & dmask], 1u);
        }
      }
    }
  }
}

__device__ __forceinline__ void clear_bins(DirectShared& sh, int nbins) {  // nbins: a multiple of 4
  uint4* h = reinterpret_cast<uint4*>(sh.hist);
  for (int b = threadIdx.x; b < nbins / 4; b += kThreads) h[b] = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
}

// The k-th largest key of the chunk (*kth) and how many elements equal to it belong to the
// top-k (*take >= 1; the k - *take others have larger keys).  Requires k <= elements.
template <int DT, bool VECTOR>
__device__ void find_kth_key(DirectShared& sh, uint4* ring, const Reader<DT, VECTOR>& rd, int k, uint32_t* kth,
                             uint32_t* take) {
  using R = Reader<DT, VECTOR>;
  constexpr int BITS = key_bits(DT);
  constexpr int SHIFT0 = BITS - kTopBits;
  clear_bins(sh, kBins);
  // First part of the chunk in full; its k-th largest bounds the chunk's from below.  A part of
  // a elements costs a atomics and lets about (n - a) k / a of the others through, least for
  // a = sqrt(n k): the smallest power-of-two multiple of 2k elements that reaches it.
  int g_part = (2 * k + R::VEC - 1) / R::VEC;
  while ((long long)g_part * g_part * R::VEC < (long long)rd.n_groups * k) g_part *= 2;
  if (g_part > rd.n_groups) g_part = rd.n_groups;
  constexpr uint32_t kPastLargest = DT == 0 ? 0x8000u : 0x80000000u;
  histogram_pass<DT, VECTOR>(sh, ring, rd, 0, g_part, 0u, kPastLargest, SHIFT0, kBins - 1);
  __syncthreads();
  if (g_part < rd.n_groups) {
    find_bin_from_top(sh, kBins, (uint32_t)k, 0);
    const uint32_t floor_key = sh.picked_bin << SHIFT0;
    histogram_pass<DT, VECTOR>(sh, ring, rd, g_part, rd.n_groups, floor_key, kPastLargest, SHIFT0, kBins - 1);
    __syncthreads();
  }
  find_bin_from_top(sh, kBins, (uint32_t)k, 1);
  uint32_t prefix = sh.picked_bin << SHIFT0;
  uint32_t remaining = sh.picked_remaining;
  // fp32: the 16 bits below the first digit, 8 at a time
  int slot = 0;
  for (int shift = SHIFT0 - 8; shift >= 0; shift -= 8) {
    __syncthreads();
    clear_bins(sh, 256);
    // the keys that start with the digits found so far: prefix .. prefix + 2^(shift + 8) - 1
    histogram_pass<DT, VECTOR>(sh, ring, rd, 0, rd.n_groups, prefix, prefix + (1u << (shift + 8)), shift, 255u);
    __syncthreads();
    find_bin_from_top(sh, 256, remaining, slot);
    slot ^= 1;
    prefix |= sh.picked_bin << shift;
    remaining = sh.picked_remaining;
  }
  *kth = prefix;
  *take = remaining;
  __syncthreads();
}
static_assert((key_bits(1) - kTopBits) % 8 == 0 && key_bits(0) == kTopBits, "digits cover the key exactly");

// Visits the chunk's top-k in ascending index order: emit(position, flat index, pattern).
template <int DT, bool VECTOR, class Emit>
__device__ void collect_in_index_order(DirectShared& sh, uint4* ring, const Reader<DT, VECTOR>& rd, int k, uint32_t kth,
                                       uint32_t take, Emit emit) {
  using R = Reader<DT, VECTOR>;
  const uint32_t n_above = (uint32_t)k - take;
  uint32_t base_above = 0, base_equal = 0;
  int slot = 0;
  rd.request(ring, (int)threadIdx.x, rd.n_groups);
  for (int t0 = 0; t0 < rd.n_groups; t0 += kUnroll * kThreads) {
    uint32_t w[kUnroll][4];
    unsigned long long above = 0, equal = 0;  // 16 bits per sub-tile
    rd.take(ring, t0 + (int)threadIdx.x, rd.n_groups, w);
    if (t0 + kUnroll * kThreads < rd.n_groups)
      rd.request_after(ring, t0 + kUnroll * kThreads + (int)threadIdx.x, rd.n_groups, w, t0 + (int)threadIdx.x,
                       rd.n_groups);
    uint32_t reach[kUnroll];  // per sub-tile: elements >= kth in bits 0..7, elements > kth in bits 8..15
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int g = t0 + u * kThreads + (int)threadIdx.x;
      reach[u] = 0;
      if (g < rd.n_groups) {
        const uint32_t ge = R::reach_mask(w[u], kth), gt = R::reach_mask(w[u], kth + 1u);
        reach[u] = ge | (gt << 8);
        const uint32_t a = (uint32_t)__popc(gt);
        above |= (unsigned long long)a << (16 * u);
        equal |= (unsigned long long)((uint32_t)__popc(ge) - a) << (16 * u);
      }
    }
    unsigned long long total_above, total_equal;
    const unsigned long long ex_above = block_scan_exclusive(sh, above, slot, &total_above);
    const unsigned long long ex_equal = block_scan_exclusive(sh, equal, slot ^ 1, &total_equal);
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int g = t0 + u * kThreads + (int)threadIdx.x;
      uint32_t above_before = base_above + (uint32_t)((ex_above >> (16 * u)) & 0xFFFFu);
      uint32_t equal_before = base_equal + (uint32_t)((ex_equal >> (16 * u)) & 0xFFFFu);
      uint32_t m = reach[u] & 0xFFu;
      while (m) {  // in index order
        const uint32_t j = (uint32_t)__ffs((int)m) - 1u;
        m &= m - 1u;
        const uint32_t pat = R::pattern_at(w[u], j);
        if ((reach[u] >> (8 + j)) & 1u) {
          emit(above_before + (equal_before < take ? equal_before : take), (uint32_t)g * R::VEC + j, R::committed(pat));
          ++above_before;
        } else {
          if (equal_before < take) emit(above_before + equal_before, (uint32_t)g * R::VEC + j, R::committed(pat));
          ++equal_before;
        }
      }
      base_above += (uint32_t)((total_above >> (16 * u)) & 0xFFFFu);
      base_equal += (uint32_t)((total_equal >> (16 * u)) & 0xFFFFu);
    }
    if (base_above == n_above && base_equal >= take) break;  // the same for every thread
  }
  if (VECTOR) asm volatile("cp.async.wait_group 0;" ::: "memory");  // a batch requested before the break
}

// One-pass selection for vector layouts.  The chunk is streamed once, in batches of
// kUnroll * kThreads vectors; every element whose key reaches the running threshold is kept as a
// candidate (flat index, pattern), in index order (a block-wide prefix sum per batch places
// them), and counted in a histogram of its upper 11 key bits.  Whenever enough candidates have
// arrived, the threshold is raised to the lowest key of the bin that holds the k-th largest
// candidate so far -- a lower bound of the chunk's k-th largest key, so nothing of the top-k is
// ever dropped.  The first batch (about 4k elements, threshold 0) seeds the histogram.  At the
// end the exact k-th key is found among the candidates (the histogram, then the bits below) and the
// top-k leaves in index order, ties to the lower index.  Returns false, having emitted nothing,
// when the candidates outgrow their buffer (data sorted upwards, say): the caller then takes
// the two-pass selection.
template <int DT> struct StoredPattern { typedef uint16_t type; };
template <> struct StoredPattern<1> { typedef uint32_t type; };

template <int DT, class Emit>
__device__ bool select_in_one_pass(DirectShared& sh, uint4* ring, const Reader<DT, true>& rd, int k, Emit emit) {
  using R = Reader<DT, true>;
  using Pat = typename StoredPattern<DT>::type;
  constexpr int kCandCap = cand_cap(DT);
  constexpr int kCoarseShift = key_bits(DT) - 11;
  uint32_t* coarse = sh.hist;
  uint32_t* cand_flat = sh.hist + kCoarseBins;
  Pat* cand_pat = reinterpret_cast<Pat*>(cand_flat + kCandCap);
  clear_bins(sh, kCoarseBins);
  int seed_groups = (4 * k > 2048 ? 4 * k : 2048) / R::VEC;
  if (seed_groups > rd.n_groups) seed_groups = rd.n_groups;
  const uint32_t raise_step = (uint32_t)(k / 2 > 64 ? k / 2 : 64);
  uint32_t thr = 0, count = 0, last_raise = 0;
  int begin = 0, end = seed_groups, slot = 0;
  bool overflow = false;
  rd.request(ring, (int)threadIdx.x, end);
  while (begin < rd.n_groups) {
    uint32_t w[kUnroll][4];
    rd.take(ring, begin + (int)threadIdx.x, end, w);
    const int next_begin = end;
    int next_end = next_begin + kUnroll * kThreads;
    if (next_end > rd.n_groups) next_end = rd.n_groups;
    if (next_begin < rd.n_groups)
      rd.request_after(ring, next_begin + (int)threadIdx.x, next_end, w, begin + (int)threadIdx.x, end);
    uint32_t reach[kUnroll];
    unsigned long long hits = 0;  // 16 bits per sub-tile
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int g = begin + u * kThreads + (int)threadIdx.x;
      reach[u] = g < end ? R::reach_mask(w[u], thr) : 0u;
      hits |= (unsigned long long)__popc(reach[u]) << (16 * u);
    }
    unsigned long long total;
    const unsigned long long before = block_scan_exclusive(sh, hits, slot, &total);
    slot ^= 1;
    uint32_t batch_total = 0;
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) batch_total += (uint32_t)((total >> (16 * u)) & 0xFFFFu);
    if (count + batch_total > (uint32_t)kCandCap) {  // the same for every thread
      overflow = true;
      break;
    }
    uint32_t tile_base = count;
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int g = begin + u * kThreads + (int)threadIdx.x;
      uint32_t at = tile_base + (uint32_t)((before >> (16 * u)) & 0xFFFFu);
      uint32_t m = reach[u];
      while (m) {  // in index order
        const uint32_t j = (uint32_t)__ffs((int)m) - 1u;
        m &= m - 1u;
        const uint32_t pat = R::pattern_at(w[u], j);
        cand_flat[at] = (uint32_t)g * R::VEC + j;
        cand_pat[at] = (Pat)pat;
        atomicAdd(&coarse[R::key(pat) >> kCoarseShift], 1u);
        ++at;
      }
      tile_base += (uint32_t)((total >> (16 * u)) & 0xFFFFu);
    }
    count += batch_total;
    if (count - last_raise >= raise_step && next_begin < rd.n_groups) {  // the same for every thread
      __syncthreads();  // this batch's counts are in
      find_bin_from_top(sh, kCoarseBins, (uint32_t)k, slot);
      slot ^= 1;
      const uint32_t floor_key = sh.picked_bin << kCoarseShift;
      if (floor_key > thr) thr = floor_key;
      last_raise = count;
    }
    begin = next_begin;
    end = next_end;
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");  // a batch requested before leaving the loop
  __syncthreads();
  if (overflow) return false;

  // The exact k-th key among the candidates: its upper 11 bits from the histogram that the
  // stream kept (it counts every candidate), the bits below 8 at a time (the last digit has 4).
  find_bin_from_top(sh, kCoarseBins, (uint32_t)k, 0);
  uint32_t kth = sh.picked_bin << kCoarseShift, known = (uint32_t)(kCoarseBins - 1) << kCoarseShift;
  uint32_t take = sh.picked_remaining;
  __syncthreads();
  for (int shift = kCoarseShift - 8, round = 1; shift > -8; shift -= 8, ++round) {
    const int low = shift < 0 ? 0 : shift, width = shift < 0 ? 8 + shift : 8;
    clear_bins(sh, 256);
    for (uint32_t i = threadIdx.x; i < count; i += kThreads) {
      const uint32_t key = R::key(cand_pat[i]);
      if ((key & known) == kth) atomicAdd(&sh.hist[(key >> low) & ((1u << width) - 1u)], 1u);
    }
    __syncthreads();
    find_bin_from_top(sh, 1 << width, take, round & 1);
    kth |= sh.picked_bin << low;
    known |= ((1u << width) - 1u) << low;
    take = sh.picked_remaining;
    __syncthreads();
  }

  // the top-k in index order: every thread takes a run of consecutive candidates
  const uint32_t per = ((count + kThreads - 1) / kThreads) | 1u;  // odd: the runs start in different banks
  const uint32_t lo = threadIdx.x * per < count ? threadIdx.x * per : count;
  const uint32_t hi = lo + per < count ? lo + per : count;
  uint32_t above = 0, equal = 0;
  for (uint32_t i = lo; i < hi; ++i) {
    const uint32_t key = R::key(cand_pat[i]);
    above += key > kth;
    equal += key == kth;
  }
  unsigned long long total;
  const unsigned long long before = block_scan_exclusive(sh, above | ((unsigned long long)equal << 32), 0, &total);
  uint32_t above_before = (uint32_t)before, equal_before = (uint32_t)(before >> 32);
  for (uint32_t i = lo; i < hi; ++i) {
    const uint32_t pat = cand_pat[i], key = R::key(pat);
    if (key > kth) {
      emit(above_before + (equal_before < take ? equal_before : take), cand_flat[i], R::committed(pat));
      ++above_before;
    } else if (key == kth) {
      if (equal_before < take) emit(above_before + equal_before, cand_flat[i], R::committed(pat));
      ++equal_before;
    }
  }
  __syncthreads();
  return true;
}


// select_unordered: selection without a barrier in its streaming loops (vector layouts).
// A first pass streams the chunk and counts every vector's largest key in a histogram of the
// upper 11 key bits: the k-th largest of these maxima is reached by at least k elements, so it
// is a sound threshold, and by few more than k, so the candidates fit a small buffer.  Then
// the elements that reach the threshold are collected, in no particular order:
//   MAP (two 512-thread blocks per SM): the first pass also left one byte per 8 elements -- the
//   11 bits of the group's largest key, counted from 2^-20 -- and the collection is a scan of
//   those bytes that parks the groups which reach the threshold's byte and fetches only them:
//   the chunk is streamed once;
//   otherwise (1024-thread block): a second streaming pass (from L2) tests every vector as a
//   whole and parks those that pass; while it runs the threshold can still rise -- whenever
//   enough new candidates have arrived, one warp (whoever gets the lock) walks the histogram of
//   the candidates' upper 11 key bits to the bin that holds the k-th largest so far and
//   publishes that bin's lowest key; at least k candidates reach it, so nothing below it can
//   belong to the top-k, whatever the other warps add meanwhile (the counts only grow).
// Parked groups are unpacked by a whole warp, 32 at a time, into the block's candidate buffer
// (slots handed out by one atomic per round).  The exact k-th key, the ties that belong to the
// top-k (lowest flat indices) and the position of every selected element in index order are
// settled at the end.  ORDERED: positions in ascending index order, by ranking the selected
// indices in a bitmap of the chunk; otherwise positions are handed out as they come.
// Returns false, having emitted nothing, when the candidates outgrow their buffer.
// Where select_unordered keeps its state; the two kernels that use it
// (a 1024-thread block per SM, or two 512-thread blocks) carve it from their shared memory.
template <int DT>
struct LooseWorkspace {
  LooseControl* ctl;
  uint32_t* coarse;      // kCoarseBins words: the histogram; later digit histograms, the tie list, per-thread prefixes
  uint32_t* cand_flat;   // cap candidates: flat index ...
  typename StoredPattern<DT>::type* cand_pat;  // ... and whole pattern
  uint32_t* park;        // kParkCap words per warp
  int cap;
  uint8_t* seen_max;     // MAP only: one byte per 8 elements (their largest key, coarsely), written by the first pass
  uint4* second_stage;   // MAP only: kUnroll * T more 16-byte slots that are idle during the first pass
  uint32_t* bitmap;      // ORDERED only: one bit per element for the ranking in index order
};

// The byte the first pass leaves for every 8 consecutive elements: the upper 11 bits of their
// largest key (exponent and three mantissa bits) counted from 2^-20, 0 for anything smaller, 255
// for 2^11.75 and above -- 32 binades around the magnitudes activations have.  A group whose byte
// reaches the threshold's byte may hold an element that reaches the threshold; a group below it
// cannot (magnitudes beyond either end of the window only make the second pass look at groups
// it need not have looked at).
constexpr uint32_t kSeenBase = (127u - 20u) << 3;
__device__ __forceinline__ uint32_t seen_byte(uint32_t bin11) {
  return bin11 < kSeenBase ? 0u : (bin11 - kSeenBase + 1u < 255u ? bin11 - kSeenBase + 1u : 255u);
}

template <int T>
__device__ __forceinline__ void clear_words(uint32_t* words, int n) {  // n: a multiple of 4; ends with a barrier
  uint4* q = reinterpret_cast<uint4*>(words);
  for (int b = threadIdx.x; b < n / 4; b += T) q[b] = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
}

// Exclusive prefix sum over a block of T threads (T / 32 <= 32 warps) of a 64-bit value; *total
// receives the block's sum.  `slot` alternates between calls so that one barrier per call is enough.
template <int T>
__device__ __forceinline__ unsigned long long scan_exclusive(LooseControl& sh, unsigned long long v, int slot,
                                                             unsigned long long* total) {
  constexpr int kW = T / 32;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned long long inc = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const unsigned long long o = __shfl_up_sync(0xFFFFFFFFu, inc, d);
    if (lane >= d) inc += o;
  }
  if (lane == 31) sh.warp_sums[slot][warp] = inc;
  __syncthreads();
  unsigned long long mine = lane < kW ? sh.warp_sums[slot][lane] : 0ull;
  unsigned long long winc = mine;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const unsigned long long o = __shfl_up_sync(0xFFFFFFFFu, winc, d);
    if (lane >= d) winc += o;
  }
  *total = __shfl_sync(0xFFFFFFFFu, winc, 31);
  const unsigned long long before_warp = __shfl_sync(0xFFFFFFFFu, winc - mine, warp);
  return before_warp + inc - v;
}

// The bin of hist[0 .. nbins), counted from the top, in which the want-th largest counted element
// lies (1 <= want <= number counted): sh.picked_bin, and sh.picked_remaining = want minus the
// elements in higher bins.  All T threads call; ends with a barrier.
template <int T>
__device__ __forceinline__ void find_from_top(LooseControl& sh, const uint32_t* hist, int nbins, uint32_t want, int slot) {
  const int per = nbins >= T ? nbins / T : 1;  // nbins and T are powers of two
  const int top = nbins - 1 - (int)threadIdx.x * per;  // this thread owns bins top, top-1, ..., top-per+1
  uint32_t s = 0;
  if (top >= 0)  // each lane starts at another offset: its bins are `per` words apart from its neighbour's
    for (int b = 0; b < per; ++b) s += hist[top - ((b + (int)threadIdx.x) & (per - 1))];
  unsigned long long total;
  const uint32_t before = (uint32_t)scan_exclusive<T>(sh, s, slot, &total);
  if (top >= 0 && before < want && want <= before + s) {
    uint32_t c = before;
    for (int b = 0; b < per; ++b) {
      const uint32_t h = hist[top - b];
      if (c + h >= want) {
        sh.picked_bin = (uint32_t)(top - b);
        sh.picked_remaining = want - c;
        break;
      }
      c += h;
    }
  }
  __syncthreads();
}

// The commitment of one chunk from its k (index, committed value) pairs in index order, held in
// shared memory: 6 bytes per pair (index low half, index high half, value).  Whole 16-byte words
// where the record's place and k allow it, coalesced 2-byte words otherwise.
template <int T>
__device__ __forceinline__ void write_commitment(uint16_t* rec, const uint32_t* flat, const uint16_t* pat, int k) {
  if ((k & 7) == 0 && (reinterpret_cast<uintptr_t>(rec) & 15u) == 0) {
    uint4* out = reinterpret_cast<uint4*>(rec);
    for (int g = threadIdx.x; g < k / 8; g += T) {
      uint32_t h[12];  // 24 half words: 8 records
#pragma unroll
      for (int r = 0; r < 8; r += 2) {
        const uint32_t f0 = flat[8 * g + r], f1 = flat[8 * g + r + 1];
        const uint32_t p0 = pat[8 * g + r], p1 = pat[8 * g + r + 1];
        h[3 * (r / 2)] = f0;                                   // low, high of the first index
        h[3 * (r / 2) + 1] = p0 | (f1 << 16);                  // its value, low half of the second
        h[3 * (r / 2) + 2] = (f1 >> 16) | (p1 << 16);          // high half of the second, its value
      }
      out[3 * g] = make_uint4(h[0], h[1], h[2], h[3]);
      out[3 * g + 1] = make_uint4(h[4], h[5], h[6], h[7]);
      out[3 * g + 2] = make_uint4(h[8], h[9], h[10], h[11]);
    }
  } else {
    for (int w = threadIdx.x; w < 3 * k; w += T) {
      const int r = w / 3, part = w - 3 * r;
      rec[w] = part == 2 ? pat[r] : (uint16_t)(part == 0 ? flat[r] & 0xFFFFu : flat[r] >> 16);
    }
  }
}

template <int DT, bool ORDERED, int T, bool MAP, bool TWO, class Emit>
__device__ bool select_unordered(const LooseWorkspace<DT>& ws, uint4* ring, const Reader<DT, true>& rd, int k, Emit emit,
                                 uint16_t* rec = nullptr) {
  using R = Reader<DT, true>;
  using Pat = typename StoredPattern<DT>::type;
  constexpr int VEC = R::VEC;
  constexpr int kCoarseShift = key_bits(DT) - 11;
  constexpr uint32_t kFull = 0xFFFFFFFFu;
  constexpr int kBatch = kUnroll * T;
  // every pointer of the workspace is shared memory: said once, so that loads, stores and atomics
  // through them compile to shared-memory instructions instead of generic ones
  __builtin_assume(__isShared(ws.ctl));
  __builtin_assume(__isShared(ws.coarse));
  __builtin_assume(__isShared(ws.cand_flat));
  __builtin_assume(__isShared(ws.cand_pat));
  __builtin_assume(__isShared(ws.park));
  __builtin_assume(__isShared(ws.bitmap));
  __builtin_assume(__isShared(ring));
  if (MAP) {
    __builtin_assume(__isShared(ws.seen_max));
    __builtin_assume(__isShared(ws.second_stage));
  }
  LooseControl& sh = *ws.ctl;
  const int kCap = ws.cap;
  uint32_t* coarse = ws.coarse;
  uint32_t* cand_flat = ws.cand_flat;
  Pat* cand_pat = ws.cand_pat;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t* park = ws.park + warp * kParkCap;
  volatile uint32_t* shared_thr = &sh.thr;
  volatile uint32_t* shared_overflow = &sh.overflow;
  volatile uint32_t* shared_last_raise = &sh.last_raise;
  if (threadIdx.x == 0) {
    sh.cand_count = 0;
    sh.thr = 0;
    sh.last_raise = 0;
    sh.raise_lock = 0;
    sh.overflow = 0;
    sh.emitted = 0;
  }
  clear_words<T>(coarse, kCoarseBins);  // ends with a barrier

  // One vector per lane: its elements that reach thr become candidates.  Returns the number of
  // candidates handed out so far (0 if the round added none).
  // MAP: the threshold no longer moves once candidates arrive, so they are counted by their
  // distance above it in steps of one 15-bit key (the last bin takes everything further up):
  // the candidates spread over hundreds of bins instead of a few, and the k-th key's upper 15 bits
  // come out of one walk.
  constexpr int kFineShift = key_bits(DT) - 15;
  // A parked entry is a vector, or (MAP) 8 elements: one or two vectors.  A round of unpacking
  // takes one entry per lane, or (TWO) two where an entry is one vector: one prefix sum and one
  // atomic for twice the entries, which is worth 7 % of the call at k = 4096; at k = 1024 the
  // rounds fill too slowly and it costs 2 %, so the caller asks for it from k = 2048 on.
  constexpr int kVecs = MAP ? 8 / VEC : 1;                       // vectors per parked entry
  constexpr int kEntriesPerLane = kVecs == 2 ? 1 : (TWO ? 2 : 1);  // entries a lane takes per round
  constexpr int kLaneVecs = kVecs * kEntriesPerLane;              // 1 or 2
  constexpr int kRound = 32 * kEntriesPerLane;
  auto fetch = [&](bool valid, uint32_t g) -> uint4 {
    return valid ? toploc_device::load_streaming(reinterpret_cast<const uint4*>(rd.address((int)g)))
                 : make_uint4(0u, 0u, 0u, 0u);
  };
  // Two vectors per lane: their elements that reach thr become candidates (one prefix sum and one
  // atomic for both).  Returns the number of candidates handed out so far (0 if the round added none).
  auto admit = [&](bool valid_a, uint32_t g_a, const uint4& w_a, bool valid_b, uint32_t g_b, const uint4& w_b,
                   uint32_t thr) -> uint32_t {
    uint32_t mask = valid_a ? toploc_device::passing_mask<DT, VEC>(w_a, thr) : 0u;
    if (kLaneVecs == 2) mask |= (valid_b ? toploc_device::passing_mask<DT, VEC>(w_b, thr) : 0u) << VEC;
    const int mine = __popc(mask);
    int incl = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int other = __shfl_up_sync(kFull, incl, off);
      if (lane >= off) incl += other;
    }
    const int total = __shfl_sync(kFull, incl, 31);
    if (total == 0) return 0u;
    uint32_t base = 0;
    if (lane == 0) base = atomicAdd(&sh.cand_count, (uint32_t)total);
    base = __shfl_sync(kFull, base, 0);
    if (base + (uint32_t)total > (uint32_t)kCap) {
      if (lane == 0) *shared_overflow = 1u;
      return base + (uint32_t)total;
    }
    uint32_t at = base + (uint32_t)(incl - mine);
    while (mask) {
      const uint32_t bit = (uint32_t)__ffs((int)mask) - 1u;
      mask &= mask - 1u;
      const bool second = kLaneVecs == 2 && bit >= (uint32_t)VEC;
      const uint32_t e = second ? bit - (uint32_t)VEC : bit;
      const uint4 w = second ? w_b : w_a;
      uint32_t key, sign;
      toploc_device::pick_element<DT, VEC>(w, e, &key, &sign);
      cand_flat[at] = (second ? g_b : g_a) * VEC + e;
      cand_pat[at] = (Pat)((sign << (DT == 0 ? 15 : 31)) | key);
      if (MAP) {
        const uint32_t above = (key - thr) >> kFineShift;
        atomicAdd(&coarse[above < (uint32_t)kCoarseBins - 1u ? above : (uint32_t)kCoarseBins - 1u], 1u);
      } else {
        atomicAdd(&coarse[key >> kCoarseShift], 1u);
      }
      ++at;
    }
    return base + (uint32_t)total;
  };

  // A sound and tight threshold before anything is collected: a first pass streams the whole chunk
  // and counts every vector's largest key in the histogram; the k-th largest of these maxima is
  // reached by at least k elements (each maximum is a different element), so the chunk's k-th key
  // cannot lie below it, and by little more than k (k vectors reach it, few of them twice).  The
  // second pass finds the chunk in L2 (one chunk per SM in flight).  A chunk of fewer than k
  // vectors starts from 0 and is streamed once.
  // MAP: the first pass also leaves seen_max, and the second pass is a scan of those bytes that
  // fetches only the groups which can hold a candidate (about k of them, from L2) -- the chunk is
  // streamed once, and the candidates may use the ring's place.
  constexpr int kPerByte = 8 / VEC;  // vectors per byte of seen_max
  if (!MAP || rd.n_groups >= k) {
    const int first_end = kBatch < rd.n_groups ? kBatch : rd.n_groups;
    rd.template request<T>(ring, (int)threadIdx.x, first_end);  // in flight meanwhile
  }
  if (rd.n_groups >= k) {
    int begin = 0;
    // One whole batch of a gap-free chunk in the first pass: its histogram entries and (MAP) bytes.
    // (shared-memory addresses taken once: the histogram and the bytes are reached through pointers
    // in a struct, and plain shared-memory instructions are cheaper than generic ones)
    const uint32_t coarse_at = (uint32_t)__cvta_generic_to_shared(coarse);
    const uint32_t seen_at = MAP ? (uint32_t)__cvta_generic_to_shared(ws.seen_max) : 0u;
    auto count_whole_batch = [&](int first, const uint4 (&v)[kUnroll]) {
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int g = first + u * T + (int)threadIdx.x;
        uint32_t bin = toploc_device::vector_max_coarse_key<DT, VEC>(v[u]) >> 4;  // upper 11 of the 15 bits
        asm volatile("red.shared.add.u32 [%0], 1;" ::"r"(coarse_at + 4u * bin) : "memory");
        if (MAP) {
          if (kPerByte == 2) {
            const uint32_t other = __shfl_xor_sync(kFull, bin, 1);
            bin = bin > other ? bin : other;
          }
          if (kPerByte == 1 || (g & 1) == 0)
            asm volatile("st.shared.u8 [%0], %1;" ::"r"(seen_at + (uint32_t)(g / kPerByte)), "r"(seen_byte(bin)) : "memory");
        }
      }
    };
    if (MAP && rd.flat && rd.n_groups >= 2 * kBatch) {
      // Rows without gaps, and room for a second batch in flight: the memory behind the ring is
      // idle until candidates arrive (ws.second_stage), so two batches are on their way while one
      // is counted -- a block that streams while its neighbour on the SM is busy with a chunk's
      // later phases then draws more than one ring's worth of bandwidth.  Whole batches only: no
      // bounds, plain pointer steps; a ragged last batch is left to the loop below.
      const int n_whole = rd.n_groups / kBatch;
      const char* mine = rd.base + (size_t)threadIdx.x * 16u;
      const uint4* stage0 = ring + threadIdx.x;
      const uint4* stage1 = ws.second_stage + threadIdx.x;
      const uint32_t slot0 = (uint32_t)__cvta_generic_to_shared(stage0), slot1 = (uint32_t)__cvta_generic_to_shared(stage1);
      // batch 0 is on its way to the ring already; batch 1 goes to the second stage
#pragma unroll
      for (int u = 0; u < kUnroll; ++u)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(slot1 + (uint32_t)(u * T * 16)),
                     "l"(mine + ((size_t)kBatch + (size_t)u * T) * 16u)
                     : "memory");
      asm volatile("cp.async.commit_group;" ::: "memory");
      for (int b = 0; b < n_whole; ++b) {
        // groups complete in order: all but the latest one have landed, batch b among them
        if (b + 1 < n_whole) asm volatile("cp.async.wait_group 1;" ::: "memory");
        else asm volatile("cp.async.wait_group 0;" ::: "memory");
        const uint4* stage = (b & 1) ? stage1 : stage0;
        const uint32_t slot = (b & 1) ? slot1 : slot0;
        uint4 v[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) v[u] = stage[u * T];
        if (b + 2 < n_whole) {
          const char* next = mine + (size_t)(b + 2) * kBatch * 16u;
#pragma unroll
          for (int u = 0; u < kUnroll; ++u) {  // (each copy's destination depends on the register read from it)
            uint32_t zero;
            asm volatile("and.b32 %0, %1, 0;" : "=r"(zero) : "r"(v[u].w));
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(slot + (uint32_t)(u * T * 16) + zero),
                         "l"(next + (size_t)u * T * 16u)
                         : "memory");
          }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");  // (an empty group keeps the count in step)
        count_whole_batch(b * kBatch, v);
      }
      begin = n_whole * kBatch;
      if (begin < rd.n_groups) rd.template request<T>(ring, begin + (int)threadIdx.x, rd.n_groups);  // the ragged rest
    } else if (rd.flat) {
      // Rows without gaps: while this batch and the next are whole, nothing needs a bound and a
      // thread's vectors lie kBatch * 16 bytes apart from batch to batch.
      const char* mine = rd.base + (size_t)threadIdx.x * 16u;
      const uint32_t slot = (uint32_t)__cvta_generic_to_shared(ring + threadIdx.x);
      for (; begin + 2 * kBatch <= rd.n_groups; begin += kBatch) {
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        uint4 v[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) v[u] = ring[u * T + threadIdx.x];
        const char* next = mine + (size_t)(begin + kBatch) * 16u;
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {  // (each copy's destination depends on the register read from it)
          uint32_t zero;
          asm volatile("and.b32 %0, %1, 0;" : "=r"(zero) : "r"(v[u].w));
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(slot + (uint32_t)(u * T * 16) + zero),
                       "l"(next + (size_t)u * T * 16u)
                       : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        count_whole_batch(begin, v);
      }
    }
    for (; begin < rd.n_groups; begin += kBatch) {
      const int end = begin + kBatch < rd.n_groups ? begin + kBatch : rd.n_groups;
      uint32_t w[kUnroll][4];
      rd.template take<T>(ring, begin + (int)threadIdx.x, end, w);
      if (end < rd.n_groups) {
        const int next_end = end + kBatch < rd.n_groups ? end + kBatch : rd.n_groups;
        rd.template request_after<T>(ring, end + (int)threadIdx.x, next_end, w, begin + (int)threadIdx.x, end);
      }
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int g = begin + u * T + (int)threadIdx.x;
        uint32_t bin = 0;
        if (g < end) {
          const uint32_t m = toploc_device::vector_max_coarse_key<DT, VEC>(make_uint4(w[u][0], w[u][1], w[u][2], w[u][3]));
          bin = m >> 4;  // upper 11 of the 15 bits
          atomicAdd(&coarse[bin], 1u);
        }
        if (MAP) {
          if (kPerByte == 2) {  // neighbouring lanes hold the two vectors of a byte (begin and T are even)
            const uint32_t other = __shfl_xor_sync(kFull, bin, 1);
            bin = bin > other ? bin : other;
          }
          if (g < end && (kPerByte == 1 || (g & 1) == 0)) ws.seen_max[g / kPerByte] = (uint8_t)seen_byte(bin);
        }
      }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    if (!MAP) {
      const int first_end = kBatch < rd.n_groups ? kBatch : rd.n_groups;
      rd.template request<T>(ring, (int)threadIdx.x, first_end);  // the second pass's first batch
    }
    __syncthreads();
    find_from_top<T>(sh, coarse, kCoarseBins, (uint32_t)k, 1);
    const uint32_t first = sh.picked_bin << kCoarseShift;
    __syncthreads();
    if (threadIdx.x == 0) sh.thr = first;
    clear_words<T>(coarse, kCoarseBins);
  }

  const uint32_t raise_step = (uint32_t)(k / 2 > 256 ? k / 2 : 256);
  uint32_t thr = *shared_thr;
  int nparked = 0;
  // Unpacks the parked vectors a full round (32 of them) at a time; what is left over waits for
  // the next drain unless this is the last one.
  static_assert(kRound <= kParkTrigger && kParkCap >= kParkTrigger - 1 + kUnroll * 32, "parking space");
  auto drain = [&](bool all) {
    __syncwarp();
    uint32_t handed_out = 0;
    const int upto = all ? nparked : nparked / kRound * kRound;
    // the next round's vectors are requested before this round's are unpacked
    uint4 cur[kLaneVecs], nxt[kLaneVecs];
    uint32_t g_cur[kLaneVecs], g_nxt[kLaneVecs];
    bool ok_cur[kLaneVecs], ok_nxt[kLaneVecs];
    auto fetch_round = [&](int b, uint32_t (&g)[kLaneVecs], uint4 (&w)[kLaneVecs], bool (&ok)[kLaneVecs]) {
#pragma unroll
      for (int i = 0; i < kEntriesPerLane; ++i) {
        const int at = b + i * 32 + lane;
        const bool valid = at < upto;
        const uint32_t entry = valid ? park[at] : 0u;
#pragma unroll
        for (int h = 0; h < kVecs; ++h) {
          const int s = i * kVecs + h;
          g[s] = entry * kVecs + h;
          ok[s] = valid && g[s] < (uint32_t)rd.n_groups;
          w[s] = fetch(ok[s], g[s]);
        }
      }
    };
    fetch_round(0, g_cur, cur, ok_cur);
    for (int b = 0; b < upto; b += kRound) {
      fetch_round(b + kRound, g_nxt, nxt, ok_nxt);
      constexpr int kLast = kLaneVecs - 1;  // (one vector per lane: the second operand is never looked at)
      const uint32_t after = admit(ok_cur[0], g_cur[0], cur[0], kLaneVecs == 2 && ok_cur[kLast], g_cur[kLast], cur[kLast], thr);
      handed_out = after > handed_out ? after : handed_out;
#pragma unroll
      for (int s = 0; s < kLaneVecs; ++s) {
        cur[s] = nxt[s];
        ok_cur[s] = ok_nxt[s];
        g_cur[s] = g_nxt[s];
      }
    }
    const int left = all ? 0 : nparked - upto;  // < kRound
    uint32_t moved[kEntriesPerLane];
#pragma unroll
    for (int i = 0; i < kEntriesPerLane; ++i) moved[i] = i * 32 + lane < left ? park[upto + i * 32 + lane] : 0u;
    __syncwarp();
#pragma unroll
    for (int i = 0; i < kEntriesPerLane; ++i)
      if (i * 32 + lane < left) park[i * 32 + lane] = moved[i];
    nparked = left;
    __syncwarp();
    // raise the threshold if enough candidates have arrived since the last time and nobody else is at it
    uint32_t go = 0;
    if (!MAP && lane == 0 && handed_out >= (uint32_t)k && handed_out <= (uint32_t)kCap &&
        handed_out - *shared_last_raise >= raise_step)
      go = atomicCAS(&sh.raise_lock, 0u, 1u) == 0u ? 1u : 0u;
    go = __shfl_sync(kFull, go, 0);
    if (go) {
      // lane l owns bins top, top - 1, ..., top - 63 (lane 0 the highest keys)
      constexpr int kPerLane = kCoarseBins / 32;
      const int top = kCoarseBins - 1 - lane * kPerLane;
      volatile uint32_t* bins = coarse;
      uint32_t sum = 0;
      for (int b = 0; b < kPerLane; ++b) sum += bins[top - ((b + lane) & (kPerLane - 1))];
      uint32_t upto = sum;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const uint32_t other = __shfl_up_sync(kFull, upto, off);
        if (lane >= off) upto += other;
      }
      const uint32_t before = upto - sum;
      if (before < (uint32_t)k && (uint32_t)k <= upto) {
        uint32_t c = before;
        for (int b = 0; b < kPerLane; ++b) {
          c += bins[top - b];
          if (c >= (uint32_t)k) {  // (counts read a second time are no smaller than the first time)
            atomicMax(&sh.thr, (uint32_t)(top - b) << kCoarseShift);
            break;
          }
        }
      }
      if (lane == 0) *shared_last_raise = handed_out;
      __syncwarp();
      if (lane == 0) {
        __threadfence_block();
        atomicExch(&sh.raise_lock, 0u);
      }
    }
  };

  if (MAP) {
    // The threshold is a bin's lowest key (or 0 for a chunk of fewer than k vectors, whose bytes
    // were never written: every byte reaches 0).
    const uint32_t bin = thr >> kCoarseShift;
    const uint32_t want = seen_byte(bin) * 0x01010101u;
    const int n_bytes = (rd.n_groups + kPerByte - 1) / kPerByte;
    const uint4* quads = reinterpret_cast<const uint4*>(ws.seen_max);  // (its place is a whole number of 16-byte words)
    // Sixteen bytes per lane and step.  The bytes that reach the threshold's are counted per lane,
    // one prefix sum over the lanes hands out the places, and every lane parks its own few.
    // A step that would not fit the parking space (dense data, or the threshold 0) is taken a word
    // (four bytes per lane) at a time with drains in between.
    auto exclusive = [&](int mine, int* total) {
      int incl = mine;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int other = __shfl_up_sync(kFull, incl, off);
        if (lane >= off) incl += other;
      }
      *total = __shfl_sync(kFull, incl, 31);
      return incl - mine;
    };
    auto park_word = [&](uint32_t bits, int first_index, int at) {  // bits: bit 0 of byte j set = entry first_index + j
      while (bits) {
        const int j = (__ffs((int)bits) - 1) >> 3;
        bits &= bits - 1u;
        park[at++] = (uint32_t)(first_index + j);
      }
      return at;
    };
    for (int q0 = 0; q0 * 16 < n_bytes; q0 += T) {
      const int qi = q0 + (int)threadIdx.x;
      uint32_t reach[4] = {0u, 0u, 0u, 0u};
      if (qi * 16 < n_bytes) {
        const uint4 b = quads[qi];
        reach[0] = __vcmpgeu4(b.x, want) & 0x01010101u;
        reach[1] = __vcmpgeu4(b.y, want) & 0x01010101u;
        reach[2] = __vcmpgeu4(b.z, want) & 0x01010101u;
        reach[3] = __vcmpgeu4(b.w, want) & 0x01010101u;
        if (qi * 16 + 16 > n_bytes) {  // the last, partial quad: entries beyond the chunk do not count
#pragma unroll
          for (int wd = 0; wd < 4; ++wd)
#pragma unroll
            for (int j = 0; j < 4; ++j)
              if (qi * 16 + wd * 4 + j >= n_bytes) reach[wd] &= ~(1u << (8 * j));
        }
      }
      const int mine = __popc(reach[0]) + __popc(reach[1]) + __popc(reach[2]) + __popc(reach[3]);
      int total;
      const int before = exclusive(mine, &total);
      if (total == 0) continue;
      if (nparked + total <= kParkCap) {
        int at = nparked + before;
#pragma unroll
        for (int wd = 0; wd < 4; ++wd) at = park_word(reach[wd], qi * 16 + wd * 4, at);
        nparked += total;
      } else {
#pragma unroll
        for (int wd = 0; wd < 4; ++wd) {
          int word_total;
          const int word_before = exclusive(__popc(reach[wd]), &word_total);
          if (nparked + word_total > kParkCap) drain(false);  // leaves fewer than kRound; a word adds at most 128
          park_word(reach[wd], qi * 16 + wd * 4, nparked + word_before);
          nparked += word_total;
        }
      }
      if (nparked >= kRound) drain(false);
      if (*shared_overflow) break;
    }
  }
  for (int begin = 0; !MAP && begin < rd.n_groups; begin += kBatch) {
    const int end = begin + kBatch < rd.n_groups ? begin + kBatch : rd.n_groups;
    uint32_t w[kUnroll][4];
    rd.template take<T>(ring, begin + (int)threadIdx.x, end, w);
    if (end < rd.n_groups) {
      const int next_end = end + kBatch < rd.n_groups ? end + kBatch : rd.n_groups;
      rd.template request_after<T>(ring, end + (int)threadIdx.x, next_end, w, begin + (int)threadIdx.x, end);
    }
    const uint32_t add = toploc_device::bf16_lane_add(thr);
    bool hit[kUnroll];
    uint32_t votes[kUnroll], any_votes = 0;
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int g = begin + u * T + (int)threadIdx.x;
      hit[u] = g < end && toploc_device::vector_reaches<DT, VEC>(make_uint4(w[u][0], w[u][1], w[u][2], w[u][3]), thr, add);
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      votes[u] = __ballot_sync(kFull, hit[u]);
      any_votes |= votes[u];
    }
    if (any_votes) {
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        if (hit[u]) park[nparked + __popc(votes[u] & ((1u << lane) - 1u))] = (uint32_t)(begin + u * T) + threadIdx.x;
        nparked += __popc(votes[u]);
      }
      if (nparked >= kRound) drain(false);
    }
    thr = *shared_thr;
    if (*shared_overflow) break;
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");  // a batch requested before leaving the loop
  if (!*shared_overflow) drain(true);
  __syncthreads();
  if (sh.overflow) return false;
  const uint32_t count = sh.cand_count;

  // The exact k-th key among the candidates: its upper 11 bits from the histogram (it counts
  // every candidate), the bits below 8 at a time (the last digit has 4).
  // (MAP: the histogram is in single 15-bit keys above the threshold, so the walk gives the upper
  // 15 bits at once -- unless the k-th key lies in the last bin, which holds everything beyond the
  // histogram's reach: then the candidates are counted again by their upper 11 bits.)
  find_from_top<T>(sh, coarse, kCoarseBins, (uint32_t)k, 0);
  bool fine = MAP && sh.picked_bin < (uint32_t)kCoarseBins - 1u;
  if (MAP && !fine) {
    __syncthreads();
    clear_words<T>(coarse, kCoarseBins);
    for (uint32_t i = threadIdx.x; i < count; i += T) atomicAdd(&coarse[R::key(cand_pat[i]) >> kCoarseShift], 1u);
    __syncthreads();
    find_from_top<T>(sh, coarse, kCoarseBins, (uint32_t)k, 0);
  }
  uint32_t kth = fine ? thr + (sh.picked_bin << kFineShift) : sh.picked_bin << kCoarseShift;
  uint32_t known = fine ? 0x7FFFu << kFineShift : (uint32_t)(kCoarseBins - 1) << kCoarseShift;
  uint32_t take = sh.picked_remaining, ties = coarse[sh.picked_bin];
  __syncthreads();
  for (int shift = (fine ? kFineShift : kCoarseShift) - 8, round = 1; shift > -8; shift -= 8, ++round) {
    const int low = shift < 0 ? 0 : shift, width = shift < 0 ? 8 + shift : 8;
    clear_words<T>(coarse, 256);
    for (uint32_t i = threadIdx.x; i < count; i += T) {
      const uint32_t key = R::key(cand_pat[i]);
      if ((key & known) == kth) atomicAdd(&coarse[(key >> low) & ((1u << width) - 1u)], 1u);
    }
    __syncthreads();
    find_from_top<T>(sh, coarse, 1 << width, take, round & 1);
    kth |= sh.picked_bin << low;
    known |= ((1u << width) - 1u) << low;
    take = sh.picked_remaining;
    ties = coarse[sh.picked_bin];  // after the last digit: the candidates equal to the k-th key
    __syncthreads();
  }
  // Of the candidates equal to the k-th key the `take` lowest flat indices belong to the top-k.
  // Usually there are a handful: they are listed and the take-th lowest index is found by counting.
  // A long list (a chunk of many equal values) takes the take-th largest of (2^24 - 1 - flat
  // index) digit by digit instead.  Nothing to find when all of them belong.
  uint32_t cut = 0;
  constexpr uint32_t kShortList = 1024;
  if (ties != take && ties <= kShortList) {
    uint32_t* list = coarse;  // (the histogram is done with)
    if (threadIdx.x == 0) sh.emitted = 0;
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < count; i += T)
      if (R::key(cand_pat[i]) == kth) list[atomicAdd(&sh.emitted, 1u)] = cand_flat[i];
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < ties; i += T) {
      const uint32_t mine = list[i];
      uint32_t lower = 0;
      for (uint32_t j = 0; j < ties; ++j) lower += list[j] < mine;
      if (lower == take - 1) sh.picked_bin = 0xFFFFFFu - mine;  // exactly one index has take - 1 below it
    }
    __syncthreads();
    cut = sh.picked_bin;
    if (threadIdx.x == 0) sh.emitted = 0;
    __syncthreads();
  } else if (ties != take) {
    uint32_t cut_known = 0;
    for (int shift = 16, round = 0; shift >= 0; shift -= 8, ++round) {
      clear_words<T>(coarse, 256);
      for (uint32_t i = threadIdx.x; i < count; i += T) {
        if (R::key(cand_pat[i]) != kth) continue;
        const uint32_t inv = 0xFFFFFFu - cand_flat[i];
        if ((inv & cut_known) == cut) atomicAdd(&coarse[(inv >> shift) & 255u], 1u);
      }
      __syncthreads();
      find_from_top<T>(sh, coarse, 256, take, round & 1);
      cut |= sh.picked_bin << shift;
      cut_known |= 255u << shift;
      take = sh.picked_remaining;
      __syncthreads();
    }
  }
  auto selected = [&](uint32_t i) {
    const uint32_t key = R::key(cand_pat[i]);
    return key > kth || (key == kth && 0xFFFFFFu - cand_flat[i] >= cut);
  };

  if (!ORDERED) {
    for (uint32_t i0 = 0; i0 < count; i0 += T) {
      const uint32_t i = i0 + threadIdx.x;
      const bool mine = i < count && selected(i);
      const uint32_t votes = __ballot_sync(kFull, mine);
      uint32_t base = 0;
      if (lane == 0 && votes) base = atomicAdd(&sh.emitted, (uint32_t)__popc(votes));
      base = __shfl_sync(kFull, base, 0);
      if (mine) emit(base + (uint32_t)__popc(votes & ((1u << lane) - 1u)), cand_flat[i], R::committed(cand_pat[i]));
    }
    __syncthreads();
    return true;
  }
  // Index order: one bit per element of the chunk for the selected ones; an element's position is
  // the number of set bits before its own.
  // The number of set bits before every group of kGroup words is kept (16 bits each, in the
  // histogram's place), so a position costs at most kGroup word counts.
  uint32_t* bitmap = ws.bitmap;  // (the caller made sure one bit per element fits)
  uint16_t* before_group = reinterpret_cast<uint16_t*>(coarse);
  const uint32_t n_words = ((uint32_t)rd.n_groups * VEC + 31u) / 32u;
  constexpr uint32_t kGroups = 2u * kCoarseBins;       // 16-bit entries the histogram's place holds
  uint32_t group_shift = 0;                             // words per group: the smallest power of two that fits
  while (((n_words + (1u << group_shift) - 1u) >> group_shift) > kGroups) ++group_shift;
  const uint32_t n_groups = (n_words + (1u << group_shift) - 1u) >> group_shift;
  const uint32_t n_quads = (n_words + 3u) / 4u;          // 16-byte words (the bitmap's place is a whole number of them)
  uint4* quads = reinterpret_cast<uint4*>(bitmap);
  for (uint32_t q = threadIdx.x; q < n_quads; q += T) quads[q] = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
  for (uint32_t i = threadIdx.x; i < count; i += T)
    if (selected(i)) atomicOr(&bitmap[cand_flat[i] >> 5], 1u << (cand_flat[i] & 31u));
  __syncthreads();
  {
    // A warp counts a contiguous stretch of the bitmap, 32 quads (one per lane) at a time, so its
    // loads and stores touch every bank once; a prefix sum over the lanes puts the counts in
    // index order.  First the stretches' totals, then the stores with the warps before added.
    constexpr int kW = T / 32;
    const uint32_t quads_per_warp = ((n_quads + kW - 1) / kW + 31u) / 32u * 32u;
    const uint32_t q_begin = (uint32_t)warp * quads_per_warp;
    uint32_t stretch = 0;
    for (uint32_t q0 = q_begin; q0 < q_begin + quads_per_warp && q0 < n_quads; q0 += 32) {
      const uint32_t q = q0 + (uint32_t)lane;
      const uint4 v = q < n_quads ? quads[q] : make_uint4(0u, 0u, 0u, 0u);
      stretch += (uint32_t)(__popc(v.x) + __popc(v.y) + __popc(v.z) + __popc(v.w));
    }
    stretch = __reduce_add_sync(kFull, stretch);
    unsigned long long total;
    // (every lane of a warp passes the same value: the scan is over warps, read from lane 0's result)
    uint32_t running = (uint32_t)scan_exclusive<T>(sh, lane == 0 ? stretch : 0u, 0, &total);
    running = __shfl_sync(kFull, running, 0);
    // (scan_exclusive's barrier lies between the histogram's last use and these stores)
    for (uint32_t q0 = q_begin; q0 < q_begin + quads_per_warp && q0 < n_quads; q0 += 32) {
      const uint32_t q = q0 + (uint32_t)lane;
      const uint4 v = q < n_quads ? quads[q] : make_uint4(0u, 0u, 0u, 0u);
      const uint32_t c[4] = {(uint32_t)__popc(v.x), (uint32_t)__popc(v.y), (uint32_t)__popc(v.z), (uint32_t)__popc(v.w)};
      const uint32_t mine = c[0] + c[1] + c[2] + c[3];
      uint32_t incl = mine;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const uint32_t other = __shfl_up_sync(kFull, incl, off);
        if (lane >= off) incl += other;
      }
      uint32_t before = running + incl - mine;
      running += __shfl_sync(kFull, incl, 31);
#pragma unroll
      for (uint32_t j = 0; j < 4; ++j) {
        const uint32_t wd = 4u * q + j;
        if (q < n_quads && wd < n_words && (wd & ((1u << group_shift) - 1u)) == 0) before_group[wd >> group_shift] = (uint16_t)before;
        before += c[j];
      }
    }
  }
  __syncthreads();
  // With room behind the candidates the pairs are first put in order in shared memory and the
  // commitment is written in whole words; otherwise every pair goes out on its own.
  const bool staged = rec != nullptr && count + (uint32_t)k <= (uint32_t)kCap;
  uint32_t* sorted_flat = cand_flat + count;
  uint16_t* sorted_pat = reinterpret_cast<uint16_t*>(cand_pat + count);
  for (uint32_t i = threadIdx.x; i < count; i += T) {
    if (!selected(i)) continue;
    const uint32_t flat = cand_flat[i], wd = flat >> 5;
    uint32_t pos = before_group[wd >> group_shift];
    for (uint32_t v = (wd >> group_shift) << group_shift; v < wd; ++v) pos += (uint32_t)__popc(bitmap[v]);
    pos += (uint32_t)__popc(bitmap[wd] & ((1u << (flat & 31u)) - 1u));
    if (staged) {
      if (pos < (uint32_t)k) {
        sorted_flat[pos] = flat;
        sorted_pat[pos] = (uint16_t)R::committed(cand_pat[i]);
      }
    } else {
      emit(pos, flat, R::committed(cand_pat[i]));
    }
  }
  __syncthreads();
  if (staged) {
    write_commitment<T>(rec, sorted_flat, sorted_pat, k);
    __syncthreads();
  }
  return true;
}

// The workspace of select_unordered inside the 1024-thread block's shared memory: histogram and
// candidates where the key histogram of the other selections lives, the parked vectors at the
// end of the spare bytes.
template <int DT>
__device__ __forceinline__ LooseWorkspace<DT> loose_workspace(DirectShared& sh, uint4* ring) {
  LooseWorkspace<DT> ws;
  ws.seen_max = nullptr;
  ws.second_stage = nullptr;
  ws.bitmap = reinterpret_cast<uint32_t*>(ring);
  ws.ctl = &sh.loose;
  ws.coarse = sh.hist;
  ws.cand_flat = sh.hist + kCoarseBins;
  ws.cap = loose_cap(DT);
  ws.cand_pat = reinterpret_cast<typename StoredPattern<DT>::type*>(ws.cand_flat + ws.cap);
  ws.park = reinterpret_cast<uint32_t*>(reinterpret_cast<unsigned char*>(sh.hist) + (size_t)kBins * 4 + kSpareBytes - kParkBytes);
  return ws;
}

template <int DT, bool VECTOR>
__device__ __forceinline__ Reader<DT, VECTOR> locate_chunk(const DirectParams& p, long long chunk) {
  using R = Reader<DT, VECTOR>;
  const long long seq = chunk / p.chunks_per_seq;
  const long long j = chunk - seq * p.chunks_per_seq;
  const long long row0 = seq * p.tokens_per_seq + j * p.chunk_len;
  const long long left = p.tokens_per_seq - j * p.chunk_len;
  const int rows = (int)(left < p.chunk_len ? left : p.chunk_len);
  R rd;
  rd.base = static_cast<const char*>(p.act) + row0 * p.row_stride * R::ESZ;
  rd.row_stride_bytes = p.row_stride * R::ESZ;
  rd.groups_per_row = p.hidden / R::VEC;
  rd.flat = p.row_stride == p.hidden;
  rd.n_groups = rows * rd.groups_per_row;
  return rd;
}

// Per-chunk status an intermediate kernel leaves for the chunks it hands on to the rescue launch
// (never seen by the caller: the rescue launch follows in the same call).
constexpr uint8_t kRetry = 0xFF;

// One chunk's commitment by a 1024-thread block.  loose_failed: the two-pass selection without
// barriers has already outgrown its buffer on this chunk (the rescue launch): go straight to the
// radix select.
template <int DT, bool VECTOR>
__device__ void commit_one_chunk(DirectShared& sh, uint4* ring, const DirectParams& p, long long chunk, uint8_t* commits,
                                 uint8_t* status, bool loose_failed) {
  using R = Reader<DT, VECTOR>;
  const R rd = locate_chunk<DT, VECTOR>(p, chunk);
  uint16_t* rec = reinterpret_cast<uint16_t*>(commits + (size_t)chunk * 6u * (size_t)p.k);
  if ((long long)rd.n_groups * R::VEC < p.k) {
    for (int i = threadIdx.x; i < 3 * p.k; i += kThreads) rec[i] = 0;
    if (threadIdx.x == 0) status[chunk] = TOPLOC_CHUNK_K_EXCEEDS_CHUNK;
    return;
  }
  auto emit = [&](uint32_t pos, uint32_t flat, uint32_t pat) {
    if (pos >= (uint32_t)p.k) return;
    rec[3 * pos] = (uint16_t)(flat & 0xFFFFu);
    rec[3 * pos + 1] = (uint16_t)(flat >> 16);
    rec[3 * pos + 2] = (uint16_t)pat;
  };
  bool done = false;
  if constexpr (VECTOR) {
    if (!loose_failed) {
      if ((long long)rd.n_groups * R::VEC <= kLooseMaxElems)
        done = select_unordered<DT, true, kThreads, false, false>(loose_workspace<DT>(sh, ring), ring, rd, p.k, emit, rec);
      else if (p.k <= kStreamMaxK) done = select_in_one_pass<DT>(sh, ring, rd, p.k, emit);
    }
  }
  if (!done) {
    uint32_t kth, take;
    find_kth_key<DT, VECTOR>(sh, ring, rd, p.k, &kth, &take);
    collect_in_index_order<DT, VECTOR>(sh, ring, rd, p.k, kth, take, emit);
  }
  if (threadIdx.x == 0) status[chunk] = TOPLOC_CHUNK_OK;
}

template <int DT, bool VECTOR>
__global__ void __launch_bounds__(kThreads, 1)
toploc_direct_commit_kernel(DirectParams p, uint8_t* commits, uint8_t* status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint4* ring = reinterpret_cast<uint4*>(smem_raw);
  DirectShared& sh = *reinterpret_cast<DirectShared*>(smem_raw + kRingBytes);
  commit_one_chunk<DT, VECTOR>(sh, ring, p, blockIdx.x, commits, status, false);
}

// What the comparison against a commitment needs besides the two lists.
struct CompareScratch {
  uint32_t bad;
  uint32_t counters[4];  // exponent mismatches, matches, mantissa difference sum, common indices
  uint32_t dev[9];
  uint32_t pad[2];
  uint32_t hist[128];    // mantissa differences 0..127
};

// A chunk that cannot be validated: zero result with its status.
__device__ __forceinline__ void refuse_chunk(const DirectVerify& io, long long chunk, int status) {
  if (threadIdx.x == 0) {
    toploc_chunk_result r = {};
    r.topk_mismatch = -1;
    r.status = (uint8_t)status;
    io.results[chunk] = r;
  }
  if (io.exp_dev != nullptr && threadIdx.x < 9) io.exp_dev[(size_t)chunk * 9 + threadIdx.x] = 0;
}

// Algorithm 2 with a look-up in place of the polynomial, by a block of T threads: the k selected
// (index, pattern) pairs are in sel_idx / sel_pat (any order, all written and visible); the
// commitment is decoded into com_idx / com_pat, checked (indices ascend strictly, lie inside the
// chunk), and every selected index is looked up in it.  Writes the chunk's result.
template <int T>
__device__ void compare_with_commitment(CompareScratch& cs, const DirectVerify& io, long long chunk, int k, uint32_t n_elems,
                                        const uint32_t* sel_idx, const uint16_t* sel_pat, uint32_t* com_idx,
                                        uint16_t* com_pat) {
  if (threadIdx.x == 0) cs.bad = 0;
  if (threadIdx.x < 4) cs.counters[threadIdx.x] = 0;
  if (threadIdx.x < 9) cs.dev[threadIdx.x] = 0;
  const uint16_t* rec = reinterpret_cast<const uint16_t*>(io.commits + (size_t)chunk * 6u * (size_t)k);
  for (int j = threadIdx.x; j < k; j += T) {
    com_idx[j] = (uint32_t)rec[3 * j] | ((uint32_t)rec[3 * j + 1] << 16);
    com_pat[j] = rec[3 * j + 2];
  }
  for (int b = threadIdx.x; b < 128; b += T) cs.hist[b] = 0;
  __syncthreads();
  {
    uint32_t bad = 0;
    for (int j = threadIdx.x; j < k; j += T) bad |= (com_idx[j] >= n_elems) | (j > 0 && com_idx[j] <= com_idx[j - 1]);
    if (bad) cs.bad = 1;
    __syncthreads();
    if (cs.bad) {
      refuse_chunk(io, chunk, TOPLOC_CHUNK_BAD_PROOF);
      return;
    }
  }
  uint32_t err_e = 0, n_match = 0, sum = 0, common = 0, dev[9] = {0, 0, 0, 0, 0, 0, 0, 0, 0};
  const int sign_in_exponent = io.thr_each ? io.thr_each[chunk].sign_in_exponent : io.thr.sign_in_exponent;
  for (int j = threadIdx.x; j < k; j += T) {
    const uint32_t want = sel_idx[j];
    int lo = 0, hi = k;  // first committed index >= want
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (com_idx[mid] < want) lo = mid + 1; else hi = mid;
    }
    if (lo == k || com_idx[lo] != want) {
      ++err_e;  // nothing was committed for this index
      continue;
    }
    ++common;
    const uint32_t committed = com_pat[lo], seen = sel_pat[j];
    const uint32_t field = sign_in_exponent ? 0x1FFu : 0xFFu;
    if (((committed >> 7) & field) == ((seen >> 7) & field)) {
      const uint32_t mp = committed & 0x7Fu, mv = seen & 0x7Fu;
      const uint32_t d = mp > mv ? mp - mv : mv - mp;
      ++n_match;
      sum += d;
      atomicAdd(&cs.hist[d], 1u);
    } else {
      ++err_e;
    }
    const int d = (int)((seen >> 7) & 0xFFu) - (int)((committed >> 7) & 0xFFu);
    const int a = d < 0 ? -d : d;
    const int bin = d == 0 ? 0 : a == 1 ? (d < 0 ? 1 : 2) : a == 2 ? (d < 0 ? 3 : 4) : a <= 10 ? (d < 0 ? 5 : 6) : a <= 99 ? 7 : 8;
#pragma unroll
    for (int b = 0; b < 9; ++b) dev[b] += bin == b;
  }
  err_e = __reduce_add_sync(0xFFFFFFFFu, err_e);
  n_match = __reduce_add_sync(0xFFFFFFFFu, n_match);
  sum = __reduce_add_sync(0xFFFFFFFFu, sum);
  common = __reduce_add_sync(0xFFFFFFFFu, common);
#pragma unroll
  for (int b = 0; b < 9; ++b) dev[b] = __reduce_add_sync(0xFFFFFFFFu, dev[b]);
  if ((threadIdx.x & 31) == 0) {
    atomicAdd(&cs.counters[0], err_e);
    atomicAdd(&cs.counters[1], n_match);
    atomicAdd(&cs.counters[2], sum);
    atomicAdd(&cs.counters[3], common);
#pragma unroll
    for (int b = 0; b < 9; ++b)
      if (dev[b]) atomicAdd(&cs.dev[b], dev[b]);
  }
  __syncthreads();
  if (io.exp_dev != nullptr && threadIdx.x < 9) io.exp_dev[(size_t)chunk * 9 + threadIdx.x] = cs.dev[threadIdx.x];
  if (threadIdx.x == 0) {
    toploc_chunk_result r = {};
    r.exp_mismatch = cs.counters[0];
    r.n_match = cs.counters[1];
    r.mant_diff_sum = cs.counters[2];
    r.topk_mismatch = k - (int)cs.counters[3];
    const toploc_thresholds thr = io.thr_each ? io.thr_each[chunk] : io.thr;
    bool reject = (long long)r.exp_mismatch > (long long)thr.t_exp;
    if (r.n_match > 0) {
      r.mant_mean = nearest_ratio(r.mant_diff_sum, r.n_match);
      // values at sorted positions (n - 1) / 2 and n / 2
      const uint32_t lo_rank = (r.n_match - 1) / 2, hi_rank = r.n_match / 2;
      uint32_t seen = 0;
      int lo_val = -1, hi_val = -1;
      for (int b = 0; b < 128 && hi_val < 0; ++b) {
        seen += cs.hist[b];
        if (lo_val < 0 && seen > lo_rank) lo_val = b;
        if (seen > hi_rank) hi_val = b;
      }
      r.mant_median = ((double)lo_val + (double)hi_val) * 0.5;
      reject = reject || r.mant_mean > thr.t_mean || r.mant_median > thr.t_median;
    } else {
      reject = true;  // nothing matched: no statistic to accept on
    }
    r.accept = reject ? 0 : 1;
    r.status = TOPLOC_CHUNK_OK;
    io.results[chunk] = r;
  }
}
static_assert(sizeof(CompareScratch) <= 4 * kListOffset, "the comparison's scratch sits below the verify lists");

// One chunk's validation by a 1024-thread block (see commit_one_chunk for loose_failed).
template <int DT, bool VECTOR>
__device__ void verify_one_chunk(DirectShared& sh, uint4* ring, const DirectParams& p, long long chunk, const DirectVerify& io,
                                 bool loose_failed) {
  // The two selections live where the key histogram was (it is done with once the k-th key is
  // known), or, after a one-pass selection, in the ring (idle by then).
  uint32_t* sel_idx = sh.hist + kListOffset;
  uint16_t* sel_pat = reinterpret_cast<uint16_t*>(sel_idx + 2 * p.k);
  using R = Reader<DT, VECTOR>;
  const int k = p.k;
  const R rd = locate_chunk<DT, VECTOR>(p, chunk);
  const uint32_t n_elems = (uint32_t)rd.n_groups * R::VEC;
  if (n_elems < (uint32_t)k) {
    refuse_chunk(io, chunk, TOPLOC_CHUNK_K_EXCEEDS_CHUNK);
    return;
  }
  auto emit = [&](uint32_t pos, uint32_t flat, uint32_t pat) {
    if (pos >= (uint32_t)k) return;
    sel_idx[pos] = flat;
    sel_pat[pos] = (uint16_t)pat;
  };
  bool done = false;
  if constexpr (VECTOR) {
    const bool loose = n_elems <= (uint32_t)kLooseMaxElems;  // the comparison needs no particular order
    if (!loose_failed && (loose || k <= kStreamMaxK)) {
      sel_idx = reinterpret_cast<uint32_t*>(ring);
      sel_pat = reinterpret_cast<uint16_t*>(sel_idx + 2 * k);
      done = loose ? select_unordered<DT, false, kThreads, false, false>(loose_workspace<DT>(sh, ring), ring, rd, k, emit)
                   : select_in_one_pass<DT>(sh, ring, rd, k, emit);
    }
  }
  if (!done) {
    sel_idx = sh.hist + kListOffset;
    sel_pat = reinterpret_cast<uint16_t*>(sel_idx + 2 * k);
    uint32_t kth, take;
    find_kth_key<DT, VECTOR>(sh, ring, rd, k, &kth, &take);
    collect_in_index_order<DT, VECTOR>(sh, ring, rd, k, kth, take, emit);
  }
  __syncthreads();
  CompareScratch& cs = *reinterpret_cast<CompareScratch*>(sh.hist);  // (below kListOffset words: free in either case)
  compare_with_commitment<kThreads>(cs, io, chunk, k, n_elems, sel_idx, sel_pat, sel_idx + k, sel_pat + k);
}

template <int DT, bool VECTOR>
__global__ void __launch_bounds__(kThreads, 1)
toploc_direct_verify_kernel(DirectParams p, DirectVerify io) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint4* ring = reinterpret_cast<uint4*>(smem_raw);
  DirectShared& sh = *reinterpret_cast<DirectShared*>(smem_raw + kRingBytes);
  verify_one_chunk<DT, VECTOR>(sh, ring, p, blockIdx.x, io, false);
}

// ---------------------------------------------------------------------------
// 512 < k, vector layouts, chunks of at most 2^18 elements: the two-pass selection without
// barriers needs little more than k candidate slots, so two 512-thread blocks share an SM (113 KB
// each) and one chunk's serial phases -- threshold, exact key, ties, ranking -- run under the
// other's loads.  A chunk whose candidates outgrow the smaller buffer (many equal values) is
// marked and taken by the rescue launch that follows in the same call: a few 1024-thread blocks
// that look at every chunk's mark and run the radix select on the marked ones.
// ---------------------------------------------------------------------------
namespace half_block {
constexpr int kT = 512;
constexpr int kW = kT / 32;
constexpr size_t kRing = (size_t)kUnroll * kT * 16;         // 32 KB; the candidates start here once the chunk has streamed
constexpr size_t kSeen = 32 * 1024;                         // a byte per 8 elements; later a bit per element, or the selection
constexpr long long kMaxElems = (long long)kSeen * 8;       // 2^18
constexpr size_t kPark = (size_t)kW * kParkCap * 4;
constexpr size_t kFixed = kSeen + sizeof(LooseControl) + sizeof(CompareScratch) + (size_t)kCoarseBins * 4 + kPark;
constexpr size_t kBlockBytes = (227 * 1024) / 2 - 1024;      // two blocks per SM, 1 KB reserved for each
__host__ __device__ constexpr int cap(int dt) { return (int)((kBlockBytes - kFixed) / (dt == 0 ? 6 : 8)) / 64 * 64; }
static_assert(kFixed % 16 == 0 && cap(0) >= 2 * 4096 && cap(1) >= 4096 + 2048, "room for the candidates of k = 4096");
static_assert((size_t)cap(0) * 6 >= kRing && (size_t)cap(1) * 8 >= kRing, "the candidates' place contains the ring");
static_assert(kBlockBytes - kFixed + kPark >= 2 * kRing, "candidates and parked groups make room for the second stage");
static_assert(6 * TOPLOC_MAX_K_DIRECT <= kSeen && 6 * TOPLOC_MAX_K_DIRECT <= 6 * 4096,
              "the selection fits the bytes' place, the decoded commitment the candidates' place");

struct Carve {
  uint4* ring;
  CompareScratch* cs;
  unsigned char* seen;  // kSeen bytes
};

template <int DT>
__device__ __forceinline__ LooseWorkspace<DT> carve(unsigned char* smem, Carve* out) {
  // from the end: histogram, comparison scratch, control, the bytes of the first pass, parked
  // groups; everything before them is the candidates' (flat indices, then patterns).  While the
  // chunk streams the first 32 KB are the ring and the next 32 KB -- the rest of the candidates'
  // place and the beginning of the parked groups', both idle until the second pass -- a second
  // stage of it.
  LooseWorkspace<DT> ws;
  out->ring = reinterpret_cast<uint4*>(smem);
  ws.cap = cap(DT);
  ws.cand_flat = reinterpret_cast<uint32_t*>(smem);
  ws.cand_pat = reinterpret_cast<typename StoredPattern<DT>::type*>(ws.cand_flat + ws.cap);
  ws.second_stage = out->ring + kRing / sizeof(uint4);
  unsigned char* at = smem + kBlockBytes - kFixed;
  ws.park = reinterpret_cast<uint32_t*>(at);
  at += kPark;
  out->seen = at;
  ws.seen_max = at;
  ws.bitmap = reinterpret_cast<uint32_t*>(at);
  at += kSeen;
  ws.ctl = reinterpret_cast<LooseControl*>(at);
  at += sizeof(LooseControl);
  out->cs = reinterpret_cast<CompareScratch*>(at);
  at += sizeof(CompareScratch);
  ws.coarse = reinterpret_cast<uint32_t*>(at);
  return ws;
}

// TWO: two parked vectors per lane and round of unpacking (bf16, k >= kTwoFrom).
constexpr int kTwoFrom = 2048;
template <int DT, bool TWO>
__global__ void __launch_bounds__(kT, 2) toploc_direct_commit_half_kernel(DirectParams p, uint8_t* commits, uint8_t* status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Carve cv;
  const LooseWorkspace<DT> ws = carve<DT>(smem_raw, &cv);
  using R = Reader<DT, true>;
  const long long chunk = blockIdx.x;
  const R rd = locate_chunk<DT, true>(p, chunk);
  uint16_t* rec = reinterpret_cast<uint16_t*>(commits + (size_t)chunk * 6u * (size_t)p.k);
  if ((long long)rd.n_groups * R::VEC < p.k) {
    for (int i = threadIdx.x; i < 3 * p.k; i += kT) rec[i] = 0;
    if (threadIdx.x == 0) status[chunk] = TOPLOC_CHUNK_K_EXCEEDS_CHUNK;
    return;
  }
  auto emit = [&](uint32_t pos, uint32_t flat, uint32_t pat) {
    if (pos >= (uint32_t)p.k) return;
    rec[3 * pos] = (uint16_t)(flat & 0xFFFFu);
    rec[3 * pos + 1] = (uint16_t)(flat >> 16);
    rec[3 * pos + 2] = (uint16_t)pat;
  };
  const bool done = select_unordered<DT, true, kT, true, TWO>(ws, cv.ring, rd, p.k, emit, rec);
  if (threadIdx.x == 0) status[chunk] = done ? TOPLOC_CHUNK_OK : kRetry;
}

template <int DT, bool TWO>
__global__ void __launch_bounds__(kT, 2) toploc_direct_verify_half_kernel(DirectParams p, DirectVerify io) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Carve cv;
  const LooseWorkspace<DT> ws = carve<DT>(smem_raw, &cv);
  using R = Reader<DT, true>;
  const long long chunk = blockIdx.x;
  const int k = p.k;
  const R rd = locate_chunk<DT, true>(p, chunk);
  const uint32_t n_elems = (uint32_t)rd.n_groups * R::VEC;
  if (n_elems < (uint32_t)k) {
    refuse_chunk(io, chunk, TOPLOC_CHUNK_K_EXCEEDS_CHUNK);
    return;
  }
  // the selection goes where the first pass's bytes were (done with once the candidates are in),
  // the decoded commitment where the candidates were (done with once the selection has been written out)
  uint32_t* sel_idx = reinterpret_cast<uint32_t*>(cv.seen);
  uint16_t* sel_pat = reinterpret_cast<uint16_t*>(sel_idx + k);
  auto emit = [&](uint32_t pos, uint32_t flat, uint32_t pat) {
    if (pos >= (uint32_t)k) return;
    sel_idx[pos] = flat;
    sel_pat[pos] = (uint16_t)pat;
  };
  if (!select_unordered<DT, false, kT, true, TWO>(ws, cv.ring, rd, k, emit)) {
    if (threadIdx.x == 0) {
      toploc_chunk_result r = {};
      r.status = kRetry;
      io.results[chunk] = r;
    }
    return;
  }
  __syncthreads();
  uint32_t* com_idx = ws.cand_flat;
  uint16_t* com_pat = reinterpret_cast<uint16_t*>(com_idx + k);
  compare_with_commitment<kT>(*cv.cs, io, chunk, k, n_elems, sel_idx, sel_pat, com_idx, com_pat);
}

// The rescue launch: 1024-thread blocks, one per SM at most, look at every chunk's mark.
template <int DT>
__global__ void __launch_bounds__(kThreads, 1) toploc_direct_commit_rescue_kernel(DirectParams p, long long num_chunks,
                                                                                  uint8_t* commits, uint8_t* status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint4* ring = reinterpret_cast<uint4*>(smem_raw);
  DirectShared& sh = *reinterpret_cast<DirectShared*>(smem_raw + kRingBytes);
  for (long long chunk = blockIdx.x; chunk < num_chunks; chunk += gridDim.x) {
    if (status[chunk] != kRetry) continue;  // (the same for every thread: the mark is only rewritten below, after barriers)
    __syncthreads();
    commit_one_chunk<DT, true>(sh, ring, p, chunk, commits, status, true);
    __syncthreads();
  }
}

template <int DT>
__global__ void __launch_bounds__(kThreads, 1) toploc_direct_verify_rescue_kernel(DirectParams p, long long num_chunks,
                                                                                  DirectVerify io) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint4* ring = reinterpret_cast<uint4*>(smem_raw);
  DirectShared& sh = *reinterpret_cast<DirectShared*>(smem_raw + kRingBytes);
  for (long long chunk = blockIdx.x; chunk < num_chunks; chunk += gridDim.x) {
    if (io.results[chunk].status != kRetry) continue;
    __syncthreads();
    verify_one_chunk<DT, true>(sh, ring, p, chunk, io, true);
    __syncthreads();
  }
}

inline bool applies(const toploc_layout* lay, bool vector) {
  const long long rows = lay->tokens_per_seq < lay->chunk_len ? lay->tokens_per_seq : lay->chunk_len;
  return vector && rows * lay->hidden <= kMaxElems;
}
}  // namespace half_block

// ---------------------------------------------------------------------------
// Small k (k <= TOPLOC_MAX_K = 512, chunks of at most 2^19 elements): one warp per chunk, the
// selection of the proof path (toploc_device::select_topk: the chunk streams once through the
// warp's ring, the exact top-k ends up in shared memory), sixteen chunks per SM in flight and
// nothing that waits on another warp (thirteen with the larger scratch of k > 256).  The
// commitment is the selection sorted by index; the validation looks every selected index up in
// the commitment.
// ---------------------------------------------------------------------------
namespace small_k {
using namespace toploc_device;

constexpr int kSmallK = SelectSharedBig::kMaxK;  // 512; k <= 256 takes the smaller scratch (sixteen warps per SM)
constexpr int kWarpsBestUpTo = SelectShared::kMaxK;  // 256: beyond it the half-block kernels are preferred where they apply
constexpr long long kMaxElems = 1ll << 19;
template <class SH>
constexpr int min_blocks() { return SH::kMaxK > 256 ? 13 : 15; }

template <int DT, int MODE>
__device__ __forceinline__ ChunkSource<DT, MODE> source_of(const DirectParams& p, long long chunk, long long* n_elems) {
  const long long seq = chunk / p.chunks_per_seq;
  const long long j = chunk - seq * p.chunks_per_seq;
  const long long row0 = seq * p.tokens_per_seq + j * p.chunk_len;
  const long long left = p.tokens_per_seq - j * p.chunk_len;
  const long long rows = left < p.chunk_len ? left : p.chunk_len;
  ChunkSource<DT, MODE> src;
  src.base = static_cast<const char*>(p.act) + row0 * p.row_stride * (DT == 0 ? 2 : 4);
  src.row_stride = p.row_stride;
  src.hidden = p.hidden;
  src.vecs_per_row = p.hidden / ChunkSource<DT, MODE>::kVec;
  *n_elems = rows * p.hidden;
  return src;
}

// flat index and committed 16-bit pattern of a candidate word
template <int DT>
__device__ __forceinline__ void unpack(unsigned long long c, uint32_t* flat, uint32_t* pattern) {
  const uint32_t key = (uint32_t)(c >> (kIdxBits + 1)), sign = (uint32_t)c & 1u;
  *flat = kIdxMask - ((uint32_t)(c >> 1) & kIdxMask);
  *pattern = (sign << 15) | (DT == 0 ? key : key >> 16);
}

template <int DT, int MODE, class SH>
__global__ void __launch_bounds__(32, min_blocks<SH>()) toploc_direct_commit_warp_kernel(DirectParams p, uint8_t* commits,
                                                                                         uint8_t* status) {
  __shared__ SH sh;
  const int lane = threadIdx.x;
  const long long chunk = blockIdx.x;
  const int k = p.k;
  uint16_t* rec = reinterpret_cast<uint16_t*>(commits + (size_t)chunk * 6u * (size_t)k);
  long long n_elems;
  const ChunkSource<DT, MODE> src = source_of<DT, MODE>(p, chunk, &n_elems);
  if (n_elems < k) {
    for (int i = lane; i < 3 * k; i += 32) rec[i] = 0;
    if (lane == 0) status[chunk] = TOPLOC_CHUNK_K_EXCEEDS_CHUNK;
    return;
  }
  select_topk<DT, MODE>(sh, src, (int)n_elems, k);
  // Ascending index order.  The candidate words are re-keyed by their index field (stored
  // complemented: larger means a lower index) and sorted downwards by a bitonic network over the
  // next power of two (padding words are 0 and sink to the end).
  int padded = 32;
  while (padded < k) padded <<= 1;
  for (int j = lane; j < padded; j += 32) {
    unsigned long long c = 0ull;
    if (j < k) {
      c = sh.cand[j];
      // index field on top, then key and sign: still one distinct word per candidate
      c = ((unsigned long long)(((uint32_t)(c >> 1)) & kIdxMask) << 40) | ((c >> (kIdxBits + 1)) << 1) | (c & 1ull) | (1ull << 39);
    }
    sh.cand[j] = c;
  }
  warp_barrier();
  for (int size = 2; size <= padded; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int t = lane; t < padded / 2; t += 32) {
        const int i = 2 * t - (t & (stride - 1));  // lower partner of pair t
        const int j = i + stride;
        const bool descending = (i & size) == 0;
        const unsigned long long a = sh.cand[i], b = sh.cand[j];
        if ((a < b) == descending) {
          sh.cand[i] = b;
          sh.cand[j] = a;
        }
      }
      warp_barrier();
    }
  }
  for (int pos = lane; pos < k; pos += 32) {
    const unsigned long long c = sh.cand[pos];
    const uint32_t flat = kIdxMask - (uint32_t)(c >> 40);
    const uint32_t key = (uint32_t)(c >> 1) & 0x7FFFFFFFu, sign = (uint32_t)c & 1u;
    const uint32_t pattern = (sign << 15) | (DT == 0 ? key : key >> 16);
    rec[3 * pos] = (uint16_t)(flat & 0xFFFFu);
    rec[3 * pos + 1] = (uint16_t)(flat >> 16);
    rec[3 * pos + 2] = (uint16_t)pattern;
  }
  if (lane == 0) status[chunk] = TOPLOC_CHUNK_OK;
}

template <int DT, int MODE, class SH>
__global__ void __launch_bounds__(32, min_blocks<SH>()) toploc_direct_verify_warp_kernel(DirectParams p, DirectVerify io) {
  constexpr int kSlots = SH::kMaxSlots;
  __shared__ SH sh;
  const int lane = threadIdx.x;
  const long long chunk = blockIdx.x;
  const int k = p.k;
  long long n_elems;
  const ChunkSource<DT, MODE> src = source_of<DT, MODE>(p, chunk, &n_elems);
  auto refuse = [&](int status) {
    if (lane == 0) {
      toploc_chunk_result r = {};
      r.topk_mismatch = -1;
      r.status = (uint8_t)status;
      io.results[chunk] = r;
    }
    if (io.exp_dev != nullptr && lane < 9) io.exp_dev[(size_t)chunk * 9 + lane] = 0;
  };
  if (n_elems < k) {
    refuse(TOPLOC_CHUNK_K_EXCEEDS_CHUNK);
    return;
  }
  select_topk<DT, MODE>(sh, src, (int)n_elems, k);
  uint32_t sel_flat[kSlots], sel_pat[kSlots];
#pragma unroll
  for (int s = 0; s < kSlots; ++s) {
    sel_flat[s] = 0;
    sel_pat[s] = 0;
    if (s * 32 + lane < k) unpack<DT>(sh.cand[s * 32 + lane], &sel_flat[s], &sel_pat[s]);
  }
  // the selection is in registers: the ring holds the commitment, the histograms the statistics
  uint32_t* com_idx = reinterpret_cast<uint32_t*>(sh.ring);
  uint32_t* com_pat = com_idx + SH::kMaxK;
  uint32_t* hist = sh.top_hist;  // a 7-bit mantissa difference is at most 127
  warp_barrier();
  const uint16_t* rec = reinterpret_cast<const uint16_t*>(io.commits + (size_t)chunk * 6u * (size_t)k);
  for (int j = lane; j < k; j += 32) {
    com_idx[j] = (uint32_t)rec[3 * j] | ((uint32_t)rec[3 * j + 1] << 16);
    com_pat[j] = rec[3 * j + 2];
  }
  for (int b = lane; b < 128; b += 32) hist[b] = 0;
  warp_barrier();
  uint32_t bad = 0;  // indices must ascend strictly and lie inside the chunk
  for (int j = lane; j < k; j += 32) bad |= (com_idx[j] >= (uint32_t)n_elems) | (j > 0 && com_idx[j] <= com_idx[j - 1]);
  if (__any_sync(0xFFFFFFFFu, bad != 0)) {
    refuse(TOPLOC_CHUNK_BAD_PROOF);
    return;
  }
  const toploc_thresholds thr = io.thr_each ? io.thr_each[chunk] : io.thr;
  const uint32_t field = thr.sign_in_exponent ? 0x1FFu : 0xFFu;
  uint32_t err_e = 0, n_match = 0, sum = 0, common = 0, dev[9] = {0, 0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
  for (int s = 0; s < kSlots; ++s) {
    if (s * 32 + lane >= k) continue;
    const uint32_t want = sel_flat[s];
    int lo = 0, hi = k;  // first committed index >= want
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (com_idx[mid] < want) lo = mid + 1; else hi = mid;
    }
    if (lo == k || com_idx[lo] != want) {
      ++err_e;  // nothing was committed for this index
      continue;
    }
    ++common;
    const uint32_t committed = com_pat[lo], seen = sel_pat[s];
    if (((committed >> 7) & field) == ((seen >> 7) & field)) {
      const uint32_t mp = committed & 0x7Fu, mv = seen & 0x7Fu;
      const uint32_t d = mp > mv ? mp - mv : mv - mp;
      ++n_match;
      sum += d;
      atomicAdd(&hist[d], 1u);
    } else {
      ++err_e;
    }
    const int d = (int)((seen >> 7) & 0xFFu) - (int)((committed >> 7) & 0xFFu);
    const int a = d < 0 ? -d : d;
    const int bin = d == 0 ? 0 : a == 1 ? (d < 0 ? 1 : 2) : a == 2 ? (d < 0 ? 3 : 4) : a <= 10 ? (d < 0 ? 5 : 6) : a <= 99 ? 7 : 8;
#pragma unroll
    for (int b = 0; b < 9; ++b) dev[b] += bin == b;
  }
  err_e = __reduce_add_sync(0xFFFFFFFFu, err_e);
  n_match = __reduce_add_sync(0xFFFFFFFFu, n_match);
  sum = __reduce_add_sync(0xFFFFFFFFu, sum);
  common = __reduce_add_sync(0xFFFFFFFFu, common);
#pragma unroll
  for (int b = 0; b < 9; ++b) dev[b] = __reduce_add_sync(0xFFFFFFFFu, dev[b]);
  warp_barrier();
  if (io.exp_dev != nullptr && lane < 9) {
    uint32_t mine = 0;
#pragma unroll
    for (int b = 0; b < 9; ++b) mine = lane == b ? dev[b] : mine;
    io.exp_dev[(size_t)chunk * 9 + lane] = mine;
  }
  // median from the histogram: sorted positions (n - 1) / 2 and n / 2; lane l owns bins 4l .. 4l + 3
  uint32_t local[4], mine = 0;
#pragma unroll
  for (int b = 0; b < 4; ++b) {
    local[b] = hist[lane * 4 + b];
    mine += local[b];
  }
  uint32_t incl = mine;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const uint32_t other = __shfl_up_sync(0xFFFFFFFFu, incl, off);
    if (lane >= off) incl += other;
  }
  int lo_val = -1, hi_val = -1;
  if (n_match > 0) {
    const uint32_t lo_pos = (n_match - 1) / 2, hi_pos = n_match / 2;
    uint32_t below = incl - mine;
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
    toploc_chunk_result r = {};
    r.exp_mismatch = err_e;
    r.n_match = n_match;
    r.mant_diff_sum = sum;
    r.topk_mismatch = k - (int)common;
    bool reject = (long long)err_e > (long long)thr.t_exp;
    if (n_match > 0) {
      r.mant_mean = nearest_ratio(sum, n_match);
      r.mant_median = ((double)lo_val + (double)hi_val) * 0.5;
      reject = reject || r.mant_mean > thr.t_mean || r.mant_median > thr.t_median;
    } else {
      reject = true;  // nothing matched: no statistic to accept on
    }
    r.accept = reject ? 0 : 1;
    r.status = TOPLOC_CHUNK_OK;
    io.results[chunk] = r;
  }
}

// 0: flat vectors, 1: aligned rows with padding, 2: element-wise (as in the proof path)
inline int layout_mode(const void* act, const toploc_layout* lay) {
  const int esz = lay->dtype == TOPLOC_DTYPE_BF16 ? 2 : 4;
  const int vec = 16 / esz;
  const bool aligned = (reinterpret_cast<uintptr_t>(act) % 16 == 0) && (lay->hidden % vec == 0) && (lay->row_stride % vec == 0);
  if (!aligned) return 2;
  return lay->row_stride == lay->hidden ? 0 : 1;
}

inline bool applies(const toploc_layout* lay) {
  const long long rows = lay->tokens_per_seq < lay->chunk_len ? lay->tokens_per_seq : lay->chunk_len;
  return lay->k <= kSmallK && rows * lay->hidden <= kMaxElems;
}

template <int DT, class SH>
void launch_commit_sized(int mode, long long n, cudaStream_t stream, const DirectParams& p, uint8_t* commits, uint8_t* status) {
  if (mode == 0) toploc_direct_commit_warp_kernel<DT, 0, SH><<<(unsigned)n, 32, 0, stream>>>(p, commits, status);
  else if (mode == 1) toploc_direct_commit_warp_kernel<DT, 1, SH><<<(unsigned)n, 32, 0, stream>>>(p, commits, status);
  else toploc_direct_commit_warp_kernel<DT, 2, SH><<<(unsigned)n, 32, 0, stream>>>(p, commits, status);
}

template <int DT>
int launch_commit(int mode, long long n, cudaStream_t stream, const DirectParams& p, uint8_t* commits, uint8_t* status) {
  if (p.k > SelectShared::kMaxK) launch_commit_sized<DT, SelectSharedBig>(mode, n, stream, p, commits, status);
  else launch_commit_sized<DT, SelectShared>(mode, n, stream, p, commits, status);
  return cudaGetLastError() == cudaSuccess ? TOPLOC_OK : TOPLOC_ERR_CUDA;
}

template <int DT, class SH>
void launch_verify_sized(int mode, long long n, cudaStream_t stream, const DirectParams& p, const DirectVerify& io) {
  if (mode == 0) toploc_direct_verify_warp_kernel<DT, 0, SH><<<(unsigned)n, 32, 0, stream>>>(p, io);
  else if (mode == 1) toploc_direct_verify_warp_kernel<DT, 1, SH><<<(unsigned)n, 32, 0, stream>>>(p, io);
  else toploc_direct_verify_warp_kernel<DT, 2, SH><<<(unsigned)n, 32, 0, stream>>>(p, io);
}

template <int DT>
int launch_verify(int mode, long long n, cudaStream_t stream, const DirectParams& p, const DirectVerify& io) {
  if (p.k > SelectShared::kMaxK) launch_verify_sized<DT, SelectSharedBig>(mode, n, stream, p, io);
  else launch_verify_sized<DT, SelectShared>(mode, n, stream, p, io);
  return cudaGetLastError() == cudaSuccess ? TOPLOC_OK : TOPLOC_ERR_CUDA;
}
}  // namespace small_k

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------

struct DirectPlan {
  DirectParams params;
  long long num_chunks;
  bool vector;
  int device;  // filled by check_device
};

int plan_direct(const void* d_act, const toploc_layout* lay, DirectPlan* plan) {
  if (lay == nullptr || d_act == nullptr) return TOPLOC_ERR_INVALID_ARGUMENT;
  if (lay->dtype != TOPLOC_DTYPE_BF16 && lay->dtype != TOPLOC_DTYPE_FP32) return TOPLOC_ERR_UNSUPPORTED;
  if (lay->hidden <= 0 || lay->chunk_len <= 0 || lay->num_seqs <= 0 || lay->tokens_per_seq <= 0 || lay->k < 1 ||
      lay->row_stride < lay->hidden)
    return TOPLOC_ERR_INVALID_ARGUMENT;
  if (lay->field != TOPLOC_FIELD_16 || lay->seq_offsets != nullptr || lay->k > TOPLOC_MAX_K_DIRECT)
    return TOPLOC_ERR_UNSUPPORTED;
  const long long rows = lay->tokens_per_seq < lay->chunk_len ? lay->tokens_per_seq : lay->chunk_len;
  if (rows * lay->hidden > kMaxChunkElems) return TOPLOC_ERR_UNSUPPORTED;
  const long long cps = (lay->tokens_per_seq + lay->chunk_len - 1) / lay->chunk_len;
  const long long n = cps * lay->num_seqs;
  if (cps > 0x7FFFFFFFll || n > 0x7FFFFFFFll) return TOPLOC_ERR_UNSUPPORTED;
  const int esz = lay->dtype == TOPLOC_DTYPE_BF16 ? 2 : 4;
  const int vec = 16 / esz;
  plan->vector = lay->hidden % vec == 0 && lay->row_stride % vec == 0 && (reinterpret_cast<uintptr_t>(d_act) & 15u) == 0;
  if (!plan->vector && (reinterpret_cast<uintptr_t>(d_act) & (uintptr_t)(esz - 1)) != 0) return TOPLOC_ERR_INVALID_ARGUMENT;
  plan->params.act = d_act;
  plan->params.row_stride = lay->row_stride;
  plan->params.tokens_per_seq = lay->tokens_per_seq;
  plan->params.hidden = lay->hidden;
  plan->params.chunk_len = lay->chunk_len;
  plan->params.k = lay->k;
  plan->params.chunks_per_seq = (int)cps;
  plan->num_chunks = n;
  return TOPLOC_OK;
}

int check_device(DirectPlan* plan) {
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return TOPLOC_ERR_CUDA;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return TOPLOC_ERR_CUDA;
  plan->device = dev;
  return major == 10 ? TOPLOC_OK : TOPLOC_ERR_ARCH;
}

template <int T = kThreads, class Kernel, class... Args>
int launch_direct(Kernel kernel, long long num_blocks, size_t smem, cudaStream_t stream, Args... args) {
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
    cudaGetLastError();
    return TOPLOC_ERR_CUDA;
  }
  kernel<<<(unsigned)num_blocks, T, smem, stream>>>(args...);
  return cudaGetLastError() == cudaSuccess ? TOPLOC_OK : TOPLOC_ERR_CUDA;
}

}  // namespace

extern "C" {

size_t toploc_direct_commit_bytes(int32_t k) { return k > 0 ? 6 * (size_t)k : 0; }

int toploc_commit_direct(const void* d_act, const toploc_layout* lay, uint8_t* d_commits, uint8_t* d_status,
                         void* cuda_stream) {
  DirectPlan plan;
  int rc = plan_direct(d_act, lay, &plan);
  if (rc != TOPLOC_OK) return rc;
  if (d_commits == nullptr || d_status == nullptr || (reinterpret_cast<uintptr_t>(d_commits) & 1u) != 0)
    return TOPLOC_ERR_INVALID_ARGUMENT;
  if ((rc = check_device(&plan)) != TOPLOC_OK) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const size_t smem = kSharedBytes;
  const DirectParams& p = plan.params;
  // k <= 256: a warp per chunk; above, two half-blocks per SM where they apply (they are level with
  // the warps on chunks of 2^18 elements and well ahead on smaller ones), else the warps up to k = 512
  const bool halves = half_block::applies(lay, plan.vector);
  if (small_k::applies(lay) && !(halves && lay->k > small_k::kWarpsBestUpTo)) {
    const int mode = small_k::layout_mode(d_act, lay);
    return lay->dtype == TOPLOC_DTYPE_BF16 ? small_k::launch_commit<0>(mode, plan.num_chunks, stream, p, d_commits, d_status)
                                           : small_k::launch_commit<1>(mode, plan.num_chunks, stream, p, d_commits, d_status);
  }
  if (halves) {
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, plan.device) != cudaSuccess) return TOPLOC_ERR_CUDA;
    const long long rescuers = plan.num_chunks < sms ? plan.num_chunks : sms;
    if (lay->dtype == TOPLOC_DTYPE_BF16) {
      rc = lay->k >= half_block::kTwoFrom
               ? launch_direct<half_block::kT>(half_block::toploc_direct_commit_half_kernel<0, true>, plan.num_chunks,
                                               half_block::kBlockBytes, stream, p, d_commits, d_status)
               : launch_direct<half_block::kT>(half_block::toploc_direct_commit_half_kernel<0, false>, plan.num_chunks,
                                               half_block::kBlockBytes, stream, p, d_commits, d_status);
      if (rc == TOPLOC_OK)
        rc = launch_direct(half_block::toploc_direct_commit_rescue_kernel<0>, rescuers, smem, stream, p, plan.num_chunks,
                           d_commits, d_status);
    } else {
      rc = launch_direct<half_block::kT>(half_block::toploc_direct_commit_half_kernel<1, false>, plan.num_chunks,
                                         half_block::kBlockBytes, stream, p, d_commits, d_status);
      if (rc == TOPLOC_OK)
        rc = launch_direct(half_block::toploc_direct_commit_rescue_kernel<1>, rescuers, smem, stream, p, plan.num_chunks,
                           d_commits, d_status);
    }
    return rc;
  }
  if (lay->dtype == TOPLOC_DTYPE_BF16)
    return plan.vector ? launch_direct(toploc_direct_commit_kernel<0, true>, plan.num_chunks, smem, stream, p, d_commits, d_status)
                       : launch_direct(toploc_direct_commit_kernel<0, false>, plan.num_chunks, smem, stream, p, d_commits, d_status);
  return plan.vector ? launch_direct(toploc_direct_commit_kernel<1, true>, plan.num_chunks, smem, stream, p, d_commits, d_status)
                     : launch_direct(toploc_direct_commit_kernel<1, false>, plan.num_chunks, smem, stream, p, d_commits, d_status);
}

}  // extern "C"

// Validation with the thresholds of the call (thr, host memory) or one entry per chunk
// (d_thr_each, device memory); exactly one of the two is given.
static int verify_direct_with(const void* d_act, const toploc_layout* lay, const uint8_t* d_commits,
                              const toploc_thresholds* thr, const toploc_thresholds* d_thr_each,
                              toploc_chunk_result* d_results, uint32_t* d_exp_dev_opt, void* cuda_stream) {
  DirectPlan plan;
  int rc = plan_direct(d_act, lay, &plan);
  if (rc != TOPLOC_OK) return rc;
  if (d_commits == nullptr || (thr == nullptr && d_thr_each == nullptr) || d_results == nullptr ||
      (reinterpret_cast<uintptr_t>(d_commits) & 1u) != 0 || (reinterpret_cast<uintptr_t>(d_results) & 7u) != 0 ||
      (reinterpret_cast<uintptr_t>(d_exp_dev_opt) & 3u) != 0 || (reinterpret_cast<uintptr_t>(d_thr_each) & 7u) != 0)
    return TOPLOC_ERR_INVALID_ARGUMENT;
  if (thr != nullptr && thr->t_exp < 0) return TOPLOC_ERR_INVALID_ARGUMENT;
  if ((rc = check_device(&plan)) != TOPLOC_OK) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  DirectVerify io;
  io.commits = d_commits;
  io.results = d_results;
  io.exp_dev = d_exp_dev_opt;
  io.thr = thr ? *thr : toploc_thresholds{};
  io.thr_each = d_thr_each;
  const size_t smem = kSharedBytes;
  const DirectParams& p = plan.params;
  const bool halves = half_block::applies(lay, plan.vector);
  if (small_k::applies(lay) && !(halves && lay->k > small_k::kWarpsBestUpTo)) {
    const int mode = small_k::layout_mode(d_act, lay);
    return lay->dtype == TOPLOC_DTYPE_BF16 ? small_k::launch_verify<0>(mode, plan.num_chunks, stream, p, io)
                                           : small_k::launch_verify<1>(mode, plan.num_chunks, stream, p, io);
  }
  if (halves) {
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, plan.device) != cudaSuccess) return TOPLOC_ERR_CUDA;
    const long long rescuers = plan.num_chunks < sms ? plan.num_chunks : sms;
    if (lay->dtype == TOPLOC_DTYPE_BF16) {
      rc = lay->k >= half_block::kTwoFrom
               ? launch_direct<half_block::kT>(half_block::toploc_direct_verify_half_kernel<0, true>, plan.num_chunks,
                                               half_block::kBlockBytes, stream, p, io)
               : launch_direct<half_block::kT>(half_block::toploc_direct_verify_half_kernel<0, false>, plan.num_chunks,
                                               half_block::kBlockBytes, stream, p, io);
      if (rc == TOPLOC_OK)
        rc = launch_direct(half_block::toploc_direct_verify_rescue_kernel<0>, rescuers, smem, stream, p, plan.num_chunks, io);
    } else {
      rc = launch_direct<half_block::kT>(half_block::toploc_direct_verify_half_kernel<1, false>, plan.num_chunks,
                                         half_block::kBlockBytes, stream, p, io);
      if (rc == TOPLOC_OK)
        rc = launch_direct(half_block::toploc_direct_verify_rescue_kernel<1>, rescuers, smem, stream, p, plan.num_chunks, io);
    }
    return rc;
  }
  if (lay->dtype == TOPLOC_DTYPE_BF16)
    return plan.vector ? launch_direct(toploc_direct_verify_kernel<0, true>, plan.num_chunks, smem, stream, p, io)
                       : launch_direct(toploc_direct_verify_kernel<0, false>, plan.num_chunks, smem, stream, p, io);
  return plan.vector ? launch_direct(toploc_direct_verify_kernel<1, true>, plan.num_chunks, smem, stream, p, io)
                     : launch_direct(toploc_direct_verify_kernel<1, false>, plan.num_chunks, smem, stream, p, io);
}

extern "C" {

int toploc_verify_direct(const void* d_act, const toploc_layout* lay, const uint8_t* d_commits,
                         const toploc_thresholds* thr, toploc_chunk_result* d_results, uint32_t* d_exp_dev_opt,
                         void* cuda_stream) {
  if (thr == nullptr) return TOPLOC_ERR_INVALID_ARGUMENT;
  return verify_direct_with(d_act, lay, d_commits, thr, nullptr, d_results, d_exp_dev_opt, cuda_stream);
}

int toploc_verify_direct_per_chunk_thresholds(const void* d_act, const toploc_layout* lay, const uint8_t* d_commits,
                                              const toploc_thresholds* d_thr_per_chunk,
                                              toploc_chunk_result* d_results, uint32_t* d_exp_dev_opt,
                                              void* cuda_stream) {
  if (d_thr_per_chunk == nullptr) return TOPLOC_ERR_INVALID_ARGUMENT;
  return verify_direct_with(d_act, lay, d_commits, nullptr, d_thr_per_chunk, d_results, d_exp_dev_opt, cuda_stream);
}

}  // extern "C"
