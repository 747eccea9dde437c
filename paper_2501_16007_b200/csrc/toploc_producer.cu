// A producer of last hidden states that commits to them as it writes them.
//
// Section 5.5 places the proof inside the inference engine: a hook takes the
// top-k values of the last hidden layer while the model decodes.  The last
// hidden states of a Llama-style decoder are the output of the final RMSNorm,
// so this file fuses the hook into that normalisation: the block that
// normalises a sequence's new row keeps the row in shared memory, writes it to
// HBM for the language-model head, and its first warp offers the same tile to
// the sequence's running top-k (include/toploc_device.cuh).  The row is never
// read back from HBM for the proof.  toploc_stream_begin / toploc_stream_finish
// open and close the chunk as they do for toploc_stream_append.
//
// Everything a foreign kernel needs is in the public header; this translation
// unit uses nothing else of the library.
#include "toploc.h"
#include "toploc_device.cuh"

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

using namespace toploc_device;

constexpr int kNormThreads = 256;

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// Two fp32 values rounded to nearest-even bf16 and packed (first value in the lower half).
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// y = x * rsqrt(mean(x^2) + eps) * w for one row per block (fp32 arithmetic, bf16 in and out),
// and, when state != nullptr, the row offered to the sequence's running selection as token
// `token` of its chunk.  hidden is a multiple of 8; x, w and y rows are 16-byte aligned.
__global__ void __launch_bounds__(kNormThreads)
toploc_rmsnorm_append_kernel(const uint4* x, long long x_row_vecs, const uint4* w, float eps, uint4* y,
                             long long y_row_vecs, int hidden, int k, int token, unsigned char* state) {
  extern __shared__ __align__(16) unsigned char dyn[];
  uint4* tile = reinterpret_cast<uint4*>(dyn);  // the row: x first, then y in place
  __shared__ SelectSharedBig sh;  // serves every k up to TOPLOC_MAX_K
  __shared__ float partial[kNormThreads / 32];
  const int tid = threadIdx.x;
  const long long seq = blockIdx.x;
  const int vecs = hidden / 8;
  const uint4* xr = x + seq * x_row_vecs;
  uint4* yr = y + seq * y_row_vecs;

  float ss = 0.f;
  for (int v = tid; v < vecs; v += kNormThreads) {
    const uint4 q = xr[v];
    tile[v] = q;
    const uint32_t words[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float a = bf16_lo(words[i]), b = bf16_hi(words[i]);
      ss = fmaf(a, a, ss);
      ss = fmaf(b, b, ss);
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, off);
  if ((tid & 31) == 0) partial[tid >> 5] = ss;
  __syncthreads();
  float total = 0.f;
#pragma unroll
  for (int i = 0; i < kNormThreads / 32; ++i) total += partial[i];
  const float scale = rsqrtf(total / (float)hidden + eps);

  for (int v = tid; v < vecs; v += kNormThreads) {  // every thread revisits the vectors it staged
    const uint4 q = tile[v], g = w[v];
    const uint32_t xs[4] = {q.x, q.y, q.z, q.w}, gs[4] = {g.x, g.y, g.z, g.w};
    uint32_t out[4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
      out[i] = pack_bf16(bf16_lo(xs[i]) * scale * bf16_lo(gs[i]), bf16_hi(xs[i]) * scale * bf16_hi(gs[i]));
    const uint4 r = make_uint4(out[0], out[1], out[2], out[3]);
    tile[v] = r;
    yr[v] = r;
  }
  if (state == nullptr) return;
  __syncthreads();  // the whole row of y is in the tile
  if (tid >= 32) return;
  unsigned char* mine = state + seq * running_selection_bytes(k);
  WarpState st = running_selection_open<0>(sh, mine, k);
  st = running_selection_offer<0>(sh, st, tile, hidden, (uint32_t)token * (uint32_t)hidden, k);
  running_selection_close<0>(sh, st, mine, k);
}

}  // namespace

extern "C" int toploc_rmsnorm_append(const void* d_x, int64_t x_row_stride, const void* d_weight, float eps,
                                     const toploc_layout* lay, int32_t token_in_chunk, void* d_y,
                                     void* d_state_opt, void* cuda_stream) {
  if (lay == nullptr || d_x == nullptr || d_weight == nullptr || d_y == nullptr) return TOPLOC_ERR_INVALID_ARGUMENT;
  if (lay->dtype != TOPLOC_DTYPE_BF16 || lay->field != TOPLOC_FIELD_16) return TOPLOC_ERR_UNSUPPORTED;
  if (lay->hidden <= 0 || lay->chunk_len <= 0 || lay->num_seqs <= 0 || lay->k < 1 || lay->row_stride < lay->hidden ||
      x_row_stride < lay->hidden)
    return TOPLOC_ERR_INVALID_ARGUMENT;
  if (lay->k > TOPLOC_MAX_K || (long long)lay->hidden * lay->chunk_len > (1ll << 24)) return TOPLOC_ERR_UNSUPPORTED;
  if (token_in_chunk < 0 || token_in_chunk >= lay->chunk_len) return TOPLOC_ERR_INVALID_ARGUMENT;
  // rows are moved as 16-byte vectors
  if (lay->hidden % 8 != 0 || lay->row_stride % 8 != 0 || x_row_stride % 8 != 0) return TOPLOC_ERR_UNSUPPORTED;
  if (reinterpret_cast<uintptr_t>(d_x) % 16 != 0 || reinterpret_cast<uintptr_t>(d_y) % 16 != 0 ||
      reinterpret_cast<uintptr_t>(d_weight) % 16 != 0 || reinterpret_cast<uintptr_t>(d_state_opt) % 16 != 0)
    return TOPLOC_ERR_INVALID_ARGUMENT;
  const size_t row_bytes = (size_t)lay->hidden * 2;
  if (row_bytes > 160 * 1024) return TOPLOC_ERR_UNSUPPORTED;  // the row must fit shared memory beside the scratch
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return TOPLOC_ERR_CUDA;
  if (major != 10) return TOPLOC_ERR_ARCH;
  if (row_bytes > 32 * 1024 &&
      cudaFuncSetAttribute(toploc_rmsnorm_append_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)row_bytes) != cudaSuccess)
    return TOPLOC_ERR_CUDA;
  toploc_rmsnorm_append_kernel<<<(unsigned)lay->num_seqs, kNormThreads, row_bytes, static_cast<cudaStream_t>(cuda_stream)>>>(
      static_cast<const uint4*>(d_x), x_row_stride / 8, static_cast<const uint4*>(d_weight), eps,
      static_cast<uint4*>(d_y), lay->row_stride / 8, lay->hidden, lay->k, token_in_chunk,
      static_cast<unsigned char*>(d_state_opt));
  return cudaGetLastError() == cudaSuccess ? TOPLOC_OK : TOPLOC_ERR_CUDA;
}
