/*
 * toploc.h -- C ABI of the TopLoc proof hot path for NVIDIA B200 (sm_100a).
 *
 * TopLoc ("A Locality Sensitive Hashing Scheme for Trustless Verifiable
 * Inference") commits, once per chunk of L tokens, to the k largest-magnitude
 * entries of the last-layer hidden states by interpolating a polynomial
 * congruence through (index mod m, value bits) and storing m plus the k
 * coefficients (Algorithm 1; 258 bytes at k = 128, Section 5.7).  A validator
 * recomputes the activations, repeats the top-k, evaluates the committed
 * polynomial at the recomputed indices and thresholds the exponent / mantissa
 * differences (Algorithm 2, thresholds in Section 5.2).
 *
 * Everything here is plain C: fixed-layout structs, raw pointers and sizes.
 * Each pointer argument says whether it is HOST or DEVICE memory.  The caller
 * owns every buffer; unless an entry point says otherwise the library
 * allocates no device memory, frees nothing of the caller's and only enqueues
 * work on the given CUDA stream.  No C++ exception crosses this boundary and
 * no kernel traps: host-detected problems come back as a negative return code,
 * per-chunk conditions as a status byte.
 */
#ifndef TOPLOC_H_
#define TOPLOC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- constants -------------------------------------------------------- */

/* Activation element types.  fp32 chunks are ranked on the full 31-bit
 * magnitude but commit only the upper 16 bits of each selected pattern
 * (Section 5.6 scales the fp32 mantissa down to bf16's), so proofs keep the
 * 2 + 2k byte size. */
#define TOPLOC_DTYPE_BF16 0
#define TOPLOC_DTYPE_FP32 1

/* Field of the committed polynomial.  TOPLOC_FIELD_16: Z_p with p = 65521,
 * 2-byte coefficients, proofs of 2 + 2k bytes (bf16 chunks; fp32 chunks scaled
 * to 16 bits as above).  TOPLOC_FIELD_32, fp32 chunks only: every selected
 * value commits its whole 32-bit pattern, the arithmetic runs in Z_q with
 * q = 4294967291 = 2^32 - 5 (the largest prime below 2^32; the subroutines
 * appendix names 2^32 as the modulus size for 32-bit types), coefficients take
 * 4 bytes little-endian and a proof 2 + 4k bytes.  Validation then compares
 * fp32 bit fields (sign, 8 exponent bits, 23 mantissa bits), which is what the
 * fp32-inference thresholds of Section 5.2 (8 / 256 / 128) are stated
 * on.  The paper prints neither q nor this layout; they are this library's
 * reading. */
#define TOPLOC_FIELD_16 0
#define TOPLOC_FIELD_32 1
#define TOPLOC_FIELD_32_PRIME 4294967291u
/* Validation only (toploc_verify_proofs and its _host variant), fp32 chunks
 * only: the proofs are TOPLOC_FIELD_16 proofs of a bf16 generator; the
 * polynomial is evaluated over Z_p, every committed 16-bit pattern is padded
 * with 16 zero bits and compared with the validator's whole fp32 pattern
 * (23-bit mantissas, the fp32 thresholds) -- the case of Section 5.6 in which
 * a bf16 model is validated in fp32.  Proofs keep 2 + 2k bytes.  The generating entry
 * points return TOPLOC_ERR_UNSUPPORTED for it. */
#define TOPLOC_FIELD_16_PADDED 2

/* Largest k of a polynomial proof and largest chunk (elements; only chunks
 * the layout really contains count, so chunk_len may exceed every sequence).
 * A chunk of more than 2^19 elements -- a prompt committed as one chunk,
 * Section 5.5 -- is selected in segments of whole rows, one warp each, whose
 * winners are merged; the result is the same top-k.  hidden itself may not
 * exceed 2^24.  k = 512 is about as far as Algorithm 6 reaches: a candidate
 * modulus m separates k indices with probability near exp(-k^2 / 2m), 0.13 at
 * k = 512 and below 1e-3 at k = 1024, so larger k are served by the direct
 * commitments below.  Proofs of k <= 256 take the smaller of two per-warp
 * scratch sizes (sixteen chunks in flight per SM instead of thirteen). */
#define TOPLOC_MAX_K 512
#define TOPLOC_MAX_CHUNK_ELEMS 0x7FFFFFFF
/* Largest k of a direct commitment (toploc_commit_direct): the largest top-k
 * the paper looks at (the exponent-error table of Section 3). */
#define TOPLOC_MAX_K_DIRECT 4096

/* Host-side return codes (0 = success, negative = nothing was enqueued). */
#define TOPLOC_OK 0
#define TOPLOC_ERR_INVALID_ARGUMENT (-1)  /* NULL pointer, non-positive size, k out of range, ... */
#define TOPLOC_ERR_UNSUPPORTED (-2)       /* dtype / k / chunk size outside what the kernels handle */
#define TOPLOC_ERR_WORKSPACE (-3)         /* workspace or staging buffer smaller than required */
#define TOPLOC_ERR_CUDA (-4)              /* a CUDA runtime call or a launch failed */
#define TOPLOC_ERR_ARCH (-5)              /* current device is not compute capability 10.x */
#define TOPLOC_ERR_BUILTIN_SCRATCH (-6)   /* batch too large for toploc_build_proofs_builtin_scratch */
#define TOPLOC_ERR_HOST_MEMORY (-7)       /* the host heap could not supply a row table (ragged batches,
                                             long chunks) or the offsets of a *_host call */

/* Size of the scratch buffer built into the library's device image (8 MiB):
 * enough for 10905 chunks at k = 128 (769 bytes each). */
#define TOPLOC_BUILTIN_SCRATCH_BYTES (8u << 20)

/* Per-chunk status codes (d_status of build, .status of a verify result). */
#define TOPLOC_CHUNK_OK 0
#define TOPLOC_CHUNK_NO_INJECTIVE_MODULUS 1 /* Algorithm 6 ran out of candidates (its "raise") */
#define TOPLOC_CHUNK_K_EXCEEDS_CHUNK 2      /* the chunk holds fewer than k elements */
#define TOPLOC_CHUNK_BAD_PROOF 3            /* decoded modulus outside [2^15+1, 2^16] or a coefficient >= p */
#define TOPLOC_CHUNK_NONFINITE_COMMITTED 4  /* a selected 16-bit pattern is >= p (a negative NaN); the
                                               proof is still produced but cannot reproduce that value */

/* ---- structs ---------------------------------------------------------- */

/* Batch layout.  Activations are a row-major matrix [total_tokens, hidden]
 * with row_stride elements between consecutive token rows.  Sequences occupy
 * consecutive row ranges; every sequence is cut into chunks of chunk_len rows
 * (the last chunk of a sequence may be shorter), and a chunk is flattened
 * row-major: flat index = token_in_chunk * hidden + channel (Section 4: an
 * index needs 4 bytes because 32 x 4096 > 2^16). */
typedef struct {
  int32_t dtype;              /* TOPLOC_DTYPE_* */
  int32_t hidden;             /* H > 0 */
  int32_t chunk_len;          /* L > 0 tokens per chunk (32 in Section 5.5) */
  int32_t k;                  /* 1..TOPLOC_MAX_K (128 in the paper) */
  int32_t num_seqs;           /* > 0 */
  int32_t field;              /* TOPLOC_FIELD_* (0 = 16-bit field, the default); fp32 only for the others */
  int64_t tokens_per_seq;     /* uniform sequence length; used when seq_offsets == NULL */
  const int64_t* seq_offsets; /* HOST, optional: num_seqs + 1 ascending row offsets (ragged batch);
                                 read before the call returns */
  int64_t row_stride;         /* elements between token rows, >= hidden */
} toploc_layout;

/* Acceptance thresholds of Algorithm 2 (Section 5.2: 38 / 10 / 8 for bf16).
 * A chunk is rejected iff exp_mismatch > t_exp or mean > t_mean or
 * median > t_median, or nothing matched, or its status is not OK.
 * sign_in_exponent != 0 compares the sign bit together with the 8 exponent
 * bits (bits 15..7), so a sign flip counts as an exponent mismatch;
 * 0 compares bits 14..7 only. */
typedef struct {
  int32_t t_exp;
  int32_t sign_in_exponent;
  double t_mean;
  double t_median;
} toploc_thresholds;

/* One per chunk, 40 bytes. */
typedef struct {
  uint32_t exp_mismatch;  /* err_e of Algorithm 2 */
  uint32_t n_match;       /* |err_m|: points whose exponent fields agree */
  uint32_t mant_diff_sum; /* exact sum of the |mantissa differences| in err_m */
  int32_t topk_mismatch;  /* k - |generator indices ∩ validator indices| (Section 5.4),
                             -1 when generator indices were not supplied */
  double mant_mean;       /* mant_diff_sum / n_match in fp64, 0 when n_match == 0 */
  double mant_median;     /* median of err_m (mean of the two middle values for an even
                             count), 0 when n_match == 0 */
  uint32_t modulus;       /* decoded m */
  uint8_t accept;         /* 1 = valid, 0 = rejected */
  uint8_t status;         /* TOPLOC_CHUNK_* */
  uint8_t pad[2];
} toploc_chunk_result;

/* ---- queries (host only, no CUDA calls) ------------------------------- */

/* Number of chunks the layout describes (sum over sequences of
 * ceil(len / chunk_len)); negative error code for an invalid layout. */
int64_t toploc_num_chunks(const toploc_layout* lay);

/* 2 + 2k: a 2-byte modulus and k 2-byte coefficients (Section 4, Section 5.7). */
size_t toploc_proof_bytes(int32_t k);

/* Proof bytes per chunk of this layout: 2 + 2k, or 2 + 4k with TOPLOC_FIELD_32;
 * 0 for an invalid layout.  Every proof buffer is [num_chunks, this many]. */
size_t toploc_layout_proof_bytes(const toploc_layout* lay);

/* Bytes of device scratch build/verify need for this layout: the selected
 * (index, pattern) pairs of every chunk (6k + 1 bytes per chunk) that the
 * select kernel hands to the arithmetic kernel, plus a per-chunk row table for
 * ragged batches (seq_offsets != NULL).  A layout with a long chunk (see
 * TOPLOC_MAX_CHUNK_ELEMS) also needs 14k + 17 bytes per segment and 16 bytes
 * per chunk.  One size serves every entry point. */
size_t toploc_workspace_bytes(const toploc_layout* lay);

/* Smallest device staging buffer the *_host entry points accept for this
 * layout: room for the longest sequence's activations plus its outputs. */
size_t toploc_staging_bytes(const toploc_layout* lay);

/* Field prime p (largest prime below 2^16; Algorithm 3's modulus M must be a
 * prime that fits the 2-byte coefficients) and the inclusive modulus search
 * range of Algorithm 6. */
void toploc_get_constants(uint32_t* p, uint32_t* m_lo, uint32_t* m_hi);

const char* toploc_status_string(int chunk_status);
const char* toploc_error_string(int return_code);

/* ---- hot path --------------------------------------------------------- */

/*
 * Proof generation, Algorithm 1, for every chunk of the batch:
 *   top-k by magnitude (key = bit pattern without the sign bit, ties to the
 *   lower flat index)  ->  largest m in [2^15+1, 2^16] for which
 *   (index mod m) mod p is injective (Algorithm 6)  ->  x = (index mod m) mod p,
 *   y = selected 16-bit pattern mod p  ->  coefficients of the unique
 *   polynomial of degree < k through the points over Z_p (Algorithm 3)  ->
 *   proof bytes: m & 0xFFFF little-endian (0 stands for 65536), then the k
 *   coefficients in ascending degree, 2 bytes little-endian each.
 *
 * d_act         DEVICE  activations, layout as described by *lay
 * lay           HOST    read before return
 * d_proofs      DEVICE  out, [num_chunks, toploc_layout_proof_bytes(lay)] bytes (2 + 2k; 2 + 4k with
 *                        TOPLOC_FIELD_32), chunks in batch order
 *                       (sequence-major); zero-filled for a chunk whose status
 *                       is NO_INJECTIVE_MODULUS or K_EXCEEDS_CHUNK
 * d_status      DEVICE  out, [num_chunks] TOPLOC_CHUNK_* bytes
 * d_indices_opt DEVICE  out, optional (NULL to skip): [num_chunks, k] selected
 *                       flat indices ordered by (magnitude desc, index asc)
 * d_workspace   DEVICE  scratch of at least toploc_workspace_bytes(lay) bytes,
 *                       16-byte aligned; contents are undefined afterwards
 * cuda_stream   a cudaStream_t (NULL = default stream)
 *
 * Alignment: d_act a multiple of the element size (2 or 4 bytes; 16-byte
 * aligned rows take the vector path), d_proofs of 2, d_indices_opt of 4, else
 * TOPLOC_ERR_INVALID_ARGUMENT -- nothing is launched with a pointer a kernel
 * could not dereference.
 *
 * Asynchronous: returns after enqueueing; results are valid once the stream
 * has been synchronised.  Returns TOPLOC_OK or a negative TOPLOC_ERR_*.
 * Uniform batches of ordinary chunks do no other host work.  A ragged batch
 * (seq_offsets != NULL) or one with a long chunk (more than 2^19 elements)
 * needs a row table: the call builds it on the host heap -- work and memory
 * proportional to the number of chunks (16 bytes per chunk or segment) --
 * and hands it to the device with a copy from pageable memory, which blocks
 * the calling thread until the bytes are staged; such a call cannot be
 * captured into a CUDA graph.  TOPLOC_ERR_HOST_MEMORY if the heap is exhausted.
 */
int toploc_build_proofs(const void* d_act, const toploc_layout* lay, uint8_t* d_proofs,
                        uint8_t* d_status, int32_t* d_indices_opt, void* d_workspace,
                        size_t workspace_bytes, void* cuda_stream);

/*
 * Proof validation, Algorithm 2, for every chunk: decode (k from the layout
 * must equal (proof length - 2) / 2), top-k on the recomputed activations,
 * x' = (index mod m) mod p, Horner evaluation of the committed polynomial at
 * every x' (Algorithm 5), split both 16-bit patterns into exponent field and
 * 7-bit mantissa, count exponent mismatches and collect |mantissa difference|
 * where the exponents agree, then threshold (strict >) as described at
 * toploc_thresholds.
 *
 * d_act             DEVICE  recomputed activations (same layout as at build)
 * d_proofs          DEVICE  [num_chunks, toploc_layout_proof_bytes(lay)] proofs
 * thr               HOST    thresholds, read before return
 * d_results         DEVICE  out, [num_chunks] toploc_chunk_result
 * d_gen_indices_opt DEVICE  optional: the generator's [num_chunks, k] indices
 *                           (d_indices_opt of build) for topk_mismatch
 * other arguments as for toploc_build_proofs (d_results 8-byte aligned;
 * thr->t_exp < 0 is refused).
 */
int toploc_verify_proofs(const void* d_act, const toploc_layout* lay, const uint8_t* d_proofs,
                         const toploc_thresholds* thr, toploc_chunk_result* d_results,
                         const int32_t* d_gen_indices_opt, void* d_workspace,
                         size_t workspace_bytes, void* cuda_stream);

/*
 * The same validation with one toploc_thresholds entry per chunk.  Section 6
 * proposes acceptance thresholds chosen for the generation at hand (model,
 * precision, sampling settings) instead of one global set; a batch that mixes
 * generations then needs a threshold per chunk.  The statistics do not depend
 * on the thresholds; only accept does (and the exponent comparison, through
 * sign_in_exponent).
 *
 * d_thr_per_chunk  DEVICE  [num_chunks] toploc_thresholds, 8-byte aligned, read
 *                          by the kernels (keep it alive until the stream has
 *                          passed the call).  An entry with a negative t_exp
 *                          rejects its chunk.
 */
int toploc_verify_proofs_per_chunk_thresholds(const void* d_act, const toploc_layout* lay,
                                              const uint8_t* d_proofs,
                                              const toploc_thresholds* d_thr_per_chunk,
                                              toploc_chunk_result* d_results,
                                              const int32_t* d_gen_indices_opt, void* d_workspace,
                                              size_t workspace_bytes, void* cuda_stream);

/*
 * Thresholds of Section 5.2 for a proof of k points: 38 / 10 / 8 at k = 128
 * for the 16-bit field (bf16, or fp32 scaled to 16 bits), 8 / 256 / 128 for
 * fp32 bit fields (TOPLOC_FIELD_32, TOPLOC_FIELD_16_PADDED).  The paper states
 * them at k = 128 only: the exponent threshold counts points and is scaled to
 * floor(t * k / 128); mean and median are per-point statistics and stay.
 * sign_in_exponent is set to 1.  thr HOST, out.  Host only, no CUDA calls.
 */
int toploc_default_thresholds(int32_t k, int32_t field, toploc_thresholds* thr);

/*
 * The selection step on its own: topk(h, k) of Algorithms 1 and 2 for every
 * chunk (Section 5.5 describes the engine-side hook as obtaining exactly
 * this: the top-k values of the last hidden layer).  Same ranking as above:
 * magnitude key, ties to the lower flat index.
 *
 * d_sel_indices         DEVICE out, [num_chunks, k] u32: the selected flat indices of each
 *                       chunk, as a set (order within a chunk is unspecified)
 * d_sel_patterns        DEVICE out, [num_chunks, k] u16: their 16-bit patterns, same order
 *                        (TOPLOC_FIELD_16 layouts only, else TOPLOC_ERR_UNSUPPORTED)
 * d_status              DEVICE out, [num_chunks]: TOPLOC_CHUNK_OK or K_EXCEEDS_CHUNK (whose rows
 *                       of the two arrays above are left untouched)
 * d_ranked_indices_opt  DEVICE out, optional: [num_chunks, k] i32 indices in rank order
 * other arguments as for toploc_build_proofs.  Asynchronous.
 */
int toploc_select_topk(const void* d_act, const toploc_layout* lay, uint32_t* d_sel_indices,
                       uint16_t* d_sel_patterns, uint8_t* d_status, int32_t* d_ranked_indices_opt,
                       void* d_workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Direct commitments.  Section 4 starts from the plain way of committing to a
 * chunk -- the top-k indices and values kept as they are, 6 bytes per point
 * (4 for the index, 2 for the value) -- before replacing it by the polynomial.
 * These two entry points are that plain form.  It is three times the size,
 * but it exists for every k: with thousands of indices (the exponent-error
 * table of Section 3 goes up to k = 4096) no modulus below 2^16 separates
 * them, so Algorithm 6 has nothing to return and a polynomial proof cannot be
 * made.  Same top-k as everywhere else (magnitude key, ties to the lower flat
 * index), 16-bit patterns (fp32 chunks commit their upper 16 bits).
 *
 * A commitment is k records of 6 bytes in ascending index order (the paper
 * fixes no order; this one makes the bytes unique): flat index, 4 bytes
 * little-endian, then the pattern, 2 bytes little-endian.
 *
 * Validation is Algorithm 2 with the polynomial evaluation replaced by a
 * look-up: for every index of the recomputed top-k, the committed pattern at
 * that index is compared as in toploc_verify_proofs; an index that was not
 * committed counts as an exponent mismatch.  topk_mismatch is always filled
 * (the commitment carries the indices), modulus is 0.  A commitment whose
 * indices do not ascend strictly or reach beyond the chunk gets
 * TOPLOC_CHUNK_BAD_PROOF.  Thresholds as in toploc_thresholds (Section 5.2
 * gives them for k = 128; the exponent threshold scales with k).
 *
 * d_commits      DEVICE  [num_chunks, 6k] bytes, 2-byte aligned; zero-filled by
 *                        toploc_commit_direct for a chunk with fewer than k elements
 * d_status       DEVICE  out, [num_chunks]: TOPLOC_CHUNK_OK or K_EXCEEDS_CHUNK
 * d_results      DEVICE  out, [num_chunks]
 * d_exp_dev_opt  DEVICE  out, optional: [num_chunks, 9] u32 counts of the exponent
 *                        deviation (exponent field seen - committed, sign bit left
 *                        out) over the indices both sides selected, in the columns of
 *                        the table in Section 3: 0, -1, +1, -2, +2, -10..-3, 3..10,
 *                        11 <= |d| <= 99, |d| >= 100
 *
 * Limits: lay->k up to TOPLOC_MAX_K_DIRECT, TOPLOC_FIELD_16, uniform batches
 * (seq_offsets == NULL), chunks of at most 2^24 elements; otherwise
 * TOPLOC_ERR_UNSUPPORTED.  No scratch memory is needed.  Asynchronous.
 */
size_t toploc_direct_commit_bytes(int32_t k); /* 6k */
int toploc_commit_direct(const void* d_act, const toploc_layout* lay, uint8_t* d_commits, uint8_t* d_status,
                         void* cuda_stream);
int toploc_verify_direct(const void* d_act, const toploc_layout* lay, const uint8_t* d_commits,
                         const toploc_thresholds* thr, toploc_chunk_result* d_results, uint32_t* d_exp_dev_opt,
                         void* cuda_stream);
/* With one thresholds entry per chunk (DEVICE, [num_chunks]), as
 * toploc_verify_proofs_per_chunk_thresholds. */
int toploc_verify_direct_per_chunk_thresholds(const void* d_act, const toploc_layout* lay, const uint8_t* d_commits,
                                              const toploc_thresholds* d_thr_per_chunk,
                                              toploc_chunk_result* d_results, uint32_t* d_exp_dev_opt,
                                              void* cuda_stream);

/*
 * toploc_build_proofs for callers that have no way to hand over scratch
 * memory.  (The paper has no counterpart to this entry point; it exists for
 * how the library gets embedded.)  Some hosts of this code may not allocate
 * device memory at the point where proofs are generated: a hook inside a
 * serving engine whose memory pool is fixed and fully handed out at start-up,
 * a plug-in that is only given pointers to the engine's tensors, code running
 * where a cudaMalloc would stall or be refused.  For them the select kernel's
 * scratch (the selected index / pattern pairs) lives in a buffer of
 * TOPLOC_BUILTIN_SCRATCH_BYTES that is part of the library itself: every GPU
 * that loads the library carries it until the process ends, and this call
 * allocates nothing, on the device or on the host heap.
 *
 * Arguments and results are those of toploc_build_proofs, minus the
 * workspace; the proofs, statuses and indices are bit-identical.  Limits and
 * rules:
 *   - toploc_workspace_bytes(lay) must not exceed TOPLOC_BUILTIN_SCRATCH_BYTES,
 *     else TOPLOC_ERR_BUILTIN_SCRATCH is returned and nothing is enqueued;
 *   - uniform batches only (seq_offsets == NULL) and no long chunks (more
 *     than 2^19 elements), else TOPLOC_ERR_UNSUPPORTED: their row tables would
 *     have to be built on the host heap;
 *   - the first call on each device looks up the buffer's device address (with
 *     that device current); make that first call outside any stream capture;
 *   - all calls on a device share the one buffer, which keeps whatever the
 *     previous call left in it (nothing in it needs clearing: every entry that
 *     is read has been written by the same call first).  Two calls whose
 *     kernels can overlap on the GPU -- different streams, no dependency --
 *     race on it: keep such calls ordered.
 */
int toploc_build_proofs_builtin_scratch(const void* d_act, const toploc_layout* lay, uint8_t* d_proofs,
                                        uint8_t* d_status, int32_t* d_indices_opt, void* cuda_stream);

/*
 * Incremental proof generation: Algorithm 1 for a provider that decodes one
 * token at a time (Section 5.5: a proof per 32 newly generated tokens).  The
 * rows of the running chunk are handed over as they are produced -- one new
 * row per sequence and step, still warm in L2 -- and every sequence keeps its
 * running top-k in d_state between the steps, so the activations of a chunk
 * never have to be gathered or read again.  The proofs, statuses and indices
 * are bit-identical to toploc_build_proofs over the assembled chunks (ties go
 * to the lower flat index = token_in_chunk * hidden + channel either way).
 *
 * lay describes the running batch: dtype, field, hidden, k, num_seqs, and
 * chunk_len = the most tokens a chunk may receive (chunk_len * hidden may not
 * exceed 2^24); row_stride = elements between the rows of consecutive
 * sequences in d_rows.  tokens_per_seq and seq_offsets are ignored.
 *
 *   toploc_stream_begin    empties the running selections (start of a chunk)
 *   toploc_stream_append   d_rows DEVICE [num_seqs, hidden]: row token_in_chunk
 *                          of every sequence's chunk; call with 0, 1, 2, ... in
 *                          order, on one stream or otherwise ordered
 *   toploc_stream_finish   modulus, interpolation and encode for the chunks as
 *                          they stand: d_proofs [num_seqs, proof bytes],
 *                          d_status [num_seqs], d_indices_opt NULL or
 *                          [num_seqs, k]; a chunk that received fewer than k
 *                          elements gets TOPLOC_CHUNK_K_EXCEEDS_CHUNK.  d_state is
 *                          not modified; begin a new chunk with toploc_stream_begin.
 *
 * d_state      DEVICE, toploc_stream_state_bytes(lay) = num_seqs * (16 + 8k) bytes,
 *              16-byte aligned, owned by the caller, opaque
 * d_workspace  DEVICE scratch for finish, toploc_stream_workspace_bytes(lay)
 * All three only enqueue work on cuda_stream; return codes as above.
 * Validation has no incremental form: a validator sees all tokens at once
 * (Section 5.1) and uses toploc_verify_proofs.
 */
size_t toploc_stream_state_bytes(const toploc_layout* lay);
size_t toploc_stream_workspace_bytes(const toploc_layout* lay);
int toploc_stream_begin(void* d_state, const toploc_layout* lay, void* cuda_stream);
int toploc_stream_append(const void* d_rows, const toploc_layout* lay, int32_t token_in_chunk, void* d_state,
                         void* cuda_stream);
int toploc_stream_finish(const void* d_state, const toploc_layout* lay, uint8_t* d_proofs, uint8_t* d_status,
                         int32_t* d_indices_opt, void* d_workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The engine-side hook of Section 5.5 fused into the kernel that produces the
 * last hidden states: a final RMSNorm (the last operation before a Llama-style
 * model's language-model head) that commits to its output while writing it.
 *   y = x * rsqrt(mean(x^2) + eps) * weight     per row, fp32 arithmetic,
 *                                               bf16 in and out (round to nearest even)
 * One block per sequence normalises the sequence's new row, keeps it in shared
 * memory, writes it to d_y, and offers the same tile to the sequence's running
 * top-k as token token_in_chunk of its chunk -- the proof never reads the row
 * from HBM.  Use it in place of toploc_stream_append: toploc_stream_begin
 * before token 0, this call once per decode step with 0, 1, 2, ..., and
 * toploc_stream_finish for the proofs, which are bit-identical to
 * toploc_build_proofs over the rows written to d_y.  The device routines it is
 * built from are public (include/toploc_device.cuh) for engines that want the
 * same hook in a kernel of their own.
 *
 * d_x          DEVICE  [num_seqs, hidden] bf16, x_row_stride elements between rows
 * d_weight     DEVICE  [hidden] bf16
 * lay          HOST    as for toploc_stream_append (dtype bf16, TOPLOC_FIELD_16;
 *                      row_stride = elements between the rows of d_y)
 * d_y          DEVICE  out, [num_seqs, hidden] bf16
 * d_state_opt  DEVICE  the running selections (toploc_stream_state_bytes), or
 *                      NULL for the normalisation alone
 * hidden and both strides must be multiples of 8 and every pointer 16-byte
 * aligned (rows move as 16-byte vectors), hidden at most 81920; else
 * TOPLOC_ERR_UNSUPPORTED / TOPLOC_ERR_INVALID_ARGUMENT.  Asynchronous.
 */
int toploc_rmsnorm_append(const void* d_x, int64_t x_row_stride, const void* d_weight, float eps,
                          const toploc_layout* lay, int32_t token_in_chunk, void* d_y, void* d_state_opt,
                          void* cuda_stream);

/*
 * The same two operations for callers whose data lives in HOST memory
 * (pinned memory gives asynchronous copies; pageable memory works).  The
 * batch is cut into groups of whole sequences that fit the staging buffer;
 * each group is copied host->device, processed, and its proofs / results are
 * copied device->host, all on cuda_stream.  The stream is synchronised before
 * returning, so the host outputs are complete on return.
 *
 * h_act / h_proofs / h_status / h_results  HOST buffers, shapes as above
 * d_staging  DEVICE scratch of staging_bytes >= toploc_staging_bytes(lay),
 *            256-byte aligned; a larger buffer means fewer, larger groups
 */
int toploc_build_proofs_host(const void* h_act, const toploc_layout* lay, uint8_t* h_proofs,
                             uint8_t* h_status, void* d_staging, size_t staging_bytes,
                             void* cuda_stream);

int toploc_verify_proofs_host(const void* h_act, const toploc_layout* lay, const uint8_t* h_proofs,
                              const toploc_thresholds* thr, toploc_chunk_result* h_results,
                              void* d_staging, size_t staging_bytes, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* TOPLOC_H_ */
