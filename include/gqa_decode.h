/*
 * gqa_decode.h -- C ABI of the second workload: one decode step of grouped-query attention over a paged
 * key-value cache, for B200 (sm_100a).  Same library (libmoe_b200.so) and conventions as moe.h: device pointers
 * owned by the caller unless a parameter says HOST, nothing allocated or freed, launches only on the given stream
 * without synchronising it, arguments checked on the host before anything is launched, status codes of
 * moe_status_t.
 *
 * The operation (K-Search paper, Sec. 4.6 "Kernel Analysis: GQA Paged Decode", and its row of Table 2): every
 * batch item contributes ONE new query token, which attends over the keys and values already stored in the paged
 * cache; Hq / Hkv query heads share one key-value head.  For batch item b, query head h (key-value head
 * g = h / (Hq / Hkv)) and the L_b cached tokens t of b:
 *     s_t      = sm_scale * sum_d q[b,h,d] * k[t,g,d]
 *     out[b,h] = sum_t softmax_t(s)_t * v[t,g,:]                      (bf16; fp32 accumulation)
 *     lse[b,h] = log sum_t exp(s_t)                                   (natural logarithm, f32; optional)
 * Token t of item b lives in page kv_indices[kv_indptr[b] + t / page_size] at slot t % page_size, and
 * L_b = (kv_indptr[b+1] - kv_indptr[b] - 1) * page_size + kv_last_page_len[b] (0 for an item without pages, whose
 * out is 0 and lse -inf).
 *
 * How it is computed (the paper's kernel, Sec. 4.6: the sequence is split across blocks, each block writes a
 * partial result to a temporary buffer, and the block that finds itself last -- a counter -- merges them; keys and
 * values are fetched in chunks while the previous chunk is being used): one block per (sequence chunk, key-value
 * head, batch item) keeps all Hq / Hkv query heads of its key-value head in registers, so every key and value is
 * read from memory once per group, streams its tokens through a pipeline of TMA copies that follow the page table
 * (one tile per page for page sizes that are powers of two of at least 8, one 256-byte row copy per token otherwise),
 * and the last block of each (item, key-value head) merges the partial results.  Results do not depend on which block
 * is last.
 */
#ifndef GQA_DECODE_B200_H_
#define GQA_DECODE_B200_H_

#include <stddef.h>
#include <stdint.h>

#include "moe.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Host-only, pure.  Bytes of workspace gqa_paged_decode needs (a status word, block counters and the partial results
 * of the sequence splits); 0 outside the supported envelope.  max_kv_len: an upper bound of the cached lengths, used to size
 * the split of the sequence (a longer sequence is still computed correctly, by its last block).
 * Envelope: D == 128; Hq a multiple of Hkv with 1 <= Hq / Hkv <= 16; B >= 0; max_kv_len >= 0. */
MOE_API size_t gqa_decode_workspace_bytes(int B, int Hq, int Hkv, int D, int max_kv_len);

/* One decode step (Sec. 4.6).
 *   q                [B,Hq,D] bf16, in
 *   k_cache, v_cache [num_pages,page_size,Hkv,D] bf16, in
 *   kv_indptr        [B+1] int32, in: item b owns pages kv_indices[kv_indptr[b] .. kv_indptr[b+1])
 *   kv_indices       [kv_indptr[B]] int32, in: page numbers in [0, num_pages)
 *   kv_last_page_len [B] int32, in: tokens in the last page of each item, in [1, page_size] (ignored without pages)
 *   sm_scale         the score scale (usually D^-0.5)
 *   out              [B,Hq,D] bf16, out
 *   lse              [B,Hq] f32, out, or NULL
 *   workspace        at least gqa_decode_workspace_bytes(...) bytes, 256-byte aligned; concurrent calls need distinct
 *                    workspaces.  Afterwards its first int32 is the call's device status, which
 *                    moe_last_status(workspace, stream) reads: MOE_OK, or MOE_ERR_DEVICE_TIMEOUT when a block's bounded
 *                    wait for its copies ran out (out is then incomplete); the rest is undefined
 * Pointers of q, the caches and out must be 16-byte aligned, the int arrays and lse 4-byte aligned.
 * B == 0 succeeds without a launch.  Page numbers and lengths are NOT validated (they live on the device); page
 * numbers outside [0, num_pages) are outside the contract.  num_pages * page_size must be below 2^31
 * (MOE_ERR_UNSUPPORTED).  Enqueues one memset and one kernel; returns MOE_ERR_CUDA when a tensor map cannot be encoded
 * or the launch fails. */
MOE_API int gqa_paged_decode(const void *q, const void *k_cache, const void *v_cache, const int32_t *kv_indptr,
                             const int32_t *kv_indices, const int32_t *kv_last_page_len, int B, int Hq, int Hkv, int D,
                             int page_size, int num_pages, int max_kv_len, float sm_scale, void *out, float *lse,
                             void *workspace, size_t workspace_bytes, void *stream);

/* Self-test of the device-side error path, as moe_selftest_wait_timeout: every wait of the decode kernel (on the
 * barriers its copies complete on) is bounded; this call enqueues one warp that waits, with a bound of a few
 * milliseconds, on a barrier at which nothing arrives.  Afterwards moe_last_status(workspace, stream) must report
 * MOE_ERR_DEVICE_TIMEOUT and the device must be usable as before.  workspace: at least 256 bytes, 256-byte aligned
 * (its first 256 bytes are overwritten). */
MOE_API int gqa_selftest_wait_timeout(void *workspace, size_t workspace_bytes, void *stream);

/* Host-only, pure.  Tokens per sequence split and number of splits the call above uses for these sizes (reporting). */
MOE_API int gqa_decode_split_tokens(int B, int Hq, int Hkv, int D, int max_kv_len);

#ifdef __cplusplus
}
#endif
#endif /* GQA_DECODE_B200_H_ */
