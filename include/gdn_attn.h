/*
 * gdn_attn.h -- C ABI of the causal softmax attention of the hybrid backbone's attention layers
 * (second workload of libgdn; status codes and gdn_stream_t come from gdn.h).
 *
 * The operation (Sections "The layout trick" and "Prefill attention: finding and removing the O(N^2) wall": scores for all queries of a block as one matrix
 * product, a softmax that normalises only the causally valid prefix and leaves exact zeros after
 * it, a second product with V; grouped-query attention by letting several query heads address
 * the same key/value block).  For every sequence b, query head h and position i:
 *
 *     s_j   = scale * <q[b,i,h,:], k[b,j,g,:]>           j = 0..i,   g = h / (Hq / Hkv)
 *     out[b,i,h,:] = sum_j softmax(s)_j * v[b,j,g,:]
 *
 * Layouts (row-major, DEVICE pointers, 16-byte aligned): q, out [B, T, Hq, d]; k, v [B, T, Hkv, d];
 * bf16 storage, fp32 scores, softmax and accumulation, `out` rounded to nearest even.
 * With cu_seqlens != NULL (B + 1 ascending int32 on the device, cu_seqlens[0] = 0, cu_seqlens[B] = T)
 * the tensors are packed [T, H, d] with T the total number of tokens, as in gdn_chunk_prefill:
 * sequence n owns tokens [cu_seqlens[n], cu_seqlens[n+1]) and attends only to itself; empty
 * sequences are allowed.
 * Supported: d = 128, Hq a positive multiple of Hkv.  Where the paper writes the score matrix to
 * a buffer (heads x T x T floats), this library keeps 128 x 128 tiles of it in tensor memory only.
 *
 * Returns GDN_OK, GDN_ERR_INVALID_ARG (null or negative arguments, scale negative or not finite),
 * GDN_ERR_UNSUPPORTED (sizes, alignment), GDN_ERR_TOO_LARGE (B*T >= 2^31), GDN_ERR_CUDA.  The call
 * is asynchronous on `stream`, allocates nothing and owns none of its arguments; B = 0 or T = 0
 * is a no-op.  A bounded wait that expires inside the kernel shows up in gdn_query_status().
 */
#ifndef GDN_ATTN_H_
#define GDN_ATTN_H_

#include "gdn.h"

#ifdef __cplusplus
extern "C" {
#endif

int gdn_attn_causal_prefill(const void* q, const void* k, const void* v, void* out,
                            const int32_t* cu_seqlens,
                            int B, int T, int Hq, int Hkv, int d, float scale,
                            gdn_stream_t stream);

#ifdef __cplusplus
}
#endif

#endif /* GDN_ATTN_H_ */
