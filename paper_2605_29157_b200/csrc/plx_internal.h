// Functions one source file of the library defines and another one calls.  Internal to the library: C++ linkage,
// not part of the C interface (that is parallax.h).
#ifndef PLX_INTERNAL_H_
#define PLX_INTERNAL_H_

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

// parallax_decode.cu: the split merge of the decode path over `rows` rows of `num_splits` records each, launched as
// a programmatic dependent of the kernel before it in the stream (which must signal or complete first).
int plx_combine_after_producer(const float* partials, void* out, int rows, int D, int num_splits, int out_dtype,
                               cudaStream_t stream);

// parallax_decode_rows.cu: multi-token decode steps of up to 32 rows per KV head on the tensor cores with the keys
// on the accumulator lanes.  q, r, out [B, Hq, Lq, D]; `records` / `record_bytes`: room for split records (may be
// null: one split).  Paged cache: block_table != nullptr, k_cache / v_cache are the page pools of pool_rows rows
// and T_max = page_size * max_pages.  `ticket`: a device int32 that is zero between calls (or nullptr): with it,
// calls of more items than SMs run one CTA per SM, each drawing (sequence, KV head, split) items from that word.
bool plx_decode_rows_supported(int Hq, int Hkv, int D, int Lq);
bool plx_decode_rows_page_size_ok(int page_size);
int plx_decode_rows_plan(int B, int Hq, int Hkv, int D, int Lq, int T_max, int page_size, int sms);
int plx_decode_rows_fwd(const void* q, const void* r, const void* k_cache, const void* v_cache, const int32_t* seqlens,
                        void* out, int B, int Hq, int Hkv, int D, int Lq, int T_max, float scale, int out_dtype,
                        void* records, size_t record_bytes, int num_splits, int32_t* status, cudaStream_t stream,
                        const int32_t* block_table, int page_size, int max_pages, long long pool_rows, int32_t* ticket);

#endif  // PLX_INTERNAL_H_
