// Internal declarations shared by the host runtime and the kernel files.
// Nothing here is part of the public ABI (see include/kvcar.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kvcar.h"

namespace kvcar {

constexpr int MAX_SRC = KVCAR_MAX_KV_HEADS;

// One place a layer's decode reads cached rows from: its own pool, or the pool of
// a lower layer that some of its heads reuse.  Device-resident, built at bind time.
struct SourcePlan {
    const void *pool;  // root layer's rows [max_pages*page_tokens][width], storage dtype
    const void *w1t;   // decoder FC1 transposed [d][m], storage dtype
    const float *s1;   // bias + BatchNorm fused per hidden feature: a = acc*s1 + t1
    const float *t1;
    const void *w2t;   // decoder FC2 transposed [m][in_dim], storage dtype
    const float *b2;   // [in_dim]
    const void *w1k;   // K-major bf16 copies for the tensor-core kernel: [m][d]
    const void *w2k;   //                                                  [in_dim][m]
    const float *qparam;  // int8 rows: (scale, zero-point) per pool row, else null
    int32_t width;     // elements per pool row (= d if compressed, = in_dim if raw)
    int32_t d, m, in_dim;
    int32_t compressed;
    int32_t src_layer;
    int32_t n_need;    // heads of the reading layer served from this source
    float slope;
    int8_t kv_head[KVCAR_MAX_KV_HEADS];  // for i < n_need: KV head of the reading layer
    int8_t slot[KVCAR_MAX_KV_HEADS];     //                 column slot (x head_dim) in the restored row
};

struct WhichPlan {
    int32_t n_src;
    int32_t pad_[3];
    SourcePlan src[MAX_SRC];
};

struct LayerPlan {
    WhichPlan w[2];
    // exact current-token rows: per KV head, the root layer's rows [max_seqs][kv_width] and the root head
    const void *cur[2][KVCAR_MAX_KV_HEADS];
    int32_t cur_head[2][KVCAR_MAX_KV_HEADS];
};

struct EncPlan {
    void *pool;       // this layer's rows
    void *cur;        // this layer's current-token rows [max_seqs][kv_width]
    const void *w1t;  // encoder FC1 transposed [in_dim][m]
    const float *s1, *t1;
    const void *w2t;  // encoder FC2 transposed [m][d]
    const float *b2;
    const void *w1r;  // encoder FC1 as given, [m][in_dim], storage dtype (rows read by one warp each)
    const void *w2r;  // encoder FC2 as given, [d][m]
    float *qparam;    // int8 rows: (scale, zero-point) per pool row, else null
    int32_t width, d, m, in_dim, compressed, n_stored;
    float slope;
    int32_t pad_;
    int8_t heads[KVCAR_MAX_KV_HEADS];  // stored heads, ascending
};

struct SeqList {
    int32_t n;
    int32_t id[KVCAR_MAX_BATCH];
};

struct DecodeArgs {
    const LayerPlan *plan;
    const int32_t *block_table;  // [max_seqs][max_pages_per_seq]
    const int32_t *seq_len;      // [max_seqs]
    const void *q;               // [n_seqs][hq][hd]
    void *out;                   // [n_seqs][hq][hd]
    float *partials;             // [n_seqs][max_chunks][hq][hd+2]
    int32_t *status;             // device status word (0 = ok)
    int32_t max_pages_per_seq, page_tokens;
    int32_t hq, hkv, hd;
    int32_t chunk_tokens, max_chunks;
    uint32_t flags;
    float scale;
    const void *raw_tmaps;  // TMA descriptors of the raw (layer, K|V) pools (descriptor of pool i at + i * 384 bytes),
                            // or null: the raw-row kernel then stages its rows with cp.async
};

struct EncodeArgs {
    const EncPlan *plan;  // [2] for this layer: K then V
    const int32_t *block_table;
    const int32_t *seq_len;
    const void *k, *v;    // [n_seqs][n_tokens][kv_width]
    int32_t max_pages_per_seq, page_tokens;
    int32_t n_tokens, kv_width, hd;
};

struct TableUpdates {
    // kind 0: block_table[a*max_pages_per_seq + b] = c ; kind 1: seq_len[a] = c
    int32_t n;
    int32_t max_pages_per_seq;
    int4 e[240];
};

// launchers implemented in kvcar_generic.cu (return cudaGetLastError())
cudaError_t launch_table_updates(int32_t *block_table, int32_t *seq_len, const TableUpdates &u, cudaStream_t st);
cudaError_t launch_encode_generic(const EncodeArgs &a, const SeqList &seqs, int dtype, int max_in, int max_m,
                                  cudaStream_t st);
// one new token per sequence, one launch per fully connected layer (kvcar_encode.cu); `hid` is an fp32 scratch of
// [2][max_batch][max_m] for the hidden activations
cudaError_t launch_encode_split(const EncodeArgs &a, const SeqList &seqs, int dtype, int max_in, int max_m, int max_d,
                                float *hid, int max_batch, cudaStream_t st);
size_t encode_split_smem(int max_in, int max_m);
cudaError_t launch_decode_generic(const DecodeArgs &a, const SeqList &seqs, int dtype, int max_d, int max_m,
                                  int grid_chunks, cudaStream_t st);
// raw K/V layers (no autoencoder), head_dim 64, <= 8 query heads per KV head (kvcar_raw.cu)
cudaError_t launch_decode_raw(const DecodeArgs &a, const SeqList &seqs, int dtype, int grid_chunks, cudaStream_t st);
// TMA descriptor of one raw bf16 pool [rows][width] with a box of 32 rows x 64 columns (one head's slice of one
// 32-token step), 128-byte swizzle; false if the driver entry point is missing or the shape is refused
bool raw_build_map(void *dst_host, const void *pool_dev, uint64_t rows, uint64_t width);
// n_chunks: tiles of the longest listed sequence (picks the kernel: a warp or a CTA per sequence and query head)
cudaError_t launch_combine(const DecodeArgs &a, const SeqList &seqs, int dtype, int n_chunks, cudaStream_t st);
size_t decode_generic_smem(int hq, int hd, int max_d, int max_m);

// Bulk encoder + append on the tensor cores (kvcar_prefill_tc.cu): bf16 storage, both K and V of the layer with an
// autoencoder, head_dim 64, hidden and latent widths multiples of 16.  Rows are worked through in blocks of
// PREFILL_TC_ROWS; `hid` is a bf16 scratch of prefill_tc_scratch_bytes(max hidden width) bytes.
constexpr int PREFILL_TC_ROWS = 32768;
struct PrefillTcArgs {
    const EncPlan *plan_dev;    // this layer's [K, V] plans on the device
    const EncPlan *plan_host;   // the same two plans, host copy (widths and weight pointers for the tensor maps)
    const int32_t *block_table;
    const int32_t *seq_len;
    int32_t *status;
    const void *src[2];         // the caller's K and V rows [n_seqs * n_tokens][kv_width]
    void *hid;
    int32_t max_m;
    int32_t max_pages_per_seq, page_tokens, n_tokens, kv_width;
};
size_t prefill_tc_scratch_bytes(int max_m);
cudaError_t launch_prefill_tc(const PrefillTcArgs &a, const SeqList &seqs, cudaStream_t st);

}  // namespace kvcar
