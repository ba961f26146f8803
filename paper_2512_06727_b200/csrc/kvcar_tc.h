// Interface between the host runtime and the tcgen05/TMEM fused kernel file.
#pragma once
#include "kvcar_internal.h"

namespace kvcar {

constexpr int TC_MAX_LAYERS = 512;
constexpr int TC_MAX_SRC = 6;    // distinct source layers per K or V of one head subset
constexpr int TC_MAX_JOBS = 24;  // accumulator jobs per K or V of one head subset
constexpr int TC_SPLIT_TILES = 160;  // the K/V split is used only while 2 x tiles <= SM count
constexpr int TC_PARTS_PER_LAYER = 9;  // head subsets: whole, halves, quarters; then the whole with absorbed K scores,
                                       // then the whole with absorbed K scores and the absorbed V side
constexpr int TC_ABS_MAX_Q = 32;       // query heads the absorbed score job takes (two CTAs x 32 columns at most)

// One source layer as the tensor-core kernel sees it.
struct TcSrc {
    const void *tm_pool, *tm_w1, *tm_w2;  // TMA descriptors (device memory): cache rows, decoder FC1, decoder FC2
    const float *s1, *t1, *b2;            // fused bias+BatchNorm scale/shift [m]; last-FC bias [in_dim]
    int32_t d, m;
    float slope;
    int32_t in_dim;
};

// One accumulator job: a chunk of hidden columns (first decoder layer) or a group of
// up to four restored heads (second decoder layer).  The TMA producer, the MMA issuer
// and the epilogue warps all walk the same list in the same order.
struct TcJob {
    uint8_t kind;    // 1 = hidden chunk, 2 = head group, 3 = absorbed scores of all query heads of the source (K only),
                     // 4 = absorbed V side: sum over the tile's tokens of p * hidden vector for all query heads of
                     // the source (for 3 and 4, c0 | nc << 16 is the mask of the source's local query heads)
    uint8_t src;     // index into TcPart::src[which]
    uint8_t nh;      // head group: real heads (1..4)
    uint8_t first;   // first job of its source
    uint16_t c0;     // hidden chunk: first hidden column
    uint16_t nc;     // hidden chunk: width (multiple of 16, <= 256)
    int8_t kvh[4];   // head group: KV head of the reading layer per head place (-1 = padding)
    int8_t slot[4];  // head group: 64-wide column slot of the restored row per head place
};

// Everything one cluster needs for one layer and one subset of its KV heads.
struct TcPart {
    int32_t n_src[2], n_jobs[2];
    int32_t h_lo, h_hi;  // KV heads [h_lo, h_hi) of the reading layer
    int32_t max_m, pad_;
    TcSrc src[2][TC_MAX_SRC];
    TcJob jobs[2][TC_MAX_JOBS];
    // absorbed tables only: per K source the local query heads it serves, in order
    uint8_t abs_n[16];
    uint8_t abs_q[TC_MAX_SRC][TC_ABS_MAX_Q];
};

struct TcLayerCfg {
    uint8_t ok;            // this layer can run on the tensor-core kernel
    uint8_t split_ok[3];   // head splits 1, 2, 4 available
    uint16_t max_m;        // widest hidden layer among the layer's sources
    uint16_t max_in;       // widest restored row among the layer's sources
    uint16_t pslots;       // parameter blocks kept in shared memory (one per source if every hidden layer is one chunk)
    uint8_t abs_ok;        // the absorbed table (index 7) exists
    uint8_t absv_ok;       // the table with the absorbed V side as well (index 8) exists
};

struct TcState {
    bool available = false;
    const char *why = "not set up";
    char *parts_dev = nullptr;  // TcPart[n_layers][8] in the weights buffer: split 1 -> [0], 2 -> [1..2], 4 -> [3..6], absorbed -> [7]
    // absorbed K scores: W4_h^T q per (K source, listed sequence, query head) as bf16 rows, q.b4_h beside them
    void *wq = nullptr;             // [max K sources][batch][nq_pad][m_pad] bf16 (workspace)
    float *qbias = nullptr;         // [max K sources][batch][nq_pad]
    const void *tm_wq = nullptr;    // TMA descriptor of wq (device memory), box = 64 columns x nq_pad rows
    int abs_nq_pad = 0, abs_m_pad = 0, abs_batch = 0, abs_max_src = 0;
    // absorbed V side: per (listed sequence, tile, query head) the m-vector sum_t p_t a_t (workspace), and which form
    // the last tile launch took (0 plain, 1 absorbed K, 2 absorbed K and V): the merge kernel has to match it
    float *ubuf = nullptr;
    int abs_max_chunks = 0;
    int last_mode = 0;
    int n_sms = 148;
    // K/V split of small grids: probabilities cross from the K cluster to the V cluster through these
    float *pbuf = nullptr;       // [TC_SPLIT_TILES][n_q_heads][132]
    uint32_t *pflags = nullptr;  // [TC_SPLIT_TILES][n_kv_heads], zero at bind time
    uint32_t epoch = 0;          // launches so far; a flag equal to it belongs to the current launch
    TcLayerCfg layer[TC_MAX_LAYERS];
};

// bytes of the per-layer job tables inside the weights buffer
size_t tc_part_bytes(int n_layers);
// bytes of the probability hand-over area (pbuf then pflags) inside the workspace
size_t tc_split_bytes(const kvcar_config &cfg);
// bytes of the absorbed-score operands inside the workspace (0 if the shape does not take the absorbed form)
size_t tc_absorb_bytes(const kvcar_config &cfg, int max_k_sources, int max_m, int batch, int max_chunks);
// place them: `ws_area` is the device address of that area, `tmap_host`/`tmap_dev` one 128-byte descriptor slot
void tc_setup_absorb(TcState &tc, const kvcar_config &cfg, int max_k_sources, int max_m, int batch, int max_chunks,
                     char *ws_area, char *tmap_host, char *tmap_dev);
// the merge of the tiles after a launch that took the absorbed V form (tc.last_mode == 2)
cudaError_t tc_launch_combine_absorbed(const TcState &tc, const DecodeArgs &a, const SeqList &seqs, cudaStream_t st);

// Build the TMA descriptors and the per-layer job tables into the host image of the
// weights buffer (at tmap_off / part_off) and decide per layer whether the tensor-core
// kernel can run it.  Never fails hard: on any problem the state stays unavailable
// with a reason and the generic kernels run.
void tc_setup(TcState &tc, const kvcar_config &cfg, const LayerPlan *plans_host, int n_layers, char *weights_dev,
              size_t tmap_off, size_t part_off, char *weights_img, size_t pool_rows);
void tc_destroy(TcState &tc);
bool tc_layer_supported(const TcState &tc, int layer);
// lens: host copy of the listed sequences' lengths (same values the device table holds)
// n_launches: kernels enqueued (2 when the absorbed form ran: its operand kernel first)
cudaError_t tc_launch_decode(TcState &tc, const DecodeArgs &a, const SeqList &seqs, const int32_t *lens,
                             int layer, cudaStream_t st, int *n_launches);

// test hook: one warp waits `limit_ns` on a barrier that nothing completes, then records code 0x7e57 in the status word
cudaError_t tc_launch_expire_wait(int32_t *status, uint64_t limit_ns, cudaStream_t st);

}  // namespace kvcar
