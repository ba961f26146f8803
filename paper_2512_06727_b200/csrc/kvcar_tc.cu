// Fused decoder + attention on Blackwell tensor cores (sm_100a): TMA-staged bf16
// operand tiles, tcgen05.mma over a pair of SMs (cta_group::2) with fp32 accumulators
// in tensor memory, restored K/V tiles consumed on the SM without ever reaching HBM.
//
// Work decomposition.  The cached tokens of all listed sequences are cut into tiles
// of 128 tokens; a cluster of two CTAs takes two tiles (any two: the decoder weights
// are shared by every token of the layer) and, optionally, a subset of the layer's KV
// heads.  CTA r owns tile r: its latents, its hidden activations, its scores.  The
// two CTAs issue every matrix product as one M=256 instruction, so each weight tile
// crosses L2 -> shared memory once per 256 tokens, half of it into each CTA.
//
// Per K (then V), per distinct source layer of the heads (own layer, or the root layer
// of a reused head), the cluster walks a host-built job list:
//   hidden chunk  H[256 tok x nc]  = Z[256 tok x d] . W1[nc x d]^T         nc <= 256
//                 a = LeakyReLU(H*s + t) -> bf16 -> shared memory (K-major, 128B swizzle)
//   head group K  Y[256 tok x 64nh] = A[256 tok x m] . W2[64nh x m]^T      nh in {4,2,1}
//                 thread = token: scores of the group's query heads, tile softmax
//   head group V  Y[(4 heads x 64) x 256 tok] = W2[256 x m] . A[256 tok x m]^T
//                 thread = (head, channel): sum over a tile's tokens of p * v
// Each job owns one of two 256-column accumulator buffers in tensor memory, so the
// epilogue of job j overlaps the products of job j+1.  Probabilities of tile r are
// written into both CTAs (distributed shared memory) because the V product of a
// head lands, for both tiles, in the CTA that loaded the head's weight rows.
//
// Grid.  At most one cluster per SM pair; a cluster walks the tile pairs with that
// stride, so loads and products of the next pair start while the epilogues of the
// current one finish.  Small grids spread one tile pair over several clusters: K and V
// on separate clusters (the K cluster publishes each head's probabilities in global
// memory behind a release/acquire flag), and the layer's KV heads in halves or quarters.
//
// Operand staging.  16-KB places: a ring beside the hidden activations, plus, during
// hidden-chunk jobs, the hidden slabs that hold no activations yet.
//
// Builds.  The kernel is a template over two properties of a launch, so that the shapes that need neither carry none
// of the code:
//   GMMA  more than two query heads per KV head: the scores and the weighted values of a group are small matrix
//         products and run on the warp-level tensor op, fed straight from tensor memory in fragment layout;
//         probabilities travel as bf16 rows, to the peer CTA by bulk copies that count their bytes on its barrier.
//   SLAB  every hidden layer is one chunk (<= 256 columns): activations are handed to the second layer's products
//         slab by slab, each source's scale/shift/bias block stays in shared memory, and the next pair's tiles,
//         cache rows and queries are fetched while the current pair's last products run.
//
// Warp roles: warps 0 and 10 = TMA producers (both CTAs; they take alternate loads),
// warp 1 = MMA issuer (leader CTA) and tensor-memory owner, warps 2-9 = epilogue (lane
// quarter = warp % 4, column half = (warp-2) / 4).
//
// All waits are bounded: a wait that runs out records a code in the status word
// and the kernel carries on to its normal exit (results are then meaningless and
// kvcar_sync_status reports KVCAR_ERR_DEVICE_TIMEOUT).
#include <cuda.h>

#include <algorithm>
#include <cstring>
#include <vector>

#include "kvcar_ptx.cuh"
#include "kvcar_tc.h"

namespace kvcar {

using namespace ptx;

namespace {

constexpr int TILE = 128;          // tokens per CTA tile
constexpr int SLOT_BYTES = 16384;  // one operand tile: 128 rows x 128 B
constexpr int HALF_BYTES = 8192;   // 64 rows x 128 B
constexpr int PSTRIDE = 132;       // floats per query head in the score / probability buffer (128 + sum + pad)
constexpr int N_EPI_WARPS = 8;
constexpr int PRODUCER2_WARP = 2 + N_EPI_WARPS;  // second TMA producer, after the epilogue warps
constexpr int NTHREADS = 32 * (PRODUCER2_WARP + 1);
constexpr int MAX_HID_GROUPS = 4;  // hidden chunks of 256 columns
constexpr int QBS = 72;    // bf16 per query row in the MMA-operand copy of the queries (padded against bank conflicts)
constexpr int PBS = 136;   // bf16 per probability row in the MMA-operand copy of the probabilities

struct TileIndex {
    int32_t n_tiles;
    uint32_t first[KVCAR_MAX_BATCH + 1];  // first tile of listed sequence i; first[n] = n_tiles
    int32_t len[KVCAR_MAX_BATCH];         // cached tokens of listed sequence i (the host's copy of the device table)
};

struct PairLaunch {
    const TcPart *parts;  // this layer's tables for the chosen split: parts[0 .. split-1]
    uint32_t off_hidden, off_ring, off_part, off_fparam, off_q, off_s, off_qb, off_pb, off_bar;
    int32_t group_mma;  // query groups of more than two heads: attention products on the warp-level tensor op
    int32_t nslot, max_m, max_in, split, nq_local;
    int32_t n_pairs;  // tile pairs of this launch; a cluster takes pairs first, first + stride, ...
    // K/V split (small grids): one cluster restores K and publishes the probabilities, another restores V
    int32_t kv_split;
    uint32_t epoch;     // value a probability flag takes in this launch
    float *pbuf;        // [tile][hq][PSTRIDE] probabilities (+ sum at 128) in global memory
    uint32_t *pflags;   // [tile][hkv]
    // absorbed K scores (job kind 3): rows of W4_h^T q per (K source, listed sequence, query head), q.b4_h beside them
    const void *tm_wq;  // TMA descriptor: box = 64 columns x nq_pad rows
    const float *qbias; // [source][abs_batch][nq_pad]
    int32_t nq_pad, abs_batch;
    // absorbed V side (job kind 4): sum over a tile's tokens of p * a (a = activated hidden vector) per query head
    float *ubuf;        // [listed sequence][tile][hq][m_pad_u]
    int32_t m_pad_u;
    uint32_t off_pop;   // shared-memory offset of the tile's probabilities as a bf16 column operand (0 = not this form)
};

// ---------------------------------------------------------------------------- waits
// Bounded wait.  `abort_flag` (shared) shortens every later wait once one has failed.
// SLEEP_NS > 0: back off between polls so that a waiting warp leaves the issue slots of its scheduler to the
// warps that share it (the MMA issuer above all).
template <bool CLUSTER = false, int SLEEP_NS = 0>
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, int32_t *status, volatile int *abort_flag,
                                          int code) {
    if (mbar_try<CLUSTER>(bar, parity)) return;
    uint32_t n = 0;
    uint64_t t0 = 0;
    while (true) {
        if (SLEEP_NS > 0) __nanosleep(SLEEP_NS);
        if (mbar_try<CLUSTER>(bar, parity)) return;
        if ((++n & 255u) == 0) {
            uint64_t now = global_ns();
            if (t0 == 0) t0 = now;
            uint64_t limit = *abort_flag ? 2000000ull : 2000000000ull;  // 2 ms after a failure, else 2 s
            if (now - t0 > limit) {
                *abort_flag = 1;
                atomicCAS(status, 0, code);
                return;
            }
        }
    }
}

__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

struct Bars {
    uint32_t full, empty;  // [nslot] each (8 B apart); `full` is used in the leader CTA only
    uint32_t jfull;        // [2] accumulator buffer holds a finished job (both CTAs)
    uint32_t jempty;       // [2] both CTAs' epilogue warps are done reading it (leader)
    uint32_t hid_ready;    // [MAX_AUX] one per 64-column hidden slab: written by both CTAs (leader)
    uint32_t p_ready;      // [1] both CTAs' probabilities of all K heads are in place (both CTAs)
    uint32_t s_free;       // [1] the peer's epilogue warps are done reading a pair's probabilities (both CTAs)
    uint32_t afull, aempty;  // [MAX_AUX] hidden slabs lent to the operand ring while they hold no activations
    uint32_t pb_ready;       // [1] absorbed V: both CTAs' probability operands of the pair are written (leader)
    uint32_t src_done;       // [1] absorbed V: every product that reads the current source's activations is complete
};
constexpr int MAX_AUX = 4 * MAX_HID_GROUPS;
constexpr uint32_t N_FIXED_BARS = 2 + 2 + MAX_AUX + 2 + 2 * MAX_AUX + 2;

struct TileInfo {
    int si, chunk, valid;  // listed-sequence index, tile index inside the sequence, valid tokens (0 = no tile)
};

__device__ __forceinline__ TileInfo locate_tile(const TileIndex &tix, int tile, int n_seqs) {
    TileInfo t{0, 0, 0};
    if (tile >= tix.n_tiles) return t;
    int lo = 0, hi = n_seqs;  // first[lo] <= tile < first[hi]
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (tix.first[mid] <= (uint32_t)tile) lo = mid; else hi = mid;
    }
    t.si = lo;
    t.chunk = tile - (int)tix.first[lo];
    const int L = tix.len[lo];
    t.valid = max(0, min(TILE, L - t.chunk * TILE));
    return t;
}

// head-place fields of a job, picked out of the packed words (no indexed byte arrays in registers)
__device__ __forceinline__ int job_kvh(const TcJob &j, int hp) {
    uint32_t w;
    memcpy(&w, j.kvh, 4);
    return (int)(int8_t)(w >> (8 * hp));
}
__device__ __forceinline__ int job_slot(const TcJob &j, int hp) {
    uint32_t w;
    memcpy(&w, j.slot, 4);
    return (int)(int8_t)(w >> (8 * hp));
}

// one 64-wide K slab: up to four K=16 steps
__device__ __forceinline__ void issue_kslab(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, int nk,
                                            bool first_slab) {
    if (first_slab)
        umma_pair<0>(d_tmem, a_desc, b_desc, idesc);
    else
        umma_pair<1>(d_tmem, a_desc, b_desc, idesc);
    if (nk > 1) umma_pair<1>(d_tmem, a_desc + 2u, b_desc + 2u, idesc);
    if (nk > 2) umma_pair<1>(d_tmem, a_desc + 4u, b_desc + 4u, idesc);
    if (nk > 3) umma_pair<1>(d_tmem, a_desc + 6u, b_desc + 6u, idesc);
}

// ---------------------------------------------------------------------------- optional time stamps
// Compile with -DKVCAR_TC_TRACE to make four threads of one cluster (lane 0 of the two producer warps, of the issuer
// warp and of the first epilogue warp, in both CTAs) record (clock64 << 8) | tag at the points marked TR below;
// kvcar_debug_trace_select picks the cluster, kvcar_debug_trace_dump fetches the records.  Without the macro the
// marks compile to nothing.  Tags: producers 1 = pair begins, 2 = a hidden-chunk slab's two loads issued, 3 = a head
// group slab's load issued; issuer 0x10 | kind = accumulator free, job begins, 0x30 = a slab's operands are in place,
// 0x31 = its products and releases are issued, 0x19 = job committed; epilogue (kind << 4) | phase with kind 4 = hidden
// chunk, 5 = K head group, 6 = V head group and phase 0 = waits for the job, 1 = job seen complete, 2 = accumulator
// read and released, 3 = the job's epilogue is finished.
#ifdef KVCAR_TC_TRACE
constexpr int TRACE_LEN = 4096;
__device__ unsigned long long g_trace[2][4][TRACE_LEN];
__device__ int g_trace_n[2][4];
__device__ int g_trace_cluster = 0;
#define TR(role, tag)                                                                                          \
    do {                                                                                                       \
        if (tr_on) {                                                                                           \
            if (tr_cnt < TRACE_LEN)                                                                            \
                g_trace[rank][role][tr_cnt] = ((unsigned long long)clock64() << 8) | (unsigned)(tag);          \
            ++tr_cnt;                                                                                          \
            g_trace_n[rank][role] = tr_cnt < TRACE_LEN ? tr_cnt : TRACE_LEN;                                   \
        }                                                                                                      \
    } while (0)
#else
#define TR(role, tag) \
    do {              \
    } while (0)
#endif

// ---------------------------------------------------------------------------- the kernel
// GMMA: query groups of more than two heads, whose attention products run on the warp-level tensor op (a separate
// instantiation, so that the code of the other shapes carries none of it)
// SLAB: no hidden layer of the launch is wider than one chunk; its activations are then handed to the second layer's
// products slab by slab (the polls this costs the issuing thread are compiled out otherwise)
template <bool GMMA, bool SLAB>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NTHREADS, 1)
    decode_pair_kernel(const __grid_constant__ DecodeArgs a, const __grid_constant__ SeqList seqs,
                       const __grid_constant__ TileIndex tix, const __grid_constant__ PairLaunch lay) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const uint32_t rank = blockIdx.x & 1u;  // rank in the cluster = which of the pair's two tiles
    const int cid = blockIdx.x >> 1;
    const int per_pair = lay.split * (lay.kv_split ? 2 : 1);  // clusters that share one pair of tiles
    const int sub = cid % per_pair;
    const int pair0 = cid / per_pair, pair_stride = (int)(gridDim.x >> 1) / per_pair;
    const int part_i = sub % lay.split;
    // this cluster's share of the work: K only, V only, or K then V
    const int which_lo = lay.kv_split ? sub / lay.split : 0, which_hi = lay.kv_split ? which_lo + 1 : 2;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int hq = a.hq, group = a.hq / a.hkv;
    const bool leader = rank == 0;
#ifdef KVCAR_TC_TRACE
    const bool tr_on = cid == g_trace_cluster && lane == 0 && (warp <= 2 || warp == PRODUCER2_WARP);
    int tr_cnt = 0;
#endif

    // carve shared memory (1024-byte aligned for the swizzled tiles; same offsets in both CTAs)
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gbase = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t s_hidden = base + lay.off_hidden;
    const uint32_t s_ring = base + lay.off_ring;
    const TcPart &P = *reinterpret_cast<const TcPart *>(gbase + lay.off_part);
    float *fparam = reinterpret_cast<float *>(gbase + lay.off_fparam);  // s1[max_m], t1[max_m], b2[max_in]
    float *qs = reinterpret_cast<float *>(gbase + lay.off_q);          // [nq_local][64], pre-scaled, own tile's sequence
    __nv_bfloat16 *qb = reinterpret_cast<__nv_bfloat16 *>(gbase + lay.off_qb);  // same as bf16 [nq_local][QBS]
    __nv_bfloat16 *Pb = reinterpret_cast<__nv_bfloat16 *>(gbase + lay.off_pb);  // probabilities as bf16 [2][nq_local][PBS]
    float *Sall = reinterpret_cast<float *>(gbase + lay.off_s);        // [2 tiles][nq_local][PSTRIDE]
    const uint32_t s_bar = base + lay.off_bar;
    Bars B;
    B.full = s_bar;
    B.empty = B.full + 8 * lay.nslot;
    B.jfull = B.empty + 8 * lay.nslot;
    B.jempty = B.jfull + 16;
    B.hid_ready = B.jempty + 16;
    B.p_ready = B.hid_ready + 8 * MAX_AUX;
    B.s_free = B.p_ready + 8;
    B.afull = B.s_free + 8;
    B.aempty = B.afull + 8 * MAX_AUX;
    B.pb_ready = B.aempty + 8 * MAX_AUX;
    B.src_done = B.pb_ready + 8;

    {  // this cluster's job tables -> shared memory
        const uint4 *src = reinterpret_cast<const uint4 *>(lay.parts + part_i);
        uint4 *dst = reinterpret_cast<uint4 *>(gbase + lay.off_part);
        for (int i = threadIdx.x; i < (int)(sizeof(TcPart) / 16); i += NTHREADS) dst[i] = src[i];
    }
    if (lay.off_pop)  // the probability operand's padding rows are never written: they must hold finite values
        for (int i = threadIdx.x; i < lay.nq_pad * 256 / 16; i += NTHREADS)
            reinterpret_cast<uint4 *>(gbase + lay.off_pop)[i] = make_uint4(0u, 0u, 0u, 0u);
    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int i = 0; i < lay.nslot; ++i) {
            mbar_init(B.full + 8 * i, 1);
            mbar_init(B.empty + 8 * i, 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(B.jfull + 8 * i, 1);
            mbar_init(B.jempty + 8 * i, 2 * N_EPI_WARPS);
        }
        for (int i = 0; i < MAX_AUX; ++i) mbar_init(B.hid_ready + 8 * i, 2 * N_EPI_WARPS);
        mbar_init(B.p_ready, GMMA ? N_EPI_WARPS : 2 * N_EPI_WARPS);
        mbar_init(B.s_free, N_EPI_WARPS);
        for (int i = 0; i < MAX_AUX; ++i) {
            mbar_init(B.afull + 8 * i, 1);
            mbar_init(B.aempty + 8 * i, 1);
        }
        mbar_init(B.pb_ready, 2 * N_EPI_WARPS);
        mbar_init(B.src_done, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {  // tensor memory: all 512 columns in both CTAs of the pair (one CTA per SM by shared memory)
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                     "r"(512u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // the peer's barriers and job tables exist before anyone signals or issues
    tc_fence_after();
    const uint32_t tmem = tmem_base_slot;
    const int h_lo = P.h_lo;

    if (warp == 0 || warp == PRODUCER2_WARP) {
        // ============================== TMA producers (both CTAs) ==============================
        // Two warps share the loads (issuing one tensor load costs its thread ~100 cycles): the loads of the job
        // list are numbered and producer `pid` issues those of its parity.  Both walk the same sequence of
        // places and wait for each of them to be free, so both see the same ring state.
        const uint32_t pid = warp == 0 ? 0u : 1u;
        if (elect_one()) {
            uint32_t slot = 0, phase = 0, aux_phase = 0, turn = 0, src_par = 0;
            // Absorbed V launches: the job that reads a source's activations last stages nothing in the ring, so a free
            // ring slot no longer proves that it is complete; the issuer signals src_done once per source instead and
            // every producer waits for it once before it stages over the hidden slabs of the next source.
            bool src_wait_due = false;
            auto src_wait = [&]() {
                mbar_wait(B.src_done, src_par ^ 1u, a.status, &abort_flag, 0x104);
                src_par ^= 1u;
                src_wait_due = false;
            };
          for (int pair = pair0; pair < lay.n_pairs; pair += pair_stride) {
            const TileInfo mine = locate_tile(tix, 2 * pair + (int)rank, seqs.n);
            TR(pid, 1);
            // pool rows of the tile's two 64-token halves (a half with no valid token re-reads a valid row block)
            int row[2] = {0, 0};
            if (mine.valid > 0) {
                const int seq = seqs.id[mine.si];
                for (int h = 0; h < 2; ++h) {
                    int t = mine.chunk * TILE + 64 * h;
                    if (64 * h >= mine.valid) t = mine.chunk * TILE;
                    const int page = a.block_table[(int64_t)seq * a.max_pages_per_seq + t / a.page_tokens];
                    row[h] = page * a.page_tokens + t % a.page_tokens;
                }
            }
            // wait for the ring slot to be free in this CTA; its owner announces the pair's bytes (leader)
            auto acquire = [&](uint32_t pair_bytes, bool own) -> uint32_t {
                mbar_wait(B.empty + 8 * slot, phase ^ 1u, a.status, &abort_flag, 0x101);
                if (own && leader) mbar_expect_tx(B.full + 8 * slot, pair_bytes);
                const uint32_t s = slot;
                if (++slot == (uint32_t)lay.nslot) { slot = 0; phase ^= 1u; }
                return s;
            };
            // Hidden-chunk jobs also stage operands in the hidden slabs that hold no activations yet (those of
            // this chunk and of later chunks): the ring alone is too shallow for the L2 latency at their rate.
            // A job takes the ring slots first and both producers wait for every place, so every product that
            // read the previous source's activations is known to be done (its ring slots have been seen free:
            // completions arrive in issue order) before the first hidden slab is overwritten.
            const int ks_hid = (lay.max_m + 63) >> 6;
            for (int which = 0; which < 2; ++which) {  // constant trip count: `which` folds into the code below
                if (which < which_lo || which >= which_hi) continue;
                const int nj = P.n_jobs[which];
                for (int j = 0; j < nj; ++j) {
                    const TcJob job = P.jobs[which][j];
                    const TcSrc &sp = P.src[which][job.src];
                    if (job.kind == 1) {
                        const int ks1 = (sp.d + 63) >> 6;
                        const int half_rows = job.nc >> 1;  // weight rows this CTA supplies
                        const int y0 = job.c0 + (int)rank * half_rows;
                        const int aux_lo = job.c0 >> 6, n_pool = lay.nslot + (ks_hid - aux_lo);
                        int r = 0;
                        if (lay.off_pop && (job.first & 1)) src_wait_due = true;
                        // next staging place of this job: smem address in `dst`, leader's full barrier in `fb`
                        auto acquire1 = [&](uint32_t pair_bytes, bool own, uint32_t &dst, uint32_t &fb) {
                            if (r < lay.nslot) {
                                const uint32_t sl = acquire(pair_bytes, own);
                                dst = s_ring + sl * SLOT_BYTES;
                                fb = map_to_cta(B.full + 8 * sl, 0);
                            } else {
                                const uint32_t x = (uint32_t)(aux_lo + r - lay.nslot);
                                if (src_wait_due) src_wait();
                                mbar_wait(B.aempty + 8 * x, ((aux_phase >> x) & 1u) ^ 1u, a.status, &abort_flag, 0x103);
                                if (own && leader) mbar_expect_tx(B.afull + 8 * x, pair_bytes);
                                aux_phase ^= 1u << x;
                                dst = s_hidden + x * SLOT_BYTES;
                                fb = map_to_cta(B.afull + 8 * x, 0);
                            }
                            if (++r == n_pool) r = 0;
                        };
                        for (int ks = 0; ks < ks1; ++ks) {
                            uint32_t dst, fb;
                            bool own = turn == pid;
                            turn ^= 1u;
                            acquire1(2 * SLOT_BYTES, own, dst, fb);
                            if (own) {
                                tma_load_2d_pair(dst, sp.tm_pool, ks * 64, row[0], fb);
                                tma_load_2d_pair(dst + HALF_BYTES, sp.tm_pool, ks * 64, row[1], fb);
                            }
                            own = turn == pid;
                            turn ^= 1u;
                            acquire1(half_rows > 64 ? 2 * SLOT_BYTES : 2 * HALF_BYTES, own, dst, fb);
                            if (own) {
                                tma_load_2d_pair(dst, sp.tm_w1, ks * 64, y0, fb);
                                if (half_rows > 64) tma_load_2d_pair(dst + HALF_BYTES, sp.tm_w1, ks * 64, y0 + 64, fb);
                            }
                            TR(pid, 2);
                        }
                        if (src_wait_due) src_wait();  // no lent slab was visited: the wait is owed once per source
                    } else if (job.kind == 4) {
                        // absorbed V: both operands are already in shared memory (activations, probabilities)
                    } else if (job.kind == 3) {
                        // absorbed scores: the column operand is this tile's sequence's W4_h^T q rows (all query heads)
                        const int ks2 = (sp.m + 63) >> 6;
                        const int y = ((int)job.src * lay.abs_batch + mine.si) * lay.nq_pad;
                        const uint32_t slab_bytes = (uint32_t)lay.nq_pad * 128u;  // one K slab of this CTA's rows
                        const int per_place = SLOT_BYTES / (int)slab_bytes;        // K slabs staged behind one barrier
                        for (int ks0 = 0; ks0 < ks2; ks0 += per_place) {
                            const int n = min(per_place, ks2 - ks0);
                            const bool own = turn == pid;
                            turn ^= 1u;
                            const uint32_t sl = acquire(2u * slab_bytes * (uint32_t)n, own);
                            if (own) {
                                const uint32_t fb = map_to_cta(B.full + 8 * sl, 0);
                                for (int i = 0; i < n; ++i)
                                    tma_load_2d_pair(s_ring + sl * SLOT_BYTES + (uint32_t)i * slab_bytes, lay.tm_wq,
                                                     (ks0 + i) * 64, y, fb);
                            }
                            TR(pid, 3);
                        }
                    } else {
                        const int ks2 = (sp.m + 63) >> 6;
                        int ya, yb = -1;  // first rows of the one or two 64-row boxes this CTA supplies
                        if (which == 1 || job.nh == 4) {
                            const int sa = job.slot[2 * rank], sb = job.slot[2 * rank + 1];
                            ya = 64 * sa;
                            yb = 64 * sb;
                        } else if (job.nh == 2) {
                            ya = 64 * job.slot[rank];
                        } else {
                            ya = 64 * job.slot[0] + 32 * (int)rank;
                        }
                        for (int ks = 0; ks < ks2; ++ks) {
                            const bool own = turn == pid;
                            turn ^= 1u;
                            const uint32_t sl = acquire(yb >= 0 ? 2 * SLOT_BYTES : 2 * HALF_BYTES, own);
                            if (own) {
                                const uint32_t fb = map_to_cta(B.full + 8 * sl, 0);
                                tma_load_2d_pair(s_ring + sl * SLOT_BYTES, sp.tm_w2, ks * 64, ya, fb);
                                if (yb >= 0)
                                    tma_load_2d_pair(s_ring + sl * SLOT_BYTES + HALF_BYTES, sp.tm_w2, ks * 64, yb, fb);
                            }
                            TR(pid, 3);
                        }
                    }
                }
            }
          }  // pairs
        }
    } else if (warp == 1) {
        // ============================== MMA issuer (leader CTA) ==============================
        // One elected lane walks the job list and issues (the compiler then knows the branch holds a single thread
        // and keeps descriptors and barrier addresses in uniform registers).
        if (leader && elect_one()) {
            constexpr bool issuer = true;
            uint32_t slot = 0, phase = 0, jc = 0, hid_phase = 0, aux_phase = 0, pair_it = 0;
            const int ks_hid = (lay.max_m + 63) >> 6;
            auto wait_full = [&]() -> uint32_t {
                mbar_wait(B.full + 8 * slot, phase, a.status, &abort_flag, 0x201);
                const uint32_t s = slot;
                if (++slot == (uint32_t)lay.nslot) { slot = 0; phase ^= 1u; }
                return s;
            };
          for (int pair = pair0; pair < lay.n_pairs; pair += pair_stride, ++pair_it) {
            bool pb_seen = false;
            for (int which = 0; which < 2; ++which) {  // constant trip count: `which` folds into the code below
                if (which < which_lo || which >= which_hi) continue;
                const int nj = P.n_jobs[which];
                for (int j = 0; j < nj; ++j, ++jc) {
                    const TcJob job = P.jobs[which][j];
                    const TcSrc &sp = P.src[which][job.src];
                    const int d = sp.d, m = sp.m;
                    const uint32_t buf = jc & 1u;
                    const uint32_t acc = tmem + 256u * buf;
                    mbar_wait(B.jempty + 8 * buf, ((jc >> 1) & 1u) ^ 1u, a.status, &abort_flag, 0x202);
                    tc_fence_after();
                    TR(2, 0x10 | job.kind);
                    if (job.kind == 1) {
                        const int ks1 = (d + 63) >> 6;
                        const uint32_t idesc = make_idesc(256, job.nc);
                        const int aux_lo = job.c0 >> 6, n_pool = lay.nslot + (ks_hid - aux_lo);
                        int r = 0;
                        // next staging place of this job (same order as the producer): smem address, its empty barrier
                        auto wait_full1 = [&](uint32_t &addr, uint32_t &ebar) {
                            if (r < lay.nslot) {
                                const uint32_t sl = wait_full();
                                addr = s_ring + sl * SLOT_BYTES;
                                ebar = B.empty + 8 * sl;
                            } else {
                                const uint32_t x = (uint32_t)(aux_lo + r - lay.nslot);
                                mbar_wait(B.afull + 8 * x, (aux_phase >> x) & 1u, a.status, &abort_flag, 0x205);
                                aux_phase ^= 1u << x;
                                addr = s_hidden + x * SLOT_BYTES;
                                ebar = B.aempty + 8 * x;
                            }
                            if (++r == n_pool) r = 0;
                        };
                        for (int ks = 0; ks < ks1; ++ks) {
                            uint32_t az, ez, aw, ew2;
                            wait_full1(az, ez);
                            wait_full1(aw, ew2);
                            tc_fence_after();
                            TR(2, 0x30);
                            if (issuer) {
                                issue_kslab(acc, make_desc(az), make_desc(aw), idesc, min(4, (d - 64 * ks) >> 4), ks == 0);
                                umma_commit_pair(ez);
                                umma_commit_pair(ew2);
                            }
                            TR(2, 0x31);
                        }
                    } else if (job.kind == 4) {
                        // absorbed V: U[feature][query] = sum over the tile's tokens of a[token][feature] * p[query][token].
                        // Row operand = the hidden slabs read feature-major (each holds [token][64 features], i.e. an
                        // MN-major tile: 64-feature atoms SLOT_BYTES apart, 8-token groups 1 KB apart); column operand =
                        // this CTA's probabilities [query][token] in two 64-token atoms.  Each CTA supplies its own
                        // tile's activations and probabilities, so its accumulator's own column block is its tile's U;
                        // 128 features per product and CTA, all feature chunks side by side in one accumulator buffer
                        // (an odd slab count repeats the second-to-last slab in the last chunk).
                        const int ks2 = (m + 63) >> 6;
                        constexpr bool slabwise = SLAB;
                        for (int ks = 0; ks < ks2; ++ks)
                            if (slabwise || (ks & 3) == 0) {
                                const int ws = slabwise ? ks : min(ks + 3, ks2 - 1);
                                mbar_wait(B.hid_ready + 8 * ws, (hid_phase >> ws) & 1u, a.status, &abort_flag, 0x204);
                                hid_phase ^= 1u << ws;
                            }
                        if (!pb_seen) {
                            mbar_wait(B.pb_ready, pair_it & 1u, a.status, &abort_flag, 0x207);
                            pb_seen = true;
                        }
                        tc_fence_after();
                        TR(2, 0x30);
                        const uint32_t idesc = make_idesc(256, 2 * lay.nq_pad) | (1u << 15);  // row operand MN-major
                        const uint32_t s_pop = base + lay.off_pop;
                        const int n_ch = (ks2 + 1) >> 1;
                        for (int c = 0; c < n_ch; ++c) {
                            const int sa = min(2 * c, ks2 - 2);
                            uint64_t da = make_desc(s_hidden + sa * SLOT_BYTES);
                            da = (da & ~((uint64_t)0x3FFF << 16)) | ((uint64_t)(SLOT_BYTES >> 4) << 16);  // leading (feature-atom) stride
                            const uint32_t acc_c = acc + (uint32_t)(c * 2 * lay.nq_pad);
#pragma unroll
                            for (int t = 0; t < TILE / 16; ++t) {
                                const uint64_t a_t = da + (uint64_t)(t * (16 * 128 >> 4));
                                const uint64_t b_t = make_desc(s_pop + (uint32_t)((t >> 2) * lay.nq_pad * 128)) + (uint64_t)((t & 3) * 2);
                                if (t == 0)
                                    umma_pair<0>(acc_c, a_t, b_t, idesc);
                                else
                                    umma_pair<1>(acc_c, a_t, b_t, idesc);
                            }
                        }
                        TR(2, 0x31);
                    } else if (job.kind == 3) {
                        // absorbed scores: the whole job's column operand is a few KB, so several K slabs share a place
                        // and a barrier round; the waits for the activations are those of a first head group
                        const int ks2 = (m + 63) >> 6;
                        const uint32_t idesc = make_idesc(256, 2 * lay.nq_pad);
                        const uint32_t slab_bytes = (uint32_t)lay.nq_pad * 128u;
                        const int per_place = SLOT_BYTES / (int)slab_bytes;
                        constexpr bool slabwise = SLAB;
                        for (int ks0 = 0; ks0 < ks2; ks0 += per_place) {
                            const int n = min(per_place, ks2 - ks0);
                            for (int ks = ks0; ks < ks0 + n; ++ks)
                                if (slabwise || (ks & 3) == 0) {
                                    const int ws = slabwise ? ks : min(ks + 3, ks2 - 1);
                                    mbar_wait(B.hid_ready + 8 * ws, (hid_phase >> ws) & 1u, a.status, &abort_flag, 0x204);
                                    hid_phase ^= 1u << ws;
                                }
                            const uint32_t sw = wait_full();
                            tc_fence_after();
                            TR(2, 0x30);
                            for (int i = 0; i < n; ++i) {
                                const int ks = ks0 + i;
                                issue_kslab(acc, make_desc(s_hidden + ks * SLOT_BYTES),
                                            make_desc(s_ring + sw * SLOT_BYTES + (uint32_t)i * slab_bytes), idesc,
                                            min(4, (m - 64 * ks) >> 4), ks == 0);
                            }
                            umma_commit_pair(B.empty + 8 * sw);
                            TR(2, 0x31);
                        }
                    } else {
                        const int ks2 = (m + 63) >> 6;
                        const uint32_t idesc = which == 0 ? make_idesc(256, 64 * job.nh) : make_idesc(256, 256);
                        const bool first_use = (job.first & 1) != 0;  // first head group of this source
                        constexpr bool slabwise = SLAB;
                        for (int ks = 0; ks < ks2; ++ks) {
                            if (first_use) {
                                // Hidden layers of one chunk are announced slab by slab (nothing else hides their
                                // epilogue); each poll costs tensor time, so wider ones are waited for chunk by chunk,
                                // through the chunk's last slab.
                                if (slabwise || (ks & 3) == 0) {
                                    const int ws = slabwise ? ks : min(ks + 3, ks2 - 1);
                                    mbar_wait(B.hid_ready + 8 * ws, (hid_phase >> ws) & 1u, a.status, &abort_flag, 0x204);
                                    hid_phase ^= 1u << ws;
                                }
                            }
                            const uint32_t sw = wait_full();
                            tc_fence_after();
                            TR(2, 0x30);
                            const uint64_t dh = make_desc(s_hidden + ks * SLOT_BYTES);
                            const uint64_t dw = make_desc(s_ring + sw * SLOT_BYTES);
                            const int nk = min(4, (m - 64 * ks) >> 4);
                            if (issuer) {
                                if (which == 0)
                                    issue_kslab(acc, dh, dw, idesc, nk, ks == 0);
                                else
                                    issue_kslab(acc, dw, dh, idesc, nk, ks == 0);
                                umma_commit_pair(B.empty + 8 * sw);
                            }
                            TR(2, 0x31);
                        }
                    }
                    if (issuer) umma_commit_pair(B.jfull + 8 * buf);
                    // absorbed V launches: last job of its source - its completion frees the hidden slabs for staging
                    if (lay.off_pop && (job.first & 2)) umma_commit_pair(B.src_done);
                    TR(2, 0x19);
                }
            }
          }  // pairs
        }
    } else if (warp < PRODUCER2_WARP) {
        // ============================== epilogue warps (both CTAs) ==============================
        const int et = threadIdx.x - 64;              // 0..255
        const int ew = warp - 2;                      // 0..7
        const int chalf = ew >> 2;                    // which half of a job's columns this warp reads
        const uint32_t lane_base = 32u * (warp & 3);  // TMEM lane quarter this warp may read
        const int row = lane_base + lane;             // accumulator row of this thread
        const uint32_t tl_addr = lane_base << 16;
        const int m_pad = (lay.max_m + 31) & ~31;  // scale/shift rows are read in whole 32-column groups
        float *s1 = fparam, *t1 = fparam + m_pad, *b2 = fparam + 2 * m_pad;  // SLAB builds: re-pointed per source
        const uint32_t jempty_leader[2] = {map_to_cta(B.jempty, 0), map_to_cta(B.jempty + 8, 0)};
        const uint32_t hid_leader = map_to_cta(B.hid_ready, 0);
        const int nq_part = (P.h_hi - h_lo) * group;
        const uint32_t ginv = 65536u / (uint32_t)group + 1u;  // (i * ginv) >> 16 == i / group for the small i used here
        uint32_t jc = 0, it = 0;
        TileInfo tl_next[2] = {};
        bool next_ready = false;  // tl_next and the queries in shared memory belong to the coming pair
      for (int pair = pair0; pair < lay.n_pairs; pair += pair_stride, ++it) {
        // With small autoencoders the start of a pair (finding the tiles, fetching the queries) is a visible share of
        // the pair's time: there it is done for the next pair while this pair's last products run (SLAB builds).
        TileInfo tl[2];
        if (SLAB && next_ready) {
            tl[0] = tl_next[0];
            tl[1] = tl_next[1];
        } else {
            tl[0] = locate_tile(tix, 2 * pair, seqs.n);
            tl[1] = locate_tile(tix, 2 * pair + 1, seqs.n);
        }
        const TileInfo mine = tl[rank];
        bool s_waited = it == 0;  // the peer has finished reading the previous pair's probabilities in its buffer
        const uint32_t peer_S = map_to_cta(smem_u32(Sall), rank ^ 1u);
        const uint32_t peer_Pb = map_to_cta(smem_u32(Pb), rank ^ 1u);
        const uint32_t peer_pready = map_to_cta(B.p_ready, rank ^ 1u);
        float *Smine = Sall + (size_t)rank * lay.nq_local * PSTRIDE;
        // pull a tile's latent rows of every source from HBM into L2 ahead of the producers' loads
        auto prefetch_rows = [&](const TileInfo &t_) {
            int item = 0;
            for (int which = which_lo; which < which_hi; ++which)
                for (int sidx = 0; sidx < P.n_src[which]; ++sidx) {
                    const TcSrc &sp = P.src[which][sidx];
                    const int n = 2 * ((sp.d + 63) >> 6);
                    if (et >= item && et < item + n) {
                        const int i = et - item, h = i & 1;
                        if (64 * h < t_.valid) {
                            const int t = t_.chunk * TILE + 64 * h;
                            const int page = a.block_table[(int64_t)seqs.id[t_.si] * a.max_pages_per_seq + t / a.page_tokens];
                            tma_prefetch_2d(sp.tm_pool, (i >> 1) * 64, page * a.page_tokens + t % a.page_tokens);
                        }
                    }
                    item += n;
                }
        };
        // eight query elements (16 B) per thread and turn: scaled, to fp32 (and to bf16 rows for the tensor op)
        auto q_store = [&](int i, const uint4 &raw) {
            const __nv_bfloat162 *h2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
            float2 f[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                f[u] = __bfloat1622float2(h2[u]);
                f[u].x *= a.scale;
                f[u].y *= a.scale;
            }
            *reinterpret_cast<float4 *>(qs + i) = make_float4(f[0].x, f[0].y, f[1].x, f[1].y);
            *reinterpret_cast<float4 *>(qs + i + 4) = make_float4(f[2].x, f[2].y, f[3].x, f[3].y);
            if (GMMA)
                *reinterpret_cast<uint4 *>(qb + (i >> 6) * QBS + (i & 63)) =
                    make_uint4(pack_bf16(f[0].x, f[0].y), pack_bf16(f[1].x, f[1].y), pack_bf16(f[2].x, f[2].y),
                               pack_bf16(f[3].x, f[3].y));
        };
        if (SLAB && next_ready) {
            epi_bar_sync();  // the queries stored during the previous pair are visible to every warp
        } else if (mine.valid > 0) {
            prefetch_rows(mine);
            const __nv_bfloat16 *qg =
                reinterpret_cast<const __nv_bfloat16 *>(a.q) + ((int64_t)mine.si * hq + h_lo * group) * 64;
            for (int i = 8 * et; i < nq_part * 64; i += 8 * 256) q_store(i, __ldg(reinterpret_cast<const uint4 *>(qg + i)));
        }
        next_ready = false;
        for (int which = 0; which < 2; ++which) {  // constant trip count: `which` folds into the code below
                if (which < which_lo || which >= which_hi) continue;
            const int nj = P.n_jobs[which];
            if (which == 1 && lay.off_pop) {
                // absorbed V: this warp's rows of the probability operand are written; the products read them
                // through the asynchronous proxy
                fence_async_smem();
                __syncwarp();
                if (elect_one()) mbar_arrive_remote(map_to_cta(B.pb_ready, 0));
            }
            if (which == 1 && !lay.kv_split) {
                if (GMMA) {
                    // this warp's probabilities are in place here; the peer's arrive as counted bytes, announced by one warp
                    __syncwarp();
                    if (elect_one()) {
                        if (ew == 0 && tl[rank ^ 1u].valid > 0)
                            mbar_expect_tx(B.p_ready, (uint32_t)nq_part * PBS * 2u);  // whole rows, see the softmax
                        else
                            mbar_arrive_local(B.p_ready);
                    }
                } else {
                    // every probability this CTA will read has been written, here and by the peer
                    asm volatile("fence.acq_rel.cluster;" ::: "memory");
                    __syncwarp();
                    if (elect_one()) {
                        mbar_arrive_cluster(map_to_cta(B.p_ready, 0));
                        mbar_arrive_cluster(map_to_cta(B.p_ready, 1));
                    }
                }
            }
            bool p_waited = false;
            for (int j = 0; j < nj; ++j, ++jc) {
                const TcJob job = P.jobs[which][j];
                const TcSrc &sp = P.src[which][job.src];
                const int m = sp.m;
                const uint32_t buf = jc & 1u;
                const uint32_t acc = tmem + 256u * buf + tl_addr;
                if (SLAB) {  // one parameter block per source, filled during the cluster's first pair
                    const int pslot = which * P.n_src[0] + job.src;
                    s1 = fparam + (size_t)pslot * (2 * m_pad + lay.max_in);
                    t1 = s1 + m_pad;
                    b2 = s1 + 2 * m_pad;
                }
                if (job.kind == 1) {
                    if ((job.first & 1) && (!SLAB || it == 0)) {
                        // this source's parameters: fetched into registers first, so that the global-memory
                        // latency overlaps the wait for the other warps
                        float ps[MAX_HID_GROUPS], pt[MAX_HID_GROUPS], pb[MAX_HID_GROUPS];
#pragma unroll
                        for (int u = 0; u < MAX_HID_GROUPS; ++u) {
                            const int i = et + 256 * u;
                            ps[u] = i < m ? sp.s1[i] : 0.f;
                            pt[u] = i < m ? sp.t1[i] : 0.f;
                            pb[u] = i < sp.in_dim ? sp.b2[i] : 0.f;
                        }
                        epi_bar_sync();  // everyone is done with the previous source's parameters
#pragma unroll
                        for (int u = 0; u < MAX_HID_GROUPS; ++u) {
                            const int i = et + 256 * u;
                            if (i < m_pad) {
                                s1[i] = ps[u];
                                t1[i] = pt[u];
                            }
                            if (i < sp.in_dim) b2[i] = pb[u];
                        }
                        epi_bar_sync();
                    }
                    // ---- bias + BatchNorm + LeakyReLU, bf16, into the swizzled hidden slabs ----
                    const float2 slope2 = make_float2(sp.slope, sp.slope);
                    const bool lr_max = sp.slope <= 1.f;
                    TR(3, 0x40);
                    mbar_wait<false, 100>(B.jfull + 8 * buf, (jc >> 1) & 1u, a.status, &abort_flag, 0x301);
                    tc_fence_after();
                    TR(3, 0x41);
                    // One 64-column slab at a time, this warp its half of it.  A hidden layer of a single chunk announces
                    // each slab as soon as it is written, so that the second layer's products start under the rest of
                    // this epilogue; a wider one announces each chunk once, through its last slab.
                    const int ngroups = (job.nc + 31) >> 5, nslabs = (job.nc + 63) >> 6;
                    constexpr bool slabwise = SLAB;
                    for (int sl = 0; sl < nslabs; ++sl) {
                        const int g = 2 * sl + chalf;
                        if (g < ngroups) {
                        float v[32];
                        tmem_ld32(acc + 32u * g, v);
                        tmem_ld_wait();
                        const int col0 = job.c0 + 32 * g;
                        const float4 *s4 = reinterpret_cast<const float4 *>(s1 + col0);  // padded to 32 columns
                        const float4 *t4 = reinterpret_cast<const float4 *>(t1 + col0);
#pragma unroll
                        for (int q8 = 0; q8 < 8; ++q8) {
                            const float4 sv = s4[q8], tv = t4[q8];
                            const float2 x0 = __ffma2_rn(make_float2(v[4 * q8], v[4 * q8 + 1]), make_float2(sv.x, sv.y),
                                                         make_float2(tv.x, tv.y));
                            const float2 x1 = __ffma2_rn(make_float2(v[4 * q8 + 2], v[4 * q8 + 3]),
                                                         make_float2(sv.z, sv.w), make_float2(tv.z, tv.w));
                            const float2 y0 = __fmul2_rn(x0, slope2), y1 = __fmul2_rn(x1, slope2);
                            // LeakyReLU: the larger of x and slope*x for slope <= 1, the smaller for slope > 1
                            v[4 * q8 + 0] = lr_max ? fmaxf(x0.x, y0.x) : fminf(x0.x, y0.x);
                            v[4 * q8 + 1] = lr_max ? fmaxf(x0.y, y0.y) : fminf(x0.y, y0.y);
                            v[4 * q8 + 2] = lr_max ? fmaxf(x1.x, y1.x) : fminf(x1.x, y1.x);
                            v[4 * q8 + 3] = lr_max ? fmaxf(x1.y, y1.y) : fminf(x1.y, y1.y);
                        }
                        // 32 columns = 4 chunks of 16 B inside slab (col0 / 64)
                        const uint32_t slab = s_hidden + (uint32_t)(col0 >> 6) * SLOT_BYTES + (uint32_t)row * 128u;
                        const int ch0 = (col0 & 63) >> 3;
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4) {
                            if (col0 + 8 * q4 < m) {
                                const uint32_t w0 = pack_bf16(v[8 * q4 + 0], v[8 * q4 + 1]);
                                const uint32_t w1 = pack_bf16(v[8 * q4 + 2], v[8 * q4 + 3]);
                                const uint32_t w2 = pack_bf16(v[8 * q4 + 4], v[8 * q4 + 5]);
                                const uint32_t w3 = pack_bf16(v[8 * q4 + 6], v[8 * q4 + 7]);
                                const uint32_t addr = slab + (uint32_t)(((ch0 + q4) ^ (row & 7)) << 4);
                                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(w0), "r"(w1),
                                             "r"(w2), "r"(w3)
                                             : "memory");
                            }
                        }
                        }
                        if (slabwise) {
                            fence_async_smem();
                            __syncwarp();
                            if (elect_one()) mbar_arrive_remote(hid_leader + 8u * (uint32_t)((job.c0 >> 6) + sl));
                        }
                    }
                    tc_fence_before();
                    if (!slabwise) fence_async_smem();
                    __syncwarp();
                    if (elect_one()) {
                        mbar_arrive_remote(jempty_leader[buf]);
                        if (!slabwise) mbar_arrive_remote(hid_leader + 8u * (uint32_t)((job.c0 >> 6) + nslabs - 1));
                    }
                    TR(3, 0x43);
                    continue;
                }
                // ---- head group ----
                if (which == 1 && lay.kv_split) {
                    // fetch the probabilities of this job's heads, both tiles, from the K cluster (global memory):
                    // wait for each row's flag, copy the row into this CTA's buffer
                    const int rows_per_tile = 4 * group, n_vec = 2 * rows_per_tile * (PSTRIDE / 4);
                    for (int idx = et; idx < n_vec; idx += 256) {
                        const int rrow = idx / (PSTRIDE / 4), v4 = idx % (PSTRIDE / 4);
                        const int th = rrow / rows_per_tile, hp = (rrow % rows_per_tile) / group, g = rrow % group;
                        const int kvh = job_kvh(job, hp);
                        if (kvh < 0 || tl[th].valid == 0) continue;
                        const int tile = 2 * pair + th;
                        const uint32_t *fl = lay.pflags + (size_t)tile * a.hkv + kvh;
                        uint32_t seen = 0, n = 0;
                        uint64_t t0 = 0;
                        while (true) {
                            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(fl) : "memory");
                            if (seen == lay.epoch) break;
                            __nanosleep(200);
                            if ((++n & 63u) == 0) {  // bounded like every other wait of this kernel
                                const uint64_t now = global_ns();
                                if (t0 == 0) t0 = now;
                                if (now - t0 > (abort_flag ? 2000000ull : 2000000000ull)) {
                                    abort_flag = 1;
                                    atomicCAS(a.status, 0, 0x304);
                                    break;
                                }
                            }
                        }
                        const int ql = (kvh - h_lo) * group + g;
                        const float4 val = __ldcg(reinterpret_cast<const float4 *>(
                                                      lay.pbuf + ((size_t)tile * hq + h_lo * group + ql) * PSTRIDE) + v4);
                        *reinterpret_cast<float4 *>(Sall + ((size_t)th * lay.nq_local + ql) * PSTRIDE + 4 * v4) = val;
                        if (GMMA) {
                            __nv_bfloat16 *prow = Pb + ((size_t)th * lay.nq_local + ql) * PBS;
                            if (v4 < 32)
                                *reinterpret_cast<uint2 *>(prow + 4 * v4) =
                                    make_uint2(pack_bf16(val.x, val.y), pack_bf16(val.z, val.w));
                            else
                                *reinterpret_cast<float *>(prow + 128) = val.x;  // the row's sum
                        }
                    }
                    epi_bar_sync();
                }
                uint4 qraw[2];
                bool q_held = false;
                if (SLAB && which == 1 && !lay.kv_split && !next_ready && nq_part <= 64) {
                    const int np = pair + pair_stride;
                    if (np < lay.n_pairs) {
                        tl_next[0] = locate_tile(tix, 2 * np, seqs.n);
                        tl_next[1] = locate_tile(tix, 2 * np + 1, seqs.n);
                        next_ready = true;
                        const TileInfo nm = tl_next[rank];
                        if (nm.valid > 0) {
                            prefetch_rows(nm);
                            const __nv_bfloat16 *qg =
                                reinterpret_cast<const __nv_bfloat16 *>(a.q) + ((int64_t)nm.si * hq + h_lo * group) * 64;
#pragma unroll
                            for (int u = 0; u < 2; ++u) {
                                const int i = 8 * et + 2048 * u;
                                if (i < nq_part * 64) qraw[u] = __ldg(reinterpret_cast<const uint4 *>(qg + i));
                            }
                            q_held = true;
                        }
                    }
                }
                TR(3, 0x50 + 0x10 * which);
                mbar_wait<false, 100>(B.jfull + 8 * buf, (jc >> 1) & 1u, a.status, &abort_flag, 0x302);
                tc_fence_after();
                TR(3, 0x51 + 0x10 * which);
                if (SLAB && q_held) {  // every warp is past this pair's scores: the query rows are free
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const int i = 8 * et + 2048 * u;
                        if (i < nq_part * 64) q_store(i, qraw[u]);
                    }
                }
                if (which == 0) {
                    // K: this thread owns token `row` of this CTA's tile; columns = (head place, channel)
                    const int nh = job.nh;
                    if (job.kind == 3) {
                        // absorbed scores: the accumulator already holds a.(W4_h^T q) for every query head of both
                        // tiles' sequences; this CTA's sequence owns columns [nq_pad * rank, nq_pad * (rank + 1))
                        const int half = lay.nq_pad >> 1;
                        const uint32_t mask = (uint32_t)job.c0 | ((uint32_t)job.nc << 16);
                        const float *qb_ = lay.qbias + ((size_t)job.src * lay.abs_batch + mine.si) * lay.nq_pad;
                        for (int c8 = 0; c8 < half; c8 += 8) {
                            const int c_lo = chalf * half + c8;
                            float sc[8];
                            tmem_ld8(acc + (uint32_t)(lay.nq_pad * (int)rank + c_lo), sc);
                            tmem_ld_wait();
#pragma unroll
                            for (int c = 0; c < 8; ++c) {
                                const int ql = c_lo + c;
                                if ((mask >> ql) & 1u)
                                    Smine[ql * PSTRIDE + row] = row < mine.valid ? sc[c] + __ldg(qb_ + ql) : -INFINITY;
                            }
                        }
                    } else if (GMMA) {
                        // scores of a query group as a small matrix product on the warp-level tensor op: the restored
                        // K rows come out of tensor memory already in the A-fragment layout (16 tokens x 16 channels per
                        // step), the group's queries are the B operand, one 16-token half of the warp's rows at a time
                        const int n = lane >> 2, kq = 2 * (lane & 3);
                        for (int hp = chalf; hp < nh; hp += 2) {
                            const int ql0 = (job_kvh(job, hp) - h_lo) * group;
                            const float *bb = b2 + job_slot(job, hp) * 64 + kq;
                            uint32_t bq[8];
#pragma unroll
                            for (int ks = 0; ks < 4; ++ks) {
                                const __nv_bfloat16 *qr = qb + (ql0 + n) * QBS + 16 * ks + kq;
                                bq[2 * ks] = n < group ? *reinterpret_cast<const uint32_t *>(qr) : 0u;
                                bq[2 * ks + 1] = n < group ? *reinterpret_cast<const uint32_t *>(qr + 8) : 0u;
                            }
                            uint32_t r[2][32];
#pragma unroll
                            for (int h = 0; h < 2; ++h) {
                                const uint32_t ta = acc + ((uint32_t)(16 * h) << 16) + 64u * hp;
                                tmem_ld_frag_x4(ta, r[h]);
                                tmem_ld_frag_x4(ta + 32u, r[h] + 16);
                            }
                            tmem_ld_wait();
                            float dsc2[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
                            for (int ks = 0; ks < 4; ++ks) {
                                const int j0 = 2 * ks, j1 = 2 * ks + 1;
                                const float2 ba = *reinterpret_cast<const float2 *>(bb + 8 * j0);
                                const float2 bc = *reinterpret_cast<const float2 *>(bb + 8 * j1);
#pragma unroll
                                for (int h = 0; h < 2; ++h) {  // two independent accumulator chains
                                    const uint32_t a0 = pack_bf16(__uint_as_float(r[h][4 * j0]) + ba.x,
                                                                  __uint_as_float(r[h][4 * j0 + 1]) + ba.y);
                                    const uint32_t a1 = pack_bf16(__uint_as_float(r[h][4 * j0 + 2]) + ba.x,
                                                                  __uint_as_float(r[h][4 * j0 + 3]) + ba.y);
                                    const uint32_t a2 = pack_bf16(__uint_as_float(r[h][4 * j1]) + bc.x,
                                                                  __uint_as_float(r[h][4 * j1 + 1]) + bc.y);
                                    const uint32_t a3 = pack_bf16(__uint_as_float(r[h][4 * j1 + 2]) + bc.x,
                                                                  __uint_as_float(r[h][4 * j1 + 3]) + bc.y);
                                    mma_16816(dsc2[h], a0, a1, a2, a3, bq[2 * ks], bq[2 * ks + 1]);
                                }
                            }
#pragma unroll
                            for (int h = 0; h < 2; ++h) {
                                const float *dsc = dsc2[h];
                                // dsc: tokens (n, n + 8) of this half, queries (kq, kq + 1) of the group
                                const int tok = (int)lane_base + 16 * h + n;
                                if (kq < group) {
                                    float *sr = Smine + (ql0 + kq) * PSTRIDE;
                                    sr[tok] = tok < mine.valid ? dsc[0] : -INFINITY;
                                    sr[tok + 8] = tok + 8 < mine.valid ? dsc[2] : -INFINITY;
                                }
                                if (kq + 1 < group) {
                                    float *sr = Smine + (ql0 + kq + 1) * PSTRIDE;
                                    sr[tok] = tok < mine.valid ? dsc[1] : -INFINITY;
                                    sr[tok + 8] = tok + 8 < mine.valid ? dsc[3] : -INFINITY;
                                }
                            }
                        }
                    } else
                    for (int hp = chalf; hp < nh; hp += 2) {
                        float y[64];
                        tmem_ld32(acc + 64u * hp, y);
                        tmem_ld32(acc + 64u * hp + 32u, y + 32);
                        tmem_ld_wait();
                        const float4 *bb = reinterpret_cast<const float4 *>(b2 + job_slot(job, hp) * 64);
                        float2 y2[32];
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            const float4 b4 = bb[c];
                            y2[2 * c] = __fadd2_rn(make_float2(y[4 * c], y[4 * c + 1]), make_float2(b4.x, b4.y));
                            y2[2 * c + 1] = __fadd2_rn(make_float2(y[4 * c + 2], y[4 * c + 3]), make_float2(b4.z, b4.w));
                        }
                        const int ql0 = (job_kvh(job, hp) - h_lo) * group;
                        for (int g = 0; g < group; ++g) {
                            const float4 *q4 = reinterpret_cast<const float4 *>(qs + (ql0 + g) * 64);
                            float2 d0 = make_float2(0.f, 0.f), d1 = make_float2(0.f, 0.f);
#pragma unroll
                            for (int c = 0; c < 16; ++c) {
                                const float4 qq = q4[c];
                                d0 = __ffma2_rn(y2[2 * c], make_float2(qq.x, qq.y), d0);
                                d1 = __ffma2_rn(y2[2 * c + 1], make_float2(qq.z, qq.w), d1);
                            }
                            const float dot = (d0.x + d0.y) + (d1.x + d1.y);
                            Smine[(ql0 + g) * PSTRIDE + row] = row < mine.valid ? dot : -INFINITY;
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (elect_one()) mbar_arrive_remote(jempty_leader[buf]);
                    TR(3, 0x52);
                    epi_bar_sync();
                    // tile softmax of the job's query heads; probabilities go to both CTAs.  A query group has several
                    // rows per warp: four per turn, so that their shuffle chains overlap
                    if (mine.valid > 0) {
                        constexpr int R = GMMA ? 4 : 1;
                        const int n_items = job.kind == 3 ? (int)P.abs_n[job.src] : nh * group;
                        for (int base = ew; base < n_items; base += R * N_EPI_WARPS) {
                            int qlv[R];
                            float4 sc[R];
                            float mx[R], sum[R];
#pragma unroll
                            for (int u = 0; u < R; ++u) {
                                const int item = base + N_EPI_WARPS * u;
                                qlv[u] = -1;
                                sc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                                if (item < n_items) {
                                    const int hp = (int)(((uint32_t)item * ginv) >> 16);  // item / group
                                    qlv[u] = job.kind == 3 ? (int)P.abs_q[job.src][item]
                                                           : (job_kvh(job, hp) - h_lo) * group + (item - hp * group);
                                    sc[u] = *reinterpret_cast<const float4 *>(Smine + qlv[u] * PSTRIDE + 4 * lane);
                                }
                                mx[u] = fmaxf(fmaxf(sc[u].x, sc[u].y), fmaxf(sc[u].z, sc[u].w));
                            }
#pragma unroll
                            for (int o = 16; o > 0; o >>= 1)
#pragma unroll
                                for (int u = 0; u < R; ++u) mx[u] = fmaxf(mx[u], __shfl_xor_sync(0xffffffffu, mx[u], o));
#pragma unroll
                            for (int u = 0; u < R; ++u) {
                                sc[u].x = __expf(sc[u].x - mx[u]); sc[u].y = __expf(sc[u].y - mx[u]);
                                sc[u].z = __expf(sc[u].z - mx[u]); sc[u].w = __expf(sc[u].w - mx[u]);
                                sum[u] = (sc[u].x + sc[u].y) + (sc[u].z + sc[u].w);
                            }
#pragma unroll
                            for (int o = 16; o > 0; o >>= 1)
#pragma unroll
                                for (int u = 0; u < R; ++u) sum[u] += __shfl_xor_sync(0xffffffffu, sum[u], o);
                            if (!lay.kv_split && !s_waited) {
                                // the peer has read the previous pair's probabilities out of its copy
                                mbar_wait<false, 100>(B.s_free, (it - 1u) & 1u, a.status, &abort_flag, 0x305);
                                s_waited = true;
                            }
#pragma unroll
                            for (int u = 0; u < R; ++u) {
                                const int ql = qlv[u];
                                if (ql < 0) continue;
                                const int qh = h_lo * group + ql;
                                float *srow = Smine + ql * PSTRIDE;
                                if (lay.off_pop) {
                                    // absorbed V: this tile's probabilities as the column operand of the U product:
                                    // [query][token] bf16, two 64-token atoms of 128-byte rows, 128-byte swizzle
                                    uint8_t *dst = gbase + lay.off_pop + (lane >> 4) * (lay.nq_pad * 128) + ql * 128 +
                                                   ((((lane & 15) >> 1) ^ (ql & 7)) << 4) + 8 * (lane & 1);
                                    *reinterpret_cast<uint2 *>(dst) =
                                        make_uint2(pack_bf16(sc[u].x, sc[u].y), pack_bf16(sc[u].z, sc[u].w));
                                }
                                if (lay.kv_split) {
                                    float *grow = lay.pbuf + ((size_t)(2 * pair + (int)rank) * hq + qh) * PSTRIDE;
                                    *reinterpret_cast<float4 *>(grow + 4 * lane) = sc[u];
                                    if (lane == 0) grow[128] = sum[u];
                                } else if (GMMA) {
                                    // the V side multiplies on the warp-level tensor op: probabilities as bf16 pairs, the
                                    // row's sum in the row's padding
                                    __nv_bfloat16 *prow = Pb + (rank * lay.nq_local + ql) * PBS;
                                    *reinterpret_cast<uint2 *>(prow + 4 * lane) =
                                        make_uint2(pack_bf16(sc[u].x, sc[u].y), pack_bf16(sc[u].z, sc[u].w));
                                    if (lane == 0) *reinterpret_cast<float *>(prow + 128) = sum[u];
                                } else {
                                    *reinterpret_cast<float4 *>(srow + 4 * lane) = sc[u];
                                    if (lane == 0) srow[128] = sum[u];
                                    const uint32_t prow = peer_S + (uint32_t)((rank * lay.nq_local + ql) * PSTRIDE) * 4u;
                                    st_cluster_v4(prow + 16u * lane, sc[u].x, sc[u].y, sc[u].z, sc[u].w);
                                    if (lane == 0) st_cluster_f32(prow + 128u * 4u, sum[u]);
                                }
                                if (lane == 0) {
                                    float *part =
                                        a.partials + (((int64_t)mine.si * a.max_chunks + mine.chunk) * hq + qh) * (64 + 2);
                                    part[0] = mx[u];
                                    part[1] = sum[u];
                                }
                            }
                            if (GMMA && !lay.kv_split) {
                                // the finished rows go to the peer whole (probabilities and sum), one copy per row
                                fence_async_smem();
                                __syncwarp();
                                int ql = -1;
#pragma unroll
                                for (int u = 0; u < R; ++u) ql = lane == u ? qlv[u] : ql;
                                if (ql >= 0) {
                                    const uint32_t off = (uint32_t)((rank * lay.nq_local + ql) * PBS) * 2u;
                                    bulk_copy_to_peer(peer_Pb + off, smem_u32(Pb) + off, PBS * 2u, peer_pready);
                                }
                            }
                        }
                    }
                    if (lay.kv_split) {
                        // publish: this job's heads of this tile are in global memory for the V cluster
                        __threadfence();
                        epi_bar_sync();
                        if (et < nh && mine.valid > 0)
                            asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(lay.pflags + (size_t)(2 * pair + (int)rank) *
                                                                                        a.hkv + job_kvh(job, et)),
                                         "r"(lay.epoch)
                                         : "memory");
                    }
                    TR(3, 0x53);
                } else if (job.kind == 4) {
                    // absorbed V: this thread owns hidden feature `row` of each 128-feature chunk; the accumulator's
                    // own column block holds U[feature][query] of this CTA's tile; it goes to the workspace as it is
                    // (the last decoder layer is applied once per sequence and head, after the tiles are merged)
                    const uint32_t mask = (uint32_t)job.c0 | ((uint32_t)job.nc << 16);
                    const int ks2 = (m + 63) >> 6, n_ch = (ks2 + 1) >> 1;
                    if (mine.valid > 0) {
                        float *ub = lay.ubuf + (((int64_t)mine.si * a.max_chunks + mine.chunk) * hq) * lay.m_pad_u;
                        for (int c = chalf; c < n_ch; c += 2) {
                            const int sa = min(2 * c, ks2 - 2);
                            const int f = sa * 64 + row;
                            const bool repeated = 2 * c > ks2 - 2 && row < 64;  // slab already covered by the chunk before
                            const uint32_t ta = acc + (uint32_t)(c * 2 * lay.nq_pad + lay.nq_pad * (int)rank);
                            for (int q0 = 0; q0 < lay.nq_pad; q0 += 16) {
                                float u[16];
                                tmem_ld8(ta + (uint32_t)q0, u);
                                tmem_ld8(ta + (uint32_t)q0 + 8u, u + 8);
                                tmem_ld_wait();
                                if (!repeated && f < m) {
#pragma unroll
                                    for (int ql = 0; ql < 16; ++ql)
                                        if ((mask >> (q0 + ql)) & 1u) ub[(int64_t)(q0 + ql) * lay.m_pad_u + f] = u[ql];
                                }
                            }
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (elect_one()) mbar_arrive_remote(jempty_leader[buf]);
                    TR(3, 0x63);
                } else {
                    // V: this thread owns (head place, channel) = row; columns = tokens of tile chalf
                    if (!lay.kv_split && !p_waited) {
                        mbar_wait<!GMMA, 100>(B.p_ready, it & 1u, a.status, &abort_flag, 0x303);
                        p_waited = true;
                    }
                    const int hp = 2 * (int)rank + (row >> 6), c = row & 63;
                    const int kvh = job_kvh(job, hp);
                    const TileInfo tt = tl[chalf];
                    if (GMMA) {
                        // restored V rows are the A operand straight from tensor memory (16 channels x 16 tokens per
                        // step), the group's probabilities the B operand; both 16-channel halves of the warp's rows
                        if (kvh >= 0 && tt.valid > 0) {
                            const int n = lane >> 2, kq = 2 * (lane & 3);
                            const int ql0 = (kvh - h_lo) * group;
                            const __nv_bfloat16 *prow = Pb + ((size_t)chalf * lay.nq_local + ql0 + n) * PBS + kq;
                            float dv[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
                            for (int gi = 0; gi < 4; ++gi) {
                                if (32 * gi >= tt.valid) break;
                                uint32_t bp[4];
#pragma unroll
                                for (int ks = 0; ks < 2; ++ks) {
                                    const __nv_bfloat16 *pr = prow + 32 * gi + 16 * ks;
                                    bp[2 * ks] = n < group ? *reinterpret_cast<const uint32_t *>(pr) : 0u;
                                    bp[2 * ks + 1] = n < group ? *reinterpret_cast<const uint32_t *>(pr + 8) : 0u;
                                }
                                // nothing between the tensor-memory loads and their wait: until then the destination
                                // registers are written behind the compiler's back, and code placed in between gives it
                                // reasons to move them
                                uint32_t r[2][16];
                                tmem_ld_frag_x4(acc + 128u * chalf + 32u * gi, r[0]);
                                tmem_ld_frag_x4(acc + (16u << 16) + 128u * chalf + 32u * gi, r[1]);
                                tmem_ld_wait();
                                if (32 * gi + 32 > tt.valid) {  // rows past the tile's end may hold anything
#pragma unroll
                                    for (int h = 0; h < 2; ++h)
#pragma unroll
                                        for (int e = 0; e < 16; ++e)
                                            if (32 * gi + 8 * (e >> 2) + kq + (e & 1) >= tt.valid) r[h][e] = 0u;
                                }
#pragma unroll
                                for (int ks = 0; ks < 2; ++ks)
#pragma unroll
                                    for (int h = 0; h < 2; ++h) {
                                        const int j0 = 2 * ks, j1 = 2 * ks + 1;
                                        const uint32_t a0 = pack_bf16(__uint_as_float(r[h][4 * j0]),
                                                                      __uint_as_float(r[h][4 * j0 + 1]));
                                        const uint32_t a1 = pack_bf16(__uint_as_float(r[h][4 * j0 + 2]),
                                                                      __uint_as_float(r[h][4 * j0 + 3]));
                                        const uint32_t a2 = pack_bf16(__uint_as_float(r[h][4 * j1]),
                                                                      __uint_as_float(r[h][4 * j1 + 1]));
                                        const uint32_t a3 = pack_bf16(__uint_as_float(r[h][4 * j1 + 2]),
                                                                      __uint_as_float(r[h][4 * j1 + 3]));
                                        mma_16816(dv[h], a0, a1, a2, a3, bp[2 * ks], bp[2 * ks + 1]);
                                    }
                            }
                            // dv[h]: channels (n, n + 8) of half h, queries (kq, kq + 1) of the group
                            const __nv_bfloat16 *psum = Pb + ((size_t)chalf * lay.nq_local + ql0) * PBS + 128;
                            const float *bv = b2 + job_slot(job, hp) * 64;
#pragma unroll
                            for (int e = 0; e < 2; ++e) {
                                if (kq + e < group) {
                                    const int qh = h_lo * group + ql0 + kq + e;
                                    float *part =
                                        a.partials + (((int64_t)tt.si * a.max_chunks + tt.chunk) * hq + qh) * (64 + 2) + 2;
                                    const float sum = *reinterpret_cast<const float *>(psum + (kq + e) * PBS);
#pragma unroll
                                    for (int h = 0; h < 2; ++h) {
                                        const int ch = (row & 32) + 16 * h + n;
                                        part[ch] = dv[h][e] + bv[ch] * sum;
                                        part[ch + 8] = dv[h][2 + e] + bv[ch + 8] * sum;
                                    }
                                }
                            }
                        }
                    } else
                    if (kvh >= 0 && tt.valid > 0) {
                        const int ql0 = (kvh - h_lo) * group;
                        const float *Sp = Sall + ((size_t)chalf * lay.nq_local + ql0) * PSTRIDE;
                        float2 accv[8];
#pragma unroll
                        for (int g = 0; g < 8; ++g) accv[g] = make_float2(0.f, 0.f);
                        for (int gi = 0; gi < 4; ++gi) {
                            if (32 * gi >= tt.valid) break;
                            float y[32];
                            tmem_ld32(acc + 128u * chalf + 32u * gi, y);
                            tmem_ld_wait();
                            if (32 * gi + 32 > tt.valid) {  // rows past the tile's end may hold anything
#pragma unroll
                                for (int t = 0; t < 32; ++t) y[t] = (32 * gi + t < tt.valid) ? y[t] : 0.f;
                            }
#pragma unroll
                            for (int g = 0; g < 8; ++g) {
                                if (g < group) {
                                    const float4 *p4 = reinterpret_cast<const float4 *>(Sp + g * PSTRIDE + 32 * gi);
                                    float2 s0 = accv[g], s1v = make_float2(0.f, 0.f);
#pragma unroll
                                    for (int t = 0; t < 8; ++t) {
                                        const float4 pp = p4[t];
                                        s0 = __ffma2_rn(make_float2(pp.x, pp.y), make_float2(y[4 * t], y[4 * t + 1]), s0);
                                        s1v = __ffma2_rn(make_float2(pp.z, pp.w), make_float2(y[4 * t + 2], y[4 * t + 3]), s1v);
                                    }
                                    accv[g] = __fadd2_rn(s0, s1v);
                                }
                            }
                        }
                        const float bias = b2[job_slot(job, hp) * 64 + c];
#pragma unroll
                        for (int g = 0; g < 8; ++g) {
                            if (g < group) {
                                const int qh = (h_lo * group) + ql0 + g;
                                float *part = a.partials + (((int64_t)tt.si * a.max_chunks + tt.chunk) * hq + qh) * (64 + 2);
                                part[2 + c] = (accv[g].x + accv[g].y) + bias * Sp[g * PSTRIDE + 128];
                            }
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (elect_one()) mbar_arrive_remote(jempty_leader[buf]);
                    TR(3, 0x63);
                }
            }
        }
        if (!lay.kv_split) {  // this CTA no longer reads the pair's probabilities: the peer may overwrite them
            __syncwarp();
            if (elect_one()) mbar_arrive_remote(map_to_cta(B.s_free, rank ^ 1u));
        }
      }  // pairs
    }
    // ---- teardown: nobody leaves while the peer may still read or write this CTA ----
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
}

// ---------------------------------------------------------------------------- host side
inline uint32_t up(uint32_t x, uint32_t a) { return (x + a - 1) / a * a; }

PairLaunch make_launch(int nq_local, int group, int max_m, int max_in, int pslots, int nslot, bool pop = false) {
    const int nq_pad_pop = nq_local <= 16 ? 16 : 32;
    PairLaunch l{};
    const int ks_hid = (max_m + 63) / 64;
    uint32_t o = 0;
    l.off_hidden = o;
    o += (uint32_t)ks_hid * SLOT_BYTES;
    l.off_ring = o;
    o += (uint32_t)nslot * SLOT_BYTES;
    l.off_part = o;
    o = up(o + (uint32_t)sizeof(TcPart), 16);
    l.off_fparam = o;
    o = up(o + (uint32_t)pslots * (uint32_t)(2 * ((max_m + 31) & ~31) + max_in) * 4, 16);  // parameter blocks
    l.off_q = o;
    o = up(o + (uint32_t)nq_local * 64 * 4, 16);
    l.off_s = o;
    o = up(o + 2u * (uint32_t)nq_local * PSTRIDE * 4, 16);
    l.group_mma = group > 2 ? 1 : 0;
    l.off_qb = o;
    if (l.group_mma) o = up(o + (uint32_t)nq_local * QBS * 2, 16);
    l.off_pb = o;
    if (l.group_mma) o = up(o + 2u * (uint32_t)nq_local * PBS * 2, 16);
    if (pop) {  // absorbed V: the tile's probabilities as a column operand, 16 or 32 rows x 256 B, on a swizzle boundary
        o = up(o, 1024);
        l.off_pop = o;
        o += (uint32_t)nq_pad_pop * 256;
    }
    l.off_bar = o;
    l.nslot = nslot;
    l.max_m = max_m;
    l.max_in = max_in;
    l.nq_local = nq_local;
    return l;
}
uint32_t launch_bytes(const PairLaunch &l) { return l.off_bar + 8u * (2 * l.nslot + N_FIXED_BARS) + 1024u; }

// ring depth that fits beside everything else (0 = does not fit)
int pick_nslot(int nq_local, int group, int max_m, int max_in, int pslots, bool pop = false) {
    for (int nslot = 10; nslot >= 3; --nslot)
        if (launch_bytes(make_launch(nq_local, group, max_m, max_in, pslots, nslot, pop)) <= 227u * 1024u) return nslot;
    return 0;
}

// Job tables of one head subset [h_lo, h_hi) of one layer.  Returns false if it does not fit the table limits.
// absorbed: the K head groups of every source are replaced by one score job over all its query heads (kind 3).
bool build_part(const LayerPlan &lp, const TcSrc (*srcs)[MAX_SRC], int h_lo, int h_hi, TcPart &out, bool absorbed = false,
                int group = 1, bool absorbed_v = false) {
    memset(&out, 0, sizeof(out));
    out.h_lo = h_lo;
    out.h_hi = h_hi;
    for (int which = 0; which < 2; ++which) {
        const WhichPlan &wp = lp.w[which];
        int nj = 0, ns = 0;
        for (int s = 0; s < wp.n_src; ++s) {
            const SourcePlan &sp = wp.src[s];
            int heads[KVCAR_MAX_KV_HEADS], slots[KVCAR_MAX_KV_HEADS], n = 0;
            for (int i = 0; i < sp.n_need; ++i)
                if (sp.kv_head[i] >= h_lo && sp.kv_head[i] < h_hi) {
                    heads[n] = sp.kv_head[i];
                    slots[n] = sp.slot[i];
                    ++n;
                }
            if (n == 0) continue;
            if (ns == TC_MAX_SRC) return false;
            out.src[which][ns] = srcs[which][s];
            out.max_m = std::max(out.max_m, sp.m);
            bool first = true;
            for (int c0 = 0; c0 < sp.m; c0 += 256) {  // hidden chunks
                if (nj == TC_MAX_JOBS) return false;
                TcJob &jb = out.jobs[which][nj++];
                jb.kind = 1;
                jb.src = (uint8_t)ns;
                jb.first = first ? 1 : 0;
                jb.c0 = (uint16_t)c0;
                jb.nc = (uint16_t)std::min(256, sp.m - c0);
                first = false;
            }
            first = true;
            if (absorbed && which == 0) {
                if (nj == TC_MAX_JOBS || (h_hi - h_lo) * group > TC_ABS_MAX_Q) return false;
                TcJob &jb = out.jobs[which][nj++];
                jb.kind = 3;
                jb.src = (uint8_t)ns;
                jb.first = 1;
                uint32_t mask = 0;
                for (int i = 0; i < n; ++i)
                    for (int g = 0; g < group; ++g) mask |= 1u << ((heads[i] - h_lo) * group + g);
                jb.c0 = (uint16_t)(mask & 0xffffu);
                jb.nc = (uint16_t)(mask >> 16);
                int cnt = 0;
                for (int ql = 0; ql < TC_ABS_MAX_Q; ++ql)
                    if ((mask >> ql) & 1u) out.abs_q[ns][cnt++] = (uint8_t)ql;
                out.abs_n[ns] = (uint8_t)cnt;
                n = 0;  // no head groups
            }
            if (absorbed_v && which == 1) {
                // one job for the whole source: at least two hidden slabs (the row operand spans two), and all
                // 128-feature chunks side by side in one 256-column accumulator buffer (2 x 16 or 2 x 32 columns each)
                const int ks2 = (sp.m + 63) / 64, nq = (h_hi - h_lo) * group, cols = 2 * (nq <= 16 ? 16 : 32);
                if (nj == TC_MAX_JOBS || nq > TC_ABS_MAX_Q || ks2 < 2 || ((ks2 + 1) / 2) * cols > 256) return false;
                TcJob &jb = out.jobs[which][nj++];
                jb.kind = 4;
                jb.src = (uint8_t)ns;
                jb.first = 1;
                uint32_t mask = 0;
                for (int i = 0; i < n; ++i)
                    for (int g = 0; g < group; ++g) mask |= 1u << ((heads[i] - h_lo) * group + g);
                jb.c0 = (uint16_t)(mask & 0xffffu);
                jb.nc = (uint16_t)(mask >> 16);
                n = 0;
            }
            for (int i = 0; i < n;) {  // head groups: K 4/2/1 real heads; V always four places, padded
                if (nj == TC_MAX_JOBS) return false;
                TcJob &jb = out.jobs[which][nj++];
                jb.kind = 2;
                jb.src = (uint8_t)ns;
                jb.first = first ? 1 : 0;
                first = false;
                int nh = n - i >= 4 ? 4 : (n - i >= 2 ? 2 : 1);
                if (which == 1) nh = std::min(4, n - i);
                jb.nh = (uint8_t)nh;
                for (int p = 0; p < 4; ++p) {
                    jb.kvh[p] = -1;
                    jb.slot[p] = (int8_t)slots[i];  // padding places load the first real head's rows
                }
                static const int order_v[4] = {0, 2, 1, 3};  // spread V heads over the two CTAs
                for (int k = 0; k < nh; ++k) {
                    const int p = which == 1 ? order_v[k] : k;
                    jb.kvh[p] = (int8_t)heads[i + k];
                    jb.slot[p] = (int8_t)slots[i + k];
                }
                i += nh;
            }
            if (absorbed_v) out.jobs[which][nj - 1].first |= 2;  // last job of its source: its completion is signalled
            ++ns;
        }
        out.n_src[which] = ns;
        out.n_jobs[which] = nj;
    }
    return true;
}

inline int part_index(int split, int i) { return (split == 1 ? 0 : split == 2 ? 1 : 3) + i; }

// A wait that nothing completes: one warp waits on a fresh barrier with the given limit, records its code in the
// status word and returns.  Exercises the path every bounded wait of this file takes when it runs out.
__global__ void expire_wait_kernel(int32_t *status, uint64_t limit_ns) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
    }
    __syncwarp();
    const uint32_t b = smem_u32(&bar);
    const uint64_t t0 = global_ns();
    while (!mbar_try(b, 0)) {
        __nanosleep(200);
        if (global_ns() - t0 > limit_ns) {
            abort_flag = 1;
            atomicCAS(status, 0, 0x7e57);
            break;
        }
    }
}

}  // namespace

cudaError_t tc_launch_expire_wait(int32_t *status, uint64_t limit_ns, cudaStream_t st) {
    expire_wait_kernel<<<1, 32, 0, st>>>(status, limit_ns);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------- absorbed K scores: operands
// scores of head h against a token = a . (W4_h^T q) + q . b4_h with a the token's activated hidden vector (the
// decoder's last layer is linear).  One block per (query head, listed sequence) forms the m-vector W4_h^T (q * scale)
// as a bf16 row - the column operand of the score job - and the scalar q . b4_h.  W4 is the K-major copy
// [in_dim][m], so consecutive threads read consecutive hidden columns.
__global__ void __launch_bounds__(128) absorb_q_kernel(const __grid_constant__ DecodeArgs a, const __grid_constant__ SeqList seqs,
                                                       __nv_bfloat16 *wq, float *qbias, int nq_pad, int m_pad, int batch) {
    __shared__ float qsm[64];
    const int qh = blockIdx.x, si = blockIdx.y, tid = threadIdx.x;
    const int kvh = qh / (a.hq / a.hkv);
    const WhichPlan &wp = a.plan->w[0];
    int s = 0, slot = 0;
    for (int i = 0; i < wp.n_src; ++i)
        for (int k = 0; k < wp.src[i].n_need; ++k)
            if (wp.src[i].kv_head[k] == kvh) {
                s = i;
                slot = wp.src[i].slot[k];
            }
    const SourcePlan &sp = wp.src[s];
    if (tid < 64)
        qsm[tid] = __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(a.q)[((int64_t)si * a.hq + qh) * 64 + tid]) * a.scale;
    __syncthreads();
    const __nv_bfloat16 *w2 = reinterpret_cast<const __nv_bfloat16 *>(sp.w2k) + (int64_t)slot * 64 * sp.m;
    __nv_bfloat16 *row = wq + (((int64_t)s * batch + si) * nq_pad + qh) * m_pad;
    for (int j = tid; j < m_pad; j += 128) {
        float acc = 0.f;
        if (j < sp.m) {
#pragma unroll 8
            for (int c = 0; c < 64; ++c) acc = fmaf(__bfloat162float(w2[(int64_t)c * sp.m + j]), qsm[c], acc);
        }
        row[j] = __float2bfloat16_rn(acc);
    }
    if (tid < 32) {
        float b = qsm[tid] * sp.b2[slot * 64 + tid] + qsm[tid + 32] * sp.b2[slot * 64 + tid + 32];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) b += __shfl_xor_sync(0xffffffffu, b, o);
        if (tid == 0) qbias[((int64_t)s * batch + si) * nq_pad + qh] = b;
    }
}

// Merge of the tiles after a launch in the absorbed V form.  A tile's partial is (maximum, sum) in the usual place
// and U = sum over its tokens of p * a (m values) in the U buffer; with w_t = exp(max_t - M) the head's output is
// (W4_h (sum_t w_t U_t) + b4_h sum_t w_t s_t [+ the exact current token]) / (sum of all weights): the last decoder
// layer is applied once, here.  One block per (query head, listed sequence); W4 is read through its transposed copy
// [m][in_dim] so that consecutive threads read consecutive channels.
constexpr int CA_THREADS = 128, CA_MAX_TILES = 512;
__global__ void __launch_bounds__(CA_THREADS) combine_absorbed_kernel(const __grid_constant__ DecodeArgs a,
                                                                      const __grid_constant__ SeqList seqs,
                                                                      const float *ubuf, int m_pad) {
    extern __shared__ float ca_smem[];  // U accumulated over the tiles [m_pad]
    __shared__ float wts[CA_MAX_TILES];
    __shared__ float red[CA_THREADS / 32];
    const int qh = blockIdx.x, si = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int seq = seqs.id[si];
    const int L = a.seq_len[seq];
    const int hq = a.hq, hd = 64;
    const int n_tiles = (L + a.chunk_tokens - 1) / a.chunk_tokens;
    const int kvh = qh / (hq / a.hkv);
    const WhichPlan &wp = a.plan->w[1];
    int s_ = 0, slot = 0;
    for (int i = 0; i < wp.n_src; ++i)
        for (int k = 0; k < wp.src[i].n_need; ++k)
            if (wp.src[i].kv_head[k] == kvh) {
                s_ = i;
                slot = wp.src[i].slot[k];
            }
    const SourcePlan &sp = wp.src[s_];
    const float *part = a.partials + ((int64_t)si * a.max_chunks * hq + qh) * (hd + 2);
    const int64_t pstride = (int64_t)hq * (hd + 2);
    auto block_max = [&](float v) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
        __syncthreads();
        if (lane == 0) red[warp] = v;
        __syncthreads();
        float r = red[0];
#pragma unroll
        for (int i = 1; i < CA_THREADS / 32; ++i) r = fmaxf(r, red[i]);
        return r;
    };
    auto block_sum = [&](float v) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        __syncthreads();
        if (lane == 0) red[warp] = v;
        __syncthreads();
        float r = red[0];
#pragma unroll
        for (int i = 1; i < CA_THREADS / 32; ++i) r += red[i];
        return r;
    };
    float M = -INFINITY;
    for (int t = tid; t < n_tiles; t += CA_THREADS) M = fmaxf(M, part[t * pstride]);
    M = block_max(M);
    float S = 0.f;
    for (int t = tid; t < n_tiles; t += CA_THREADS) {
        const float mt = part[t * pstride];
        const float w = mt == -INFINITY ? 0.f : expf(mt - M);
        wts[t] = w;
        S += w * part[t * pstride + 1];
    }
    S = block_sum(S);  // (the barriers inside also publish wts)
    const float *ub = ubuf + (((int64_t)si * a.max_chunks) * hq + qh) * m_pad;
    const int64_t ustride = (int64_t)hq * m_pad;
    for (int j = tid; j < sp.m; j += CA_THREADS) {
        float acc = 0.f;
#pragma unroll 4
        for (int t = 0; t < n_tiles; ++t) acc = fmaf(wts[t], ub[t * ustride + j], acc);
        ca_smem[j] = acc;
    }
    __syncthreads();
    // channel c of the head: two threads split the hidden range
    const int c = tid & 63, half = tid >> 6;
    const __nv_bfloat16 *w2t = reinterpret_cast<const __nv_bfloat16 *>(sp.w2t) + slot * hd + c;
    float o = 0.f;
    for (int j = half; j < sp.m; j += 2) o = fmaf(__bfloat162float(w2t[(int64_t)j * sp.in_dim]), ca_smem[j], o);
    __shared__ float o2[64];
    if (half == 1) o2[c] = o;
    __syncthreads();
    float acc = half == 0 ? o + o2[c] + sp.b2[slot * hd + c] * S : 0.f;
    if (a.flags & KVCAR_INCLUDE_CURRENT_EXACT) {
        const int W = a.hkv * hd;
        const __nv_bfloat16 *kc = reinterpret_cast<const __nv_bfloat16 *>(a.plan->cur[0][kvh]) + (int64_t)seq * W + a.plan->cur_head[0][kvh] * hd;
        const __nv_bfloat16 *vc = reinterpret_cast<const __nv_bfloat16 *>(a.plan->cur[1][kvh]) + (int64_t)seq * W + a.plan->cur_head[1][kvh] * hd;
        const __nv_bfloat16 *qg = reinterpret_cast<const __nv_bfloat16 *>(a.q) + ((int64_t)si * hq + qh) * hd;
        const float sc = block_sum(half == 0 ? __bfloat162float(qg[c]) * __bfloat162float(kc[c]) : 0.f) * a.scale;
        const float Mn = fmaxf(M, sc);
        const float c0 = M == -INFINITY ? 0.f : expf(M - Mn), c1 = expf(sc - Mn);
        S = S * c0 + c1;
        acc = acc * c0 + __bfloat162float(vc[c]) * c1;
    }
    if (half == 0)
        reinterpret_cast<__nv_bfloat16 *>(a.out)[((int64_t)si * hq + qh) * hd + c] = __float2bfloat16_rn(S > 0.f ? acc / S : 0.f);
}

cudaError_t tc_launch_combine_absorbed(const TcState &tc, const DecodeArgs &a, const SeqList &seqs, cudaStream_t st) {
    combine_absorbed_kernel<<<dim3(a.hq, seqs.n), CA_THREADS, (size_t)tc.abs_m_pad * sizeof(float), st>>>(a, seqs, tc.ubuf,
                                                                                                        tc.abs_m_pad);
    return cudaGetLastError();
}

// absorbed V side: bytes of the U vectors (0 where the form is not taken: more than 16 query heads, or more than
// 512 tiles per sequence, which the merge kernel's weight table does not hold)
static size_t absorb_u_bytes(const kvcar_config &cfg, int max_m, int batch, int max_chunks) {
    if (cfg.n_q_heads > TC_ABS_MAX_Q || max_chunks > 512) return 0;
    const size_t m_pad = ((size_t)max_m + 63) / 64 * 64;
    return (size_t)batch * max_chunks * cfg.n_q_heads * m_pad * sizeof(float);
}
size_t tc_absorb_bytes(const kvcar_config &cfg, int max_k_sources, int max_m, int batch, int max_chunks) {
    if (cfg.storage != KVCAR_BF16 || cfg.n_q_heads > TC_ABS_MAX_Q || max_k_sources <= 0 || max_m <= 0) return 0;
    const size_t nq_pad = cfg.n_q_heads <= 16 ? 16 : 32, m_pad = ((size_t)max_m + 63) / 64 * 64;
    const size_t rows = (size_t)max_k_sources * batch * nq_pad;
    return (rows * m_pad * 2 + 255) / 256 * 256 + (rows * sizeof(float) + 255) / 256 * 256 +
           absorb_u_bytes(cfg, max_m, batch, max_chunks);
}

void tc_setup_absorb(TcState &tc, const kvcar_config &cfg, int max_k_sources, int max_m, int batch, int max_chunks,
                     char *ws_area, char *tmap_host, char *tmap_dev) {
    tc.wq = nullptr;
    tc.ubuf = nullptr;
    if (!tc.available || tc_absorb_bytes(cfg, max_k_sources, max_m, batch, max_chunks) == 0) return;
    EncodeTiledFn fn = tensor_map_encoder();
    if (!fn) return;
    const int nq_pad = cfg.n_q_heads <= 16 ? 16 : 32, m_pad = (max_m + 63) / 64 * 64;
    const size_t rows = (size_t)max_k_sources * batch * nq_pad;
    if (!encode_bf16_map(fn, tmap_host, ws_area, rows, (uint64_t)m_pad, (uint64_t)m_pad, (uint32_t)nq_pad)) return;
    tc.wq = ws_area;
    tc.qbias = reinterpret_cast<float *>(ws_area + (rows * m_pad * 2 + 255) / 256 * 256);
    tc.tm_wq = tmap_dev;
    tc.abs_nq_pad = nq_pad;
    tc.abs_m_pad = m_pad;
    tc.abs_batch = batch;
    tc.abs_max_src = max_k_sources;
    if (absorb_u_bytes(cfg, max_m, batch, max_chunks)) {
        tc.ubuf = reinterpret_cast<float *>(ws_area + (rows * m_pad * 2 + 255) / 256 * 256 + (rows * sizeof(float) + 255) / 256 * 256);
        tc.abs_max_chunks = max_chunks;
    }
}

size_t tc_part_bytes(int n_layers) { return (size_t)n_layers * TC_PARTS_PER_LAYER * sizeof(TcPart); }
size_t tc_split_bytes(const kvcar_config &cfg) {
    return (size_t)TC_SPLIT_TILES * ((size_t)cfg.n_q_heads * PSTRIDE * sizeof(float) + (size_t)cfg.n_kv_heads * sizeof(uint32_t));
}

void tc_setup(TcState &tc, const kvcar_config &cfg, const LayerPlan *plans, int n_layers, char *weights_dev,
              size_t tmap_off, size_t part_off, char *img, size_t pool_rows) {
    tc.available = false;
    tc.parts_dev = weights_dev + part_off;
    memset(tc.layer, 0, sizeof(tc.layer));
    static_assert(sizeof(TcPart) % 16 == 0, "job tables are copied in 16-byte words");
    if (cfg.storage != KVCAR_BF16) {
        tc.why = "storage type is not bf16";
        return;
    }
    if (cfg.head_dim != 64 || cfg.page_tokens % 64 != 0 || n_layers > TC_MAX_LAYERS) {
        tc.why = "needs head_dim 64 and a page size that is a multiple of 64";
        return;
    }
    if (cfg.n_q_heads / cfg.n_kv_heads > 8) {
        tc.why = "more than 8 query heads per KV head";
        return;
    }
    EncodeTiledFn fn = tensor_map_encoder();
    if (!fn) {
        tc.why = "cuTensorMapEncodeTiled is not available (no driver)";
        return;
    }
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    tc.n_sms = sms;
    std::vector<char> built((size_t)n_layers * 2, 0);
    bool any = false;
    const int group = cfg.n_q_heads / cfg.n_kv_heads;
    for (int l = 0; l < n_layers; ++l) {
        bool ok = true;
        int max_m = 0, max_in = 0;
        TcSrc srcs[2][MAX_SRC];
        for (int which = 0; which < 2 && ok; ++which) {
            const WhichPlan &wp = plans[l].w[which];
            for (int s = 0; s < wp.n_src && ok; ++s) {
                const SourcePlan &sp = wp.src[s];
                if (!sp.compressed || sp.qparam /* int8 rows: generic kernel */ || sp.d % 16 || sp.m % 16 || sp.d < 16 || sp.m < 16 || sp.m > 256 * MAX_HID_GROUPS || sp.in_dim > 256 * MAX_HID_GROUPS ||
                    sp.in_dim % 64 || sp.width != sp.d) {
                    ok = false;
                    break;
                }
                const int idx = sp.src_layer * 2 + which;
                char *host = img + tmap_off + (size_t)idx * 3 * 128;
                char *devp = weights_dev + tmap_off + (size_t)idx * 3 * 128;
                if (!built[idx]) {
                    if (!encode_bf16_map(fn, host, sp.pool, pool_rows, (uint64_t)sp.width, (uint64_t)sp.width) ||
                        !encode_bf16_map(fn, host + 128, sp.w1k, (uint64_t)sp.m, (uint64_t)sp.d, (uint64_t)sp.d) ||
                        !encode_bf16_map(fn, host + 256, sp.w2k, (uint64_t)sp.in_dim, (uint64_t)sp.m, (uint64_t)sp.m)) {
                        ok = false;
                        break;
                    }
                    built[idx] = 1;
                }
                TcSrc &t = srcs[which][s];
                t.tm_pool = devp;
                t.tm_w1 = devp + 128;
                t.tm_w2 = devp + 256;
                t.s1 = sp.s1;
                t.t1 = sp.t1;
                t.b2 = sp.b2;
                t.d = sp.d;
                t.m = sp.m;
                t.slope = sp.slope;
                t.in_dim = sp.in_dim;
                max_m = std::max(max_m, sp.m);
                max_in = std::max(max_in, sp.in_dim);
            }
        }
        if (!ok || max_m == 0) continue;
        TcPart *parts = reinterpret_cast<TcPart *>(img + part_off) + (size_t)l * TC_PARTS_PER_LAYER;
        TcLayerCfg &lc = tc.layer[l];
        // hidden layers of a single chunk: every source keeps its parameter block in shared memory (see SLAB)
        const int pslots = max_m <= 256 ? plans[l].w[0].n_src + plans[l].w[1].n_src : 1;
        const int splits[3] = {1, 2, 4};
        for (int si = 0; si < 3; ++si) {
            const int split = splits[si];
            if (cfg.n_kv_heads % split) continue;
            const int per = cfg.n_kv_heads / split;
            bool fits = pick_nslot(per * group, group, max_m, max_in, pslots) >= 3;
            for (int i = 0; i < split && fits; ++i)
                fits = build_part(plans[l], srcs, i * per, (i + 1) * per, parts[part_index(split, i)]);
            lc.split_ok[si] = fits ? 1 : 0;
        }
        if (!lc.split_ok[0]) continue;
        lc.abs_ok = cfg.n_q_heads <= TC_ABS_MAX_Q && build_part(plans[l], srcs, 0, cfg.n_kv_heads, parts[7], true, group) ? 1 : 0;
        lc.absv_ok = lc.abs_ok &&
                     pick_nslot(cfg.n_kv_heads * group, group, max_m, max_in, pslots, true) >= 3 &&
                     build_part(plans[l], srcs, 0, cfg.n_kv_heads, parts[8], true, group, true) ? 1 : 0;
        lc.ok = 1;
        lc.max_m = (uint16_t)max_m;
        lc.max_in = (uint16_t)max_in;
        lc.pslots = (uint16_t)pslots;
        any = true;
    }
    if (!any) {
        tc.why = "no layer fits the tensor-core kernel (raw layers, unsupported widths, or shared memory)";
        return;
    }
    tc.available = true;
    tc.why = "ok";
}

void tc_destroy(TcState &) {}

bool tc_layer_supported(const TcState &tc, int layer) {
    return tc.available && layer >= 0 && layer < TC_MAX_LAYERS && tc.layer[layer].ok;
}

cudaError_t tc_launch_decode(TcState &tc, const DecodeArgs &a, const SeqList &seqs, const int32_t *lens,
                             int layer, cudaStream_t st, int *n_launches) {
    *n_launches = 1;
    const TcLayerCfg &lc = tc.layer[layer];
    TileIndex tix;
    uint32_t t = 0;
    for (int i = 0; i < seqs.n; ++i) {
        tix.first[i] = t;
        tix.len[i] = lens[i];
        t += (uint32_t)((lens[i] + TILE - 1) / TILE);
    }
    tix.first[seqs.n] = t;
    tix.n_tiles = (int32_t)t;
    if (t == 0) return cudaSuccess;
    const int n_pairs = (int)((t + 1) / 2);
    // Small grids: spread the work of a tile pair over more clusters while everything still runs in one wave.
    // First K and V go to separate clusters (nothing is computed twice: the probabilities cross through global
    // memory behind per-head flags); then the KV heads are split (each cluster repeats the hidden layer for its
    // heads).  A V cluster waits for flags that the K cluster of the same pair sets, and a K cluster waits for no
    // other cluster.  The K cluster has the lower block index (cluster id = pair * clusters per pair + part, K
    // parts first), and thread blocks are handed to the SMs in increasing block-index order: when a V cluster
    // starts, its K cluster is already resident or finished, whatever else shares the machine (the encoder
    // launches of kvcar_step_layer, other streams).  The flag wait is bounded all the same.
    int split = 1, kv_split = 0;
    if (tc.pbuf && 4 * n_pairs <= tc.n_sms) {
        kv_split = 1;
        if (lc.split_ok[1] && 8 * n_pairs <= tc.n_sms) split = 2;
    } else if (lc.split_ok[2] && 2 * n_pairs * 4 <= tc.n_sms) {
        split = 4;
    } else if (lc.split_ok[1] && 2 * n_pairs * 2 <= tc.n_sms) {
        split = 2;
    }
    const int group = a.hq / a.hkv;
    const int nq_local = a.hkv / split * group;
    // the absorbed forms: only where one cluster takes a pair's whole layer (no head or K/V split)
    const bool absorbed = (a.flags & KVCAR_ABSORBED) && lc.abs_ok && tc.wq && split == 1 && !kv_split && seqs.n <= tc.abs_batch;
    const bool absorbed_v = absorbed && (a.flags & KVCAR_ABSORBED_V) && lc.absv_ok && tc.ubuf && a.max_chunks <= tc.abs_max_chunks;
    tc.last_mode = absorbed_v ? 2 : absorbed ? 1 : 0;
    PairLaunch lay = make_launch(nq_local, group, lc.max_m, lc.max_in, lc.pslots,
                                 pick_nslot(nq_local, group, lc.max_m, lc.max_in, lc.pslots, absorbed_v), absorbed_v);
    lay.split = split;
    lay.n_pairs = n_pairs;
    lay.kv_split = kv_split;
    lay.epoch = ++tc.epoch;
    lay.pbuf = tc.pbuf;
    lay.pflags = tc.pflags;
    lay.parts = reinterpret_cast<const TcPart *>(tc.parts_dev) + (size_t)layer * TC_PARTS_PER_LAYER + part_index(split, 0);
    if (absorbed) {
        absorb_q_kernel<<<dim3(a.hq, seqs.n), 128, 0, st>>>(a, seqs, reinterpret_cast<__nv_bfloat16 *>(tc.wq), tc.qbias,
                                                            tc.abs_nq_pad, tc.abs_m_pad, tc.abs_batch);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        *n_launches = 2;
        lay.parts = reinterpret_cast<const TcPart *>(tc.parts_dev) + (size_t)layer * TC_PARTS_PER_LAYER + (absorbed_v ? 8 : 7);
        lay.ubuf = tc.ubuf;
        lay.m_pad_u = tc.abs_m_pad;
        lay.tm_wq = tc.tm_wq;
        lay.qbias = tc.qbias;
        lay.nq_pad = tc.abs_nq_pad;
        lay.abs_batch = tc.abs_batch;
    }
    // never less than half an SM's shared memory: two CTAs on one SM would both want all of tensor memory
    const int smem = (int)std::max(launch_bytes(lay), 120u * 1024u);
    // at most one resident cluster per SM pair; clusters walk the pairs with that stride
    const int per_pair = split * (kv_split ? 2 : 1);
    const int n_clusters = std::min(n_pairs * per_pair, std::max(per_pair, tc.n_sms / 2 / per_pair * per_pair));
    dim3 grid(2 * n_clusters);
    using Kernel = void (*)(const DecodeArgs, const SeqList, const TileIndex, const PairLaunch);
    static const Kernel kernels[4] = {decode_pair_kernel<false, false>, decode_pair_kernel<false, true>,
                                      decode_pair_kernel<true, false>, decode_pair_kernel<true, true>};
    static int configured_smem[64][4] = {};  // per device: the attribute belongs to the device's copy of the kernel
    const int ki = (lay.group_mma ? 2 : 0) + (lc.max_m <= 256 ? 1 : 0);
    int dev = 0;
    cudaGetDevice(&dev);
    const bool known = dev >= 0 && dev < 64;
    if (!known || smem > configured_smem[dev][ki]) {
        cudaError_t e = cudaFuncSetAttribute(kernels[ki], cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        if (known) configured_smem[dev][ki] = smem;
    }
    kernels[ki]<<<grid, NTHREADS, smem, st>>>(a, seqs, tix, lay);
    return cudaGetLastError();
}

}  // namespace kvcar

#ifdef KVCAR_TC_TRACE
// Trace builds only: choose the cluster whose threads record, and fetch what they recorded
// (out: [2 CTAs][4 roles][4096] entries of (clock64 << 8) | tag; n: entries per CTA and role).
extern "C" int kvcar_debug_trace_select(int cluster) {
    return (int)cudaMemcpyToSymbol(kvcar::g_trace_cluster, &cluster, sizeof(int));
}
extern "C" int kvcar_debug_trace_dump(unsigned long long *out, int *n) {
    cudaError_t e = cudaMemcpyFromSymbol(out, kvcar::g_trace, sizeof(kvcar::g_trace));
    if (e == cudaSuccess) e = cudaMemcpyFromSymbol(n, kvcar::g_trace_n, sizeof(kvcar::g_trace_n));
    return (int)e;
}
#endif
