// Bulk encoder + append on the tensor cores (many new tokens per sequence: cache prefill).
//
// The two fully connected layers of the encoder are two launches of one tiled product kernel:
//   stage 1   H[rows x m]  = X[rows x in_dim] . W1[m x in_dim]^T ; a = LeakyReLU(H * s + t) -> bf16 -> scratch
//   stage 2   Z[rows x d]  = A[rows x m] . W2[d x m]^T ; z = Z + b2 -> bf16 -> the rows' places in the page pool
// X is the caller's K (or V) buffer, read through a tensor map built for the call: K slab ks of X is the 64-wide
// slice of stored head ks.  A pair of CTAs (a cluster of two) owns a 256-row x (<= 256)-column output tile, CTA r its
// rows 128 r ..: each loads its own rows of the row operand and its half of the tile's weight rows, and the leader
// issues every product as one tcgen05.mma.cta_group::2 of M = 256, so a weight tile crosses L2 -> shared memory once
// per 256 rows and a k-step costs each SM 32 KB of loads instead of 48 (the one-CTA form was bound by those loads).
// Per CTA two TMA producer warps, an MMA warp (the leader's issues) and eight epilogue warps; five operand stages and
// two accumulator buffers; a pair walks several tiles, its epilogue of one under the products of the next.
// Unlike the decode-time encoder, the hidden activations pass through bf16 here (they are an operand of the second
// product), so a latent written by this path may differ from the fp32-hidden one by a few bf16 ulps of its scale.
// All waits are bounded and record a code in the status word.
#include <cuda.h>

#include <algorithm>
#include <cstring>

#include "kvcar_internal.h"
#include "kvcar_ptx.cuh"

namespace kvcar {

using namespace ptx;

namespace {

constexpr int PF_M = 128;          // rows per CTA
constexpr int PF_N = 256;          // columns per CTA at most
constexpr int PF_STAGES = 5;       // 32 KB each: one CTA per SM
constexpr int PF_A_BYTES = PF_M * 128;   // one 64-wide K slab of the row tile (bf16, 128-byte rows)
constexpr int PF_B_BYTES = (PF_N / 2) * 128;  // this CTA's half of the column tile's weight rows
constexpr int PF_STAGE_BYTES = PF_A_BYTES + PF_B_BYTES;
constexpr int PF_EPI_WARPS = 8;    // two per tensor-memory lane quarter: even and odd 64-column blocks
constexpr int PF_THREADS = 32 * (3 + PF_EPI_WARPS);  // warp 0 producer (row operand), warp 1 MMA + tensor memory,
                                                     // warps 2-9 epilogue, warp 10 producer (weights)
constexpr int PF_SMEM = PF_STAGES * PF_STAGE_BYTES + 1024 /* alignment */ + 128 /* barriers */ +
                        PF_EPI_WARPS * 4096 /* store staging, 32 rows x 128 B per epilogue warp */;

struct PfArgs {
    const EncPlan *plan;         // [2]: K then V (device)
    const int32_t *block_table;
    const int32_t *seq_len;
    int32_t *status;
    const void *src[2];          // the caller's K and V rows [n_rows_total][kv_width] (stage 1: exact current rows)
    __nv_bfloat16 *hid;          // scratch [2][hid_rows][hid_pitch]
    int32_t hid_rows, hid_pitch;
    int32_t max_pages_per_seq, page_tokens;
    int32_t n_tokens, kv_width;
    int32_t row0, n_rows_blk;    // this launch covers rows row0 .. row0 + n_rows_blk - 1 of the call
};

// bounded wait: 2 s, then the kernel records `code` and carries on to its exit (results are then meaningless)
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int32_t *status, int code) {
    if (mbar_try(bar, parity)) return true;
    uint32_t n = 0;
    uint64_t t0 = 0;
    while (true) {
        __nanosleep(32);
        if (mbar_try(bar, parity)) return true;
        if ((++n & 255u) == 0) {
            const uint64_t now = global_ns();
            if (t0 == 0) t0 = now;
            if (now - t0 > 2000000000ull) {
                atomicCAS(status, 0, code);
                return false;
            }
        }
    }
}

// grid = (2 x clusters, 1, 2 [K, V]); STAGE 1 or 2 as in the file header.  A cluster walks the output tiles of its K or V
// (tile t = row pair t / n_ct, column tile t % n_ct: the column tiles of a row pair follow each other, so its rows are
// re-read from L2) with the stride of the cluster count; the operand ring and the two accumulator buffers run on
// across tiles, so the producer and the issuer are in the next tile while the epilogue warps drain the last one.
template <int STAGE>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(PF_THREADS, 1)
    prefill_fc_kernel(const __grid_constant__ CUtensorMap map_a0, const __grid_constant__ CUtensorMap map_a1,
                      const __grid_constant__ CUtensorMap map_b0, const __grid_constant__ CUtensorMap map_b1,
                      const __grid_constant__ PfArgs a, const __grid_constant__ SeqList seqs) {
    extern __shared__ uint8_t pf_smem[];
    __shared__ uint32_t tmem_slot;
    __shared__ __align__(16) float prm[2][PF_N];  // the tile's columns of scale and shift (stage 1) or bias (stage 2)
    const int which = blockIdx.z;
    const EncPlan &pl = a.plan[which];
    const int kdim = STAGE == 1 ? pl.in_dim : pl.m, ndim = STAGE == 1 ? pl.m : pl.d;
    const uint32_t rank = blockIdx.x & 1u;
    const bool leader = rank == 0;
    const int cluster = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const CUtensorMap *map_a = which == 0 ? &map_a0 : &map_a1;
    const CUtensorMap *map_b = which == 0 ? &map_b0 : &map_b1;
    const uint32_t base = (smem_u32(pf_smem) + 1023u) & ~1023u;
    const uint32_t bars = base + PF_STAGES * PF_STAGE_BYTES;  // full[S] (leader's are used), empty[S], acc_full[2], acc_empty[2]
    const uint32_t bar_accf = bars + 16 * PF_STAGES, bar_acce = bar_accf + 16;
    const uint32_t stage_base = bars + 128;  // 128-byte aligned (the stages are 1024-byte multiples)
    const int n_slabs = (kdim + 63) >> 6;
    const int n_ct = (ndim + PF_N - 1) / PF_N;
    const int n_tiles = ((a.n_rows_blk + 2 * PF_M - 1) / (2 * PF_M)) * n_ct;

    if (threadIdx.x == 0) {
        for (int i = 0; i < PF_STAGES; ++i) {
            mbar_init(bars + 8 * i, 1);
            mbar_init(bars + 8 * (PF_STAGES + i), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar_accf + 8 * i, 1);
            mbar_init(bar_acce + 8 * i, 2 * PF_EPI_WARPS);  // the epilogue warps of both CTAs (leader's copy is the one used)
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {  // both accumulator buffers; one CTA per SM (shared memory), so every CTA gets columns 0..511
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(512u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // both CTAs' barriers exist before either signals the other's
    tc_fence_after();
    const uint32_t tmem = tmem_slot;

    if (warp == 0 || warp == 2 + PF_EPI_WARPS) {
        // two producers share a k-step's loads (a tensor load costs its thread ~100 cycles here): warp 0 the row operand,
        // the last warp the weights; both wait for the stage, the leader's warp 0 announces the bytes of both CTAs
        const bool rows_side = warp == 0;
        if (elect_one()) {
            uint32_t g = 0;  // k-steps issued so far: stage g % S, in its (g / S)-th use
            bool ok = true;
            for (int t = cluster; t < n_tiles && ok; t += n_clusters) {
                const int n0 = (t % n_ct) * PF_N, r0 = (t / n_ct) * 2 * PF_M + (int)rank * PF_M;
                const int nt = min(PF_N, ndim - n0), half = nt >> 1;  // this CTA supplies `half` weight rows
                const int b_boxes = (half + 63) >> 6;                 // in 64-row boxes; rows past the half are never read
                for (int ks = 0; ks < n_slabs; ++ks, ++g) {
                    const uint32_t s = g % PF_STAGES, use = g / PF_STAGES;
                    if (use > 0 && !mbar_wait(bars + 8 * (PF_STAGES + s), (use - 1u) & 1u, a.status, 0x401)) {
                        ok = false;
                        break;
                    }
                    const uint32_t sa = base + s * PF_STAGE_BYTES, sb = sa + PF_A_BYTES;
                    const uint32_t full = map_to_cta(bars + 8 * s, 0);  // the leader's barrier counts both CTAs' bytes
                    if (leader && rows_side) mbar_expect_tx(bars + 8 * s, 2u * (2u * 8192u + (uint32_t)b_boxes * 8192u));
                    // stage 1: K slab ks of X is stored head ks's 64-wide slice; stage 2: columns 64 ks.. of the scratch
                    const int ax = STAGE == 1 ? pl.heads[ks] * 64 : 64 * ks;
                    const int ay = STAGE == 1 ? a.row0 + r0 : which * a.hid_rows + r0;
                    if (rows_side) {
                        tma_load_2d_pair(sa, map_a, ax, ay, full);
                        tma_load_2d_pair(sa + 8192, map_a, ax, ay + 64, full);
                    } else {
                        for (int i = 0; i < b_boxes; ++i)
                            tma_load_2d_pair(sb + 8192 * i, map_b, 64 * ks, n0 + (int)rank * half + 64 * i, full);
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (leader && elect_one()) {
            uint32_t g = 0, it = 0;
            bool ok = true;
            for (int t = cluster; t < n_tiles && ok; t += n_clusters, ++it) {
                const int n0 = (t % n_ct) * PF_N;
                const int nt = min(PF_N, ndim - n0);
                const uint32_t idesc = make_idesc(2 * PF_M, nt);
                const uint32_t buf = it & 1u, acc = tmem + 256u * buf;
                // the epilogue warps of both CTAs are done with this buffer's previous tile
                if (it >= 2 && !mbar_wait(bar_acce + 8 * buf, ((it >> 1) - 1u) & 1u, a.status, 0x404)) break;
                tc_fence_after();
                for (int ks = 0; ks < n_slabs; ++ks, ++g) {
                    const uint32_t s = g % PF_STAGES, use = g / PF_STAGES;
                    if (!mbar_wait(bars + 8 * s, use & 1u, a.status, 0x402)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t sa = base + s * PF_STAGE_BYTES, sb = sa + PF_A_BYTES;
                    const uint64_t da = make_desc(sa), db = make_desc(sb);
                    const int nk = min(4, (kdim - 64 * ks) >> 4);
                    for (int k = 0; k < nk; ++k) {
                        if (ks | k)
                            umma_pair<1>(acc, da + 2u * k, db + 2u * k, idesc);
                        else
                            umma_pair<0>(acc, da + 2u * k, db + 2u * k, idesc);
                    }
                    umma_commit_pair(bars + 8 * (PF_STAGES + s));  // the stage is free in both CTAs once these products are done
                }
                if (ok) umma_commit_pair(bar_accf + 8 * buf);
            }
        }
    } else if (warp < 2 + PF_EPI_WARPS) {
        // epilogue: thread = one row of the CTA's half of the tile (tensor-memory lane quarter = warp % 4) and every
        // other block of 64 columns
        const int q = warp & 3, rl = 32 * q + lane, chalf = (warp - 2) >> 2;
        const uint32_t acce_leader = map_to_cta(bar_acce, 0);
        const float slope = pl.slope;
        uint32_t it = 0;
        for (int t = cluster; t < n_tiles; t += n_clusters, ++it) {
            const int n0 = (t % n_ct) * PF_N, r0 = (t / n_ct) * 2 * PF_M + (int)rank * PF_M;
            const int nt = min(PF_N, ndim - n0);
            const uint32_t buf = it & 1u, acc = tmem + 256u * buf;
            const int64_t r = (int64_t)a.row0 + r0 + rl;           // row of the call
            const bool row_ok = r0 + rl < a.n_rows_blk;
            const int si = row_ok ? (int)(r / a.n_tokens) : 0, tk = row_ok ? (int)(r % a.n_tokens) : 0;
            const int seq = seqs.id[si];
            if (STAGE == 1 && n0 == 0 && chalf == 0 && row_ok && tk == a.n_tokens - 1) {
                // the sequence's newest token: keep its exact row (all heads) as the layer's current token
                const uint4 *s4 = reinterpret_cast<const uint4 *>(reinterpret_cast<const __nv_bfloat16 *>(a.src[which]) +
                                                                  r * a.kv_width);
                uint4 *d4 = reinterpret_cast<uint4 *>(reinterpret_cast<__nv_bfloat16 *>(pl.cur) + (int64_t)seq * a.kv_width);
                for (int i = 0; i < a.kv_width / 8; ++i) d4[i] = s4[i];
            }
            __nv_bfloat16 *dst;
            if (STAGE == 1) {
                dst = a.hid + ((int64_t)which * a.hid_rows + r0 + rl) * a.hid_pitch + n0;
            } else {
                const int tok = a.seq_len[seq] + tk;
                const int64_t prow =
                    (int64_t)a.block_table[(int64_t)seq * a.max_pages_per_seq + tok / a.page_tokens] * a.page_tokens +
                    tok % a.page_tokens;
                dst = reinterpret_cast<__nv_bfloat16 *>(pl.pool) + prow * pl.width + n0;
            }
            {
                const float *g0 = STAGE == 1 ? pl.s1 + n0 : pl.b2 + n0;
                const float *g1 = STAGE == 1 ? pl.t1 + n0 : nullptr;
                asm volatile("bar.sync 1, 256;" ::: "memory");  // the last tile's reads of the parameters are over
                for (int i = threadIdx.x - 64; i < nt; i += 32 * PF_EPI_WARPS) {
                    prm[0][i] = g0[i];
                    if (STAGE == 1) prm[1][i] = g1[i];
                }
                asm volatile("bar.sync 1, 256;" ::: "memory");
            }
            if (!mbar_wait(bar_accf + 8 * buf, (it >> 1) & 1u, a.status, 0x403)) break;
            tc_fence_after();
            // 64 columns (a 128-byte row segment) at a time, the two warps of a lane quarter alternating.  A thread owns a
            // row, so storing from registers would touch 32 rows with 16 bytes each per instruction; the 32 x 128-byte block
            // goes through a swizzled staging area of the warp instead and leaves as whole 128-byte lines, four rows per
            // instruction (lane = 8 l_row + chunk).
            const uint32_t stg = stage_base + (uint32_t)(warp - 2) * 4096u;
            const uint64_t dst_bits = reinterpret_cast<uint64_t>(dst);
            for (int b64 = chalf; 64 * b64 < nt; b64 += 2) {
#pragma unroll
                for (int hg = 0; hg < 2; ++hg) {
                    const int g = 2 * b64 + hg;
                    if (32 * g >= nt) break;  // warp-uniform
                    float v[32];
                    tmem_ld32(acc + ((uint32_t)(32 * q) << 16) + 32u * g, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int c8 = 0; c8 < 4; ++c8) {
                        const int c = 32 * g + 8 * c8;
                        if (c >= nt) break;
                        float o[8], pa[8], pb[8];
                        *reinterpret_cast<float4 *>(pa) = *reinterpret_cast<const float4 *>(&prm[0][c]);
                        *reinterpret_cast<float4 *>(pa + 4) = *reinterpret_cast<const float4 *>(&prm[0][c + 4]);
                        if (STAGE == 1) {
                            *reinterpret_cast<float4 *>(pb) = *reinterpret_cast<const float4 *>(&prm[1][c]);
                            *reinterpret_cast<float4 *>(pb + 4) = *reinterpret_cast<const float4 *>(&prm[1][c + 4]);
                        }
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const float x = v[8 * c8 + e];
                            if (STAGE == 1) {
                                const float y = fmaf(x, pa[e], pb[e]);
                                o[e] = y > 0.f ? y : y * slope;
                            } else {
                                o[e] = x + pa[e];
                            }
                        }
                        const uint32_t chunk = (uint32_t)(4 * hg + c8);  // 16-byte chunk of the row's 128-byte segment
                        const uint32_t addr = stg + (uint32_t)lane * 128u + ((chunk ^ ((uint32_t)lane & 7u)) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(pack_bf16(o[0], o[1])),
                                     "r"(pack_bf16(o[2], o[3])), "r"(pack_bf16(o[4], o[5])), "r"(pack_bf16(o[6], o[7]))
                                     : "memory");
                    }
                }
                __syncwarp();
                const uint32_t chunk = (uint32_t)lane & 7u;
                const bool col_ok = 64 * b64 + 8 * (int)chunk < nt;  // widths are multiples of 16: whole chunks
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int rr = 4 * i + (lane >> 3);  // row of the warp's 32
                    const uint64_t d_row = __shfl_sync(0xffffffffu, dst_bits, rr);
                    const int ok_row = __shfl_sync(0xffffffffu, (int)row_ok, rr);
                    uint32_t w0, w1, w2, w3;
                    const uint32_t addr = stg + (uint32_t)rr * 128u + ((chunk ^ ((uint32_t)rr & 7u)) << 4);
                    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(w0), "=r"(w1), "=r"(w2), "=r"(w3) : "r"(addr) : "memory");
                    if (ok_row && col_ok)
                        *reinterpret_cast<uint4 *>(reinterpret_cast<__nv_bfloat16 *>(d_row) + 64 * b64 + 8 * (int)chunk) =
                            make_uint4(w0, w1, w2, w3);
                }
                __syncwarp();  // the staging area is free for the next block
            }
            // this warp is done reading the buffer: one arrival of the sixteen the issuer waits for
            tc_fence_before();
            __syncwarp();
            if (elect_one()) mbar_arrive_remote(acce_leader + 8 * buf);
        }
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // nobody leaves while the peer may still signal this CTA's barriers or read its operands
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
}

// bf16 matrix [rows][cols] with `pitch` elements between rows -> [64 rows][64 cols] boxes, 128B swizzle, zero fill
bool make_map(CUtensorMap *m, const void *ptr, uint64_t rows, uint64_t cols, uint64_t pitch) {
    static EncodeTiledFn fn = tensor_map_encoder();
    return fn != nullptr && encode_bf16_map(fn, m, ptr, rows, cols, pitch);
}

}  // namespace

size_t prefill_tc_scratch_bytes(int max_m) {
    const int pitch = (max_m + 63) & ~63;
    return (size_t)2 * PREFILL_TC_ROWS * pitch * sizeof(__nv_bfloat16);
}

cudaError_t launch_prefill_tc(const PrefillTcArgs &h, const SeqList &seqs, cudaStream_t st) {
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(prefill_fc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, PF_SMEM);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(prefill_fc_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, PF_SMEM);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    const int pitch = (h.max_m + 63) & ~63;
    const int64_t n_rows = (int64_t)seqs.n * h.n_tokens;
    CUtensorMap ax[2], ah[2], w1[2], w2[2];
    for (int w = 0; w < 2; ++w) {
        const EncPlan &pl = h.plan_host[w];
        if (!make_map(&ax[w], h.src[w], (uint64_t)n_rows, (uint64_t)h.kv_width, (uint64_t)h.kv_width) ||
            !make_map(&ah[w], h.hid, (uint64_t)2 * PREFILL_TC_ROWS, (uint64_t)pitch, (uint64_t)pitch) ||
            !make_map(&w1[w], pl.w1r, (uint64_t)pl.m, (uint64_t)pl.in_dim, (uint64_t)pl.in_dim) ||
            !make_map(&w2[w], pl.w2r, (uint64_t)pl.d, (uint64_t)pl.m, (uint64_t)pl.m))
            return cudaErrorInvalidValue;
    }
    const int max_m = std::max(h.plan_host[0].m, h.plan_host[1].m), max_d = std::max(h.plan_host[0].d, h.plan_host[1].d);
    for (int64_t row0 = 0; row0 < n_rows; row0 += PREFILL_TC_ROWS) {
        PfArgs a{};
        a.plan = h.plan_dev;
        a.block_table = h.block_table;
        a.seq_len = h.seq_len;
        a.status = h.status;
        a.src[0] = h.src[0];
        a.src[1] = h.src[1];
        a.hid = reinterpret_cast<__nv_bfloat16 *>(h.hid);
        a.hid_rows = PREFILL_TC_ROWS;
        a.hid_pitch = pitch;
        a.max_pages_per_seq = h.max_pages_per_seq;
        a.page_tokens = h.page_tokens;
        a.n_tokens = h.n_tokens;
        a.kv_width = h.kv_width;
        a.row0 = (int32_t)row0;
        a.n_rows_blk = (int32_t)std::min<int64_t>(PREFILL_TC_ROWS, n_rows - row0);
        // 37 clusters per K or V (every SM pair of the device between them), fewer when there are fewer tiles
        const int row_pairs = (a.n_rows_blk + 2 * PF_M - 1) / (2 * PF_M);
        const unsigned c1 = (unsigned)std::min(37, row_pairs * ((max_m + PF_N - 1) / PF_N));
        const unsigned c2 = (unsigned)std::min(37, row_pairs * ((max_d + PF_N - 1) / PF_N));
        prefill_fc_kernel<1><<<dim3(2 * c1, 1, 2), PF_THREADS, PF_SMEM, st>>>(ax[0], ax[1], w1[0], w1[1], a, seqs);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        prefill_fc_kernel<2><<<dim3(2 * c2, 1, 2), PF_THREADS, PF_SMEM, st>>>(ah[0], ah[1], w2[0], w2[1], a, seqs);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace kvcar
