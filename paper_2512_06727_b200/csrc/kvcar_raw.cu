// Decode attention over layers that store raw K/V rows (no autoencoder): the uncompressed twin of the latent
// path.  There is no decoder, so the cost is reading every cached K and V row once: the kernels are built to keep
// HBM busy.  One warp owns one (sequence, 128-token tile, KV head); the tile's (max, sum, weighted values) go to
// the split-KV partials; the combine kernel merges tiles and the exact current token.  A reused head reads the
// lower layer's rows.
//
// bf16 rows (decode_raw_gq_kernel, below): 32 tokens at a time through shared memory into the warp-level tensor
// op, for every group size (a group of one query head is padded like any other; the products are nowhere near
// the limit).
//
// fp32 rows (decode_raw_kernel): K phase with lane = token; the lane reads its token's 64-wide K slice in 16-byte
// loads and dots it with the group's pre-scaled queries (shared memory, broadcast reads).  Online softmax over
// the tile's four 32-token groups (shuffle max / sum).  V phase: lane = channel pair; the warp reads one V row
// per step, the row index and the probabilities come from the owning lane through shared memory.
#include <cuda.h>

#include "kvcar_internal.h"
#include "kvcar_ptx.cuh"

namespace kvcar {

namespace {

constexpr int RT = 128;  // tokens per tile (= split-KV chunk)
constexpr int RW = 4;    // warps (= KV heads) per CTA

template <typename T>
struct Row64;
template <>
struct Row64<__nv_bfloat16> {
    // 64 values of one token and head -> fp32
    static __device__ __forceinline__ void load(const __nv_bfloat16 *p, float *x) {
        const uint4 *q = reinterpret_cast<const uint4 *>(p);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint4 v = __ldg(q + i);
            const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                x[8 * i + 2 * j] = __uint_as_float(u[j] << 16);
                x[8 * i + 2 * j + 1] = __uint_as_float(u[j] & 0xFFFF0000u);
            }
        }
    }
    static __device__ __forceinline__ float2 load2(const __nv_bfloat16 *p) {  // two adjacent channels
        const uint32_t u = __ldg(reinterpret_cast<const uint32_t *>(p));
        return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xFFFF0000u));
    }
    static __device__ __forceinline__ float one(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
};
template <>
struct Row64<float> {
    static __device__ __forceinline__ void load(const float *p, float *x) {
        const float4 *q = reinterpret_cast<const float4 *>(p);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const float4 v = __ldg(q + i);
            x[4 * i] = v.x; x[4 * i + 1] = v.y; x[4 * i + 2] = v.z; x[4 * i + 3] = v.w;
        }
    }
    static __device__ __forceinline__ float2 load2(const float *p) { return __ldg(reinterpret_cast<const float2 *>(p)); }
    static __device__ __forceinline__ float one(const float *p) { return __ldg(p); }
};

// where KV head h of this layer reads its rows: pool base, row width, first column
struct HeadSrc {
    const void *pool;
    int width, col, src_layer;
};
__device__ __forceinline__ HeadSrc find_head(const WhichPlan &wp, int h) {
    HeadSrc r{nullptr, 0, 0, 0};
    for (int s = 0; s < wp.n_src; ++s) {
        const SourcePlan &sp = wp.src[s];
        for (int i = 0; i < sp.n_need; ++i)
            if (sp.kv_head[i] == h) {
                r.pool = sp.pool;
                r.width = sp.width;
                r.col = sp.slot[i] * 64;
                r.src_layer = sp.src_layer;
            }
    }
    return r;
}

// grid = (tiles, ceil(hkv / RW), n_seqs); block = RW warps; head_dim 64, at most 8 query heads per KV head
template <typename T>
__global__ void __launch_bounds__(RW * 32, 4) decode_raw_kernel(const __grid_constant__ DecodeArgs a,
                                                             const __grid_constant__ SeqList seqs) {
    __shared__ __align__(16) float qs[RW][8][64];
    __shared__ __align__(16) float ps[RW][8][32];  // probabilities of the current 32-token group
    __shared__ int64_t rows[RW][32];                // and their cache rows
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tile = blockIdx.x, h = blockIdx.y * RW + warp, si = blockIdx.z;
    if (h >= a.hkv) return;
    const int seq = seqs.id[si];
    const int L = a.seq_len[seq];
    const int t0 = tile * RT;
    if (t0 >= L) return;
    const int valid = min(RT, L - t0);
    const int group = a.hq / a.hkv;
    const HeadSrc ks = find_head(a.plan->w[0], h), vs = find_head(a.plan->w[1], h);
    const T *kpool = reinterpret_cast<const T *>(ks.pool) + ks.col;
    const T *vpool = reinterpret_cast<const T *>(vs.pool) + vs.col + 2 * lane;

    const T *qg = reinterpret_cast<const T *>(a.q) + ((int64_t)si * a.hq + h * group) * 64;
    for (int i = lane; i < group * 64; i += 32) qs[warp][i >> 6][i & 63] = Row64<T>::one(qg + i) * a.scale;
    __syncwarp();

    float m[8], l[8];
    float2 o[8];
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        m[g] = -INFINITY;
        l[g] = 0.f;
        o[g] = make_float2(0.f, 0.f);
    }
    const int32_t *bt = a.block_table + (int64_t)seq * a.max_pages_per_seq;
    for (int grp = 0; grp * 32 < valid; ++grp) {
        const int n_here = min(32, valid - 32 * grp);
        const bool ok = lane < n_here;
        const int t = t0 + 32 * grp + (ok ? lane : 0);
        const int64_t row = (int64_t)bt[t / a.page_tokens] * a.page_tokens + t % a.page_tokens;
        float p[8];
        {
            float x[64];
            Row64<T>::load(kpool + row * ks.width, x);
#pragma unroll
            for (int g = 0; g < 8; ++g) {
                if (g < group) {
                    const float4 *q4 = reinterpret_cast<const float4 *>(qs[warp][g]);
                    float d0 = 0.f, d1 = 0.f, d2 = 0.f, d3 = 0.f;
#pragma unroll
                    for (int c = 0; c < 16; ++c) {
                        const float4 qq = q4[c];
                        d0 = fmaf(x[4 * c], qq.x, d0);
                        d1 = fmaf(x[4 * c + 1], qq.y, d1);
                        d2 = fmaf(x[4 * c + 2], qq.z, d2);
                        d3 = fmaf(x[4 * c + 3], qq.w, d3);
                    }
                    p[g] = ok ? (d0 + d1) + (d2 + d3) : -INFINITY;
                }
            }
        }
#pragma unroll
        for (int g = 0; g < 8; ++g) {
            if (g < group) {
                float mx = p[g];
#pragma unroll
                for (int s = 16; s > 0; s >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, s));
                const float m_new = fmaxf(m[g], mx);
                const float corr = m[g] == -INFINITY ? 0.f : __expf(m[g] - m_new);
                p[g] = ok ? __expf(p[g] - m_new) : 0.f;
                float ps = p[g];
#pragma unroll
                for (int s = 16; s > 0; s >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, s);
                l[g] = l[g] * corr + ps;
                o[g].x *= corr;
                o[g].y *= corr;
                m[g] = m_new;
            }
        }
        // V: one row per step, eight rows in flight; row indices and probabilities come through shared memory
        // (probabilities of lanes past the tile's end are zero, their row is a valid one)
        __syncwarp();
        rows[warp][lane] = row;
#pragma unroll
        for (int g = 0; g < 8; ++g)
            if (g < group) ps[warp][g][lane] = p[g];
        __syncwarp();
        for (int tt = 0; tt < n_here; tt += 8) {
            float2 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = Row64<T>::load2(vpool + rows[warp][(tt + u) & 31] * vs.width);
#pragma unroll
            for (int g = 0; g < 8; ++g) {
                if (g < group) {
                    const float4 pa = *reinterpret_cast<const float4 *>(&ps[warp][g][tt]);
                    const float4 pb = *reinterpret_cast<const float4 *>(&ps[warp][g][tt + 4]);
                    o[g].x = fmaf(pa.x, v[0].x, o[g].x); o[g].y = fmaf(pa.x, v[0].y, o[g].y);
                    o[g].x = fmaf(pa.y, v[1].x, o[g].x); o[g].y = fmaf(pa.y, v[1].y, o[g].y);
                    o[g].x = fmaf(pa.z, v[2].x, o[g].x); o[g].y = fmaf(pa.z, v[2].y, o[g].y);
                    o[g].x = fmaf(pa.w, v[3].x, o[g].x); o[g].y = fmaf(pa.w, v[3].y, o[g].y);
                    o[g].x = fmaf(pb.x, v[4].x, o[g].x); o[g].y = fmaf(pb.x, v[4].y, o[g].y);
                    o[g].x = fmaf(pb.y, v[5].x, o[g].x); o[g].y = fmaf(pb.y, v[5].y, o[g].y);
                    o[g].x = fmaf(pb.z, v[6].x, o[g].x); o[g].y = fmaf(pb.z, v[6].y, o[g].y);
                    o[g].x = fmaf(pb.w, v[7].x, o[g].x); o[g].y = fmaf(pb.w, v[7].y, o[g].y);
                }
            }
        }
    }
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        if (g < group) {
            float *part = a.partials + (((int64_t)si * a.max_chunks + tile) * a.hq + h * group + g) * (64 + 2);
            if (lane == 0) {
                part[0] = m[g];
                part[1] = l[g];
            }
            *reinterpret_cast<float2 *>(part + 2 + 2 * lane) = o[g];
        }
    }
}

// ---------------------------------------------------------------------------------------------------------
// bf16 rows.  With several query heads per KV head the dots of a group against a row are a small matrix product,
// and on the CUDA cores they, not HBM, set the pace (8 heads: 1024 FMA per cached row and KV head); and even with
// one head per group a warp that walks its tile with plain loads keeps too few bytes in flight.  Same
// decomposition (one warp per sequence, 128-token tile and KV head), but 32 tokens at a time go through shared
// memory (cp.async, 16-byte chunks swizzled by row, the next 32 tokens in flight meanwhile) into the warp-level
// tensor op: scores^T[8 queries x 8 tokens] = Q . K^T with the K rows as the "column-major" operand they already
// are; the probabilities come out in the layout the next product wants as its row operand (queries x tokens), and
// V enters through transposing matrix loads.  Online softmax across the four 32-token steps, fp32.  Groups of
// fewer than 8 heads leave the other operand rows zero.
// TMA build: where a 32-token step lies inside one page (page size a multiple of 32) and the pools have tensor
// maps, one elected lane fetches a step with two tensor loads (a 32-row x 64-column box of the K pool and of the V
// pool, 128-byte swizzle: the same layout the cp.async build writes by hand) that count their bytes on a barrier
// of the warp, instead of sixteen 16-byte copies and eight page-table look-ups per lane.  (Requesting
// the whole tile at once - four buffers per warp - halves the resident warps and measured slower at every size.)
constexpr int GQ_STEP = 32;                      // tokens per step
constexpr int GQ_BUF = GQ_STEP * 64 * 2;         // bytes of one K (or V) step buffer: 32 rows x 128 B
constexpr int GQ_WARP_SMEM = 4 * GQ_BUF;         // K and V, two steps each
constexpr int GQ_RW = 2;                         // warps (= KV heads) per CTA: small CTAs pack the SMs evenly
constexpr int GQ_SMEM = GQ_RW * GQ_WARP_SMEM;

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t *r) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t *r) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
// D[16 x 8] += A[16 x 16] . B[16 x 8], bf16 in, fp32 out; rows 8..15 of A are zero here (a1 = a3 = 0)
__device__ __forceinline__ void mma_q8(float *d, uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %5}, {%7, %8}, {%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(0u), "r"(a2), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&v);
}

template <bool TMA>
__global__ void __launch_bounds__(GQ_RW * 32) decode_raw_gq_kernel(const __grid_constant__ DecodeArgs a,
                                                               const __grid_constant__ SeqList seqs) {
    extern __shared__ __align__(128) uint8_t gq_smem[];
    __shared__ __align__(8) uint64_t step_bar[GQ_RW][2];  // TMA build: bytes of a step buffer pair have landed
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tile = blockIdx.x, h = blockIdx.y * GQ_RW + warp, si = blockIdx.z;
    if (h >= a.hkv) return;
    const int seq = seqs.id[si];
    const int L = a.seq_len[seq];
    const int t0 = tile * RT;
    if (t0 >= L) return;
    const int valid = min(RT, L - t0);
    const int group = a.hq / a.hkv;
    const HeadSrc ks = find_head(a.plan->w[0], h), vs = find_head(a.plan->w[1], h);
    const __nv_bfloat16 *kpool = reinterpret_cast<const __nv_bfloat16 *>(ks.pool) + ks.col;
    const __nv_bfloat16 *vpool = reinterpret_cast<const __nv_bfloat16 *>(vs.pool) + vs.col;
    const int32_t *bt = a.block_table + (int64_t)seq * a.max_pages_per_seq;
    // K step buffers 0, 1, then V step buffers 0, 1 (1024-byte aligned: the swizzle pattern of the tensor loads is a
    // function of the address)
    const uint32_t sbase = ((smem_addr(gq_smem) + 1023u) & ~1023u) + warp * GQ_WARP_SMEM;
    uint8_t *gbase = gq_smem + (sbase - smem_addr(gq_smem));
    const uint32_t bar0 = smem_addr(&step_bar[warp][0]);
    const char *kmap = nullptr, *vmap = nullptr;
    if (TMA) {
        kmap = reinterpret_cast<const char *>(a.raw_tmaps) + (size_t)(ks.src_layer * 2) * 384;
        vmap = reinterpret_cast<const char *>(a.raw_tmaps) + (size_t)(vs.src_layer * 2 + 1) * 384;
        if (lane == 0) {
            ptx::mbar_init(bar0, 1);
            ptx::mbar_init(bar0 + 8, 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        ptx::fence_async_smem();
        __syncwarp();
    }
    const int g = lane >> 2, t = lane & 3;

    // this lane's part of the row operand Q[16 x 64] (rows >= group are zero): per 16-channel step, channels
    // 2t, 2t+1 and 2t+8, 2t+9 of query g
    uint32_t qa[4][2];
    {
        const __nv_bfloat16 *qg = reinterpret_cast<const __nv_bfloat16 *>(a.q) + ((int64_t)si * a.hq + h * group + g) * 64;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            qa[k][0] = g < group ? __ldg(reinterpret_cast<const uint32_t *>(qg + 16 * k + 2 * t)) : 0u;
            qa[k][1] = g < group ? __ldg(reinterpret_cast<const uint32_t *>(qg + 16 * k + 8 + 2 * t)) : 0u;
        }
    }
    // fetch one 32-token step: lane = (row within a group of four, 16-byte chunk); rows past the tile's end re-read
    // the tile's first row (their probabilities are zero)
    auto fetch = [&](int step, int buf) {
        if (TMA) {
            if (ptx::elect_one()) {
                const int tok = t0 + GQ_STEP * step;  // the step's 32 tokens lie in one page
                const int row = bt[tok / a.page_tokens] * a.page_tokens + tok % a.page_tokens;
                ptx::mbar_expect_tx(bar0 + 8 * buf, 2 * GQ_BUF);
                ptx::tma_load_2d(sbase + buf * GQ_BUF, kmap, ks.col, row, bar0 + 8 * buf);
                ptx::tma_load_2d(sbase + (2 + buf) * GQ_BUF, vmap, vs.col, row, bar0 + 8 * buf);
            }
            return;
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int r = 4 * i + (lane >> 3), c = lane & 7;
            int tok = t0 + GQ_STEP * step + r;
            if (tok >= t0 + valid) tok = t0;
            const int64_t row = (int64_t)bt[tok / a.page_tokens] * a.page_tokens + tok % a.page_tokens;
            const uint32_t off = (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4));
            cp_async16(sbase + buf * GQ_BUF + off, kpool + row * ks.width + 8 * c);
            cp_async16(sbase + (2 + buf) * GQ_BUF + off, vpool + row * vs.width + 8 * c);
        }
        cp_async_commit();
    };

    float m_run = -INFINITY, l_run = 0.f;  // of query g (the four lanes of a group hold copies)
    float o[8][4];                         // o[n][0..1]: query g, channels 8n + 2t, 8n + 2t + 1
#pragma unroll
    for (int n = 0; n < 8; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
    const int n_steps = (valid + GQ_STEP - 1) / GQ_STEP;
    fetch(0, 0);
    for (int step = 0; step < n_steps; ++step) {
        const int buf = step & 1;
        if (step + 1 < n_steps) fetch(step + 1, buf ^ 1);
        if (TMA) {
            // bounded like every wait on a barrier in this library: on expiry a code goes to the status word and the
            // warp carries on to its normal exit
            uint32_t n = 0;
            uint64_t t_start = 0;
            while (!ptx::mbar_try(bar0 + 8 * buf, (uint32_t)(step >> 1) & 1u)) {
                if ((++n & 255u) == 0) {
                    const uint64_t now = ptx::global_ns();
                    if (t_start == 0) t_start = now;
                    if (now - t_start > 2000000000ull) {
                        atomicCAS(a.status, 0, 0x501);
                        break;
                    }
                }
            }
            // rows past the tile's end hold whatever the page holds: their probabilities are zero, but zero times a
            // stray NaN is not, so they are cleared
            const int r_end = valid - GQ_STEP * step;
            if (r_end < GQ_STEP && lane >= r_end) {
                uint4 *kr = reinterpret_cast<uint4 *>(gbase + buf * GQ_BUF + lane * 128);
                uint4 *vr = reinterpret_cast<uint4 *>(gbase + (2 + buf) * GQ_BUF + lane * 128);
#pragma unroll
                for (int i = 0; i < 8; ++i) kr[i] = vr[i] = make_uint4(0u, 0u, 0u, 0u);
            }
        } else if (step + 1 < n_steps) {
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncwarp();
        const uint32_t kb = sbase + buf * GQ_BUF, vb = sbase + (2 + buf) * GQ_BUF;
        // scores^T: four blocks of 8 tokens; sc[nt][0..1] = query g, tokens 8 nt + 2t, + 1
        float sc[4][4];
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
            const int r = 8 * nt + (lane & 7);
#pragma unroll
            for (int kp = 0; kp < 2; ++kp) {  // two 16-channel steps per matrix load
                uint32_t b[4];
                ldmatrix_x4(kb + r * 128 + (((4 * kp + (lane >> 3)) ^ (r & 7)) << 4), b);
                mma_q8(sc[nt], qa[2 * kp][0], qa[2 * kp][1], b[0], b[1]);
                mma_q8(sc[nt], qa[2 * kp + 1][0], qa[2 * kp + 1][1], b[2], b[3]);
            }
        }
        // online softmax of query g over this step's 32 tokens
        float mx = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int tok = GQ_STEP * step + 8 * nt + 2 * t + e;
                sc[nt][e] = tok < valid ? sc[nt][e] * a.scale : -INFINITY;
                mx = fmaxf(mx, sc[nt][e]);
            }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m_run, mx);  // finite: the step holds at least one valid token
        const float corr = m_run == -INFINITY ? 0.f : __expf(m_run - m_new);
        float psum = 0.f;
        uint32_t pa[2][2];  // the probabilities as row operand: [16-token step][tokens 2t.. | 2t+8..]
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            const float p0 = __expf(sc[nt][0] - m_new), p1 = __expf(sc[nt][1] - m_new);
            psum += p0 + p1;
            pa[nt >> 1][nt & 1] = pack2_bf16(p0, p1);
        }
        psum += __shfl_xor_sync(0xffffffffu, psum, 1);
        psum += __shfl_xor_sync(0xffffffffu, psum, 2);
        l_run = l_run * corr + psum;
        m_run = m_new;
#pragma unroll
        for (int n = 0; n < 8; ++n) {
            o[n][0] *= corr;
            o[n][1] *= corr;
        }
        // weighted values: two 16-token steps x eight 8-channel blocks (two blocks per transposing matrix load)
#pragma unroll
        for (int kk = 0; kk < 2; ++kk) {
            const int r = 16 * kk + 8 * ((lane >> 3) & 1) + (lane & 7);
#pragma unroll
            for (int np = 0; np < 4; ++np) {
                uint32_t b[4];
                ldmatrix_x4_trans(vb + r * 128 + (((2 * np + (lane >> 4)) ^ (r & 7)) << 4), b);
                mma_q8(o[2 * np], pa[kk][0], pa[kk][1], b[0], b[1]);
                mma_q8(o[2 * np + 1], pa[kk][0], pa[kk][1], b[2], b[3]);
            }
        }
        __syncwarp();  // every lane is done reading this step's buffers before the step after next refills them
    }
    if (g < group) {
        float *part = a.partials + (((int64_t)si * a.max_chunks + tile) * a.hq + h * group + g) * (64 + 2);
        if (t == 0) {
            part[0] = m_run;
            part[1] = l_run;
        }
#pragma unroll
        for (int n = 0; n < 8; ++n) *reinterpret_cast<float2 *>(part + 2 + 8 * n + 2 * t) = make_float2(o[n][0], o[n][1]);
    }
}

}  // namespace

bool raw_build_map(void *dst_host, const void *pool_dev, uint64_t rows, uint64_t width) {
    static EncodeTiledFn fn = tensor_map_encoder();
    if (!fn || width % 8 != 0) return false;
    return encode_bf16_map(fn, dst_host, pool_dev, rows, width, width, GQ_STEP);
}

cudaError_t launch_decode_raw(const DecodeArgs &a, const SeqList &seqs, int dtype, int grid_chunks, cudaStream_t st) {
    dim3 grid(grid_chunks, (a.hkv + RW - 1) / RW, seqs.n);
    if (dtype == KVCAR_BF16) {
        static bool configured[64] = {};  // per device: the attribute belongs to the device's copy of the kernel
        int dev = 0;
        cudaGetDevice(&dev);
        constexpr int smem = GQ_SMEM + 1024;  // + room to align the step buffers
        if (dev < 0 || dev >= 64 || !configured[dev]) {
            cudaError_t e = cudaFuncSetAttribute(decode_raw_gq_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            if (e == cudaSuccess)
                e = cudaFuncSetAttribute(decode_raw_gq_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            if (e != cudaSuccess) return e;
            if (dev >= 0 && dev < 64) configured[dev] = true;
        }
        grid.y = (a.hkv + GQ_RW - 1) / GQ_RW;
        if (a.raw_tmaps && a.page_tokens % GQ_STEP == 0)
            decode_raw_gq_kernel<true><<<grid, GQ_RW * 32, smem, st>>>(a, seqs);
        else
            decode_raw_gq_kernel<false><<<grid, GQ_RW * 32, smem, st>>>(a, seqs);
        return cudaGetLastError();
    }
    if (dtype == KVCAR_F32)
        decode_raw_kernel<float><<<grid, RW * 32, 0, st>>>(a, seqs);
    else
        decode_raw_kernel<__nv_bfloat16><<<grid, RW * 32, 0, st>>>(a, seqs);
    return cudaGetLastError();
}

}  // namespace kvcar
