// Decode attention over layers that store raw K/V rows (no autoencoder): the uncompressed twin of the latent
// path.  There is no decoder, so the cost is reading every cached K and V row once: the kernel is built to keep
// HBM busy, not the tensor cores.
//
// One warp owns one (sequence, 128-token tile, KV head).  K phase: lane = token; the lane reads its token's
// 64-wide K slice (128 B in 16-byte loads) and dots it with the group's pre-scaled queries (shared memory,
// broadcast reads).  Online softmax over the tile's four 32-token groups (shuffle max / sum).  V phase: lane =
// channel pair; the warp reads one V row per step (128 contiguous bytes), the row index and the probabilities
// come from the owning lane by shuffle.  The tile's (max, sum, weighted values) go to the split-KV partials;
// the combine kernel merges tiles and the exact current token.  A reused head reads the lower layer's rows.
#include "kvcar_internal.h"

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
    int width, col;
};
__device__ __forceinline__ HeadSrc find_head(const WhichPlan &wp, int h) {
    HeadSrc r{nullptr, 0, 0};
    for (int s = 0; s < wp.n_src; ++s) {
        const SourcePlan &sp = wp.src[s];
        for (int i = 0; i < sp.n_need; ++i)
            if (sp.kv_head[i] == h) {
                r.pool = sp.pool;
                r.width = sp.width;
                r.col = sp.slot[i] * 64;
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

}  // namespace

cudaError_t launch_decode_raw(const DecodeArgs &a, const SeqList &seqs, int dtype, int grid_chunks, cudaStream_t st) {
    dim3 grid(grid_chunks, (a.hkv + RW - 1) / RW, seqs.n);
    if (dtype == KVCAR_F32)
        decode_raw_kernel<float><<<grid, RW * 32, 0, st>>>(a, seqs);
    else
        decode_raw_kernel<__nv_bfloat16><<<grid, RW * 32, 0, st>>>(a, seqs);
    return cudaGetLastError();
}

}  // namespace kvcar
