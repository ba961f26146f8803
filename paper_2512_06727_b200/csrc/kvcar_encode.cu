// Decode-time encoder + append (one new token per sequence).
//
// A batch of B rows meets weights that are far larger than the rows (GPT-2 shape:
// 0.9 MB per K or V encoder), so the cost is streaming the weights once, and one
// SM cannot stream them fast enough.  A cluster of 8 CTAs shares each block of 8
// rows: every CTA computes one eighth of the hidden features (one warp per
// feature row of FC1, lanes over the input dimension, 16-byte loads), broadcasts
// its slice of the activated hidden vector into all 8 CTAs' shared memory, and
// after a cluster barrier computes one eighth of the latent features the same way.
#include "kvcar_internal.h"

namespace kvcar {

namespace {

constexpr int CR = 8;     // rows per cluster
constexpr int CSIZE = 8;  // CTAs per cluster
constexpr int NW = 8;     // warps per CTA

template <typename T>
struct Ld16;
template <>
struct Ld16<float> {
    static constexpr int N = 4;
    static __device__ __forceinline__ void load(const float *p, float *w) {
        float4 v = __ldg(reinterpret_cast<const float4 *>(p));
        w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
    }
    static __device__ __forceinline__ float one(const float *p) { return __ldg(p); }
    static __device__ __forceinline__ void store(float *p, float v) { *p = v; }
};
template <>
struct Ld16<__nv_bfloat16> {
    static constexpr int N = 8;
    static __device__ __forceinline__ void load(const __nv_bfloat16 *p, float *w) {
        uint4 v = __ldg(reinterpret_cast<const uint4 *>(p));
        const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            w[2 * i] = __uint_as_float(u[i] << 16);
            w[2 * i + 1] = __uint_as_float(u[i] & 0xFFFF0000u);
        }
    }
    static __device__ __forceinline__ float one(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
    static __device__ __forceinline__ void store(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }
};

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// one warp: dot products of weight row `wrow` (length n) with CR activation rows in shared memory
template <typename T>
__device__ __forceinline__ void warp_dots(const T *wrow, const float *x, int n, int lane, float *acc) {
    constexpr int VL = Ld16<T>::N;
#pragma unroll
    for (int r = 0; r < CR; ++r) acc[r] = 0.f;
    for (int k0 = lane * VL; k0 < n; k0 += 32 * VL) {
        float w[VL];
        Ld16<T>::load(wrow + k0, w);
#pragma unroll
        for (int r = 0; r < CR; ++r) {
            const float4 *xr = reinterpret_cast<const float4 *>(x + r * n + k0);
#pragma unroll
            for (int i = 0; i < VL / 4; ++i) {
                float4 xv = xr[i];
                acc[r] = fmaf(w[4 * i + 0], xv.x, acc[r]);
                acc[r] = fmaf(w[4 * i + 1], xv.y, acc[r]);
                acc[r] = fmaf(w[4 * i + 2], xv.z, acc[r]);
                acc[r] = fmaf(w[4 * i + 3], xv.w, acc[r]);
            }
        }
    }
#pragma unroll
    for (int r = 0; r < CR; ++r) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc[r] += __shfl_xor_sync(0xffffffffu, acc[r], o);
    }
}

template <typename T>
__global__ void __cluster_dims__(CSIZE, 1, 1) __launch_bounds__(NW * 32)
    encode_cluster_kernel(const __grid_constant__ EncodeArgs a, const __grid_constant__ SeqList seqs) {
    extern __shared__ __align__(16) float smem[];
    const int which = blockIdx.y;
    const EncPlan &pl = a.plan[which];
    const int rank = blockIdx.x % CSIZE, r0 = (blockIdx.x / CSIZE) * CR;
    const int n_rows = seqs.n;
    const int in_dim = pl.in_dim, m = pl.m, d = pl.d;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float *xs = smem;                // [CR][in_dim]
    float *hs = smem + CR * in_dim;  // [CR][m], filled by all CTAs of the cluster
    __shared__ int64_t rows[CR];
    const T *src = reinterpret_cast<const T *>(which == 0 ? a.k : a.v);

    if (threadIdx.x < CR) {
        const int r = r0 + threadIdx.x;
        int64_t row = -1;
        if (r < n_rows) {
            const int seq = seqs.id[r];
            const int t = a.seq_len[seq];
            const int page = a.block_table[(int64_t)seq * a.max_pages_per_seq + t / a.page_tokens];
            row = (int64_t)page * a.page_tokens + t % a.page_tokens;
        }
        rows[threadIdx.x] = row;
    }
    if (rank == 0) {  // exact current-token rows (all heads)
        for (int idx = threadIdx.x; idx < CR * a.kv_width; idx += blockDim.x) {
            const int rr = idx / a.kv_width, c = idx % a.kv_width, r = r0 + rr;
            if (r < n_rows)
                reinterpret_cast<T *>(pl.cur)[(int64_t)seqs.id[r] * a.kv_width + c] = src[(int64_t)r * a.kv_width + c];
        }
    }
    for (int idx = threadIdx.x; idx < CR * in_dim; idx += blockDim.x) {
        const int rr = idx / in_dim, c = idx % in_dim, r = r0 + rr;
        float v = 0.f;
        if (r < n_rows) v = Ld16<T>::one(src + (int64_t)r * a.kv_width + pl.heads[c / a.hd] * a.hd + c % a.hd);
        xs[idx] = v;
    }
    __syncthreads();
    T *pool = reinterpret_cast<T *>(pl.pool);
    if (!pl.compressed) {  // raw layer: copy (whole cluster takes this branch, nobody waits on anybody)
        if (rank == 0)
            for (int idx = threadIdx.x; idx < CR * in_dim; idx += blockDim.x)
                if (rows[idx / in_dim] >= 0) Ld16<T>::store(pool + rows[idx / in_dim] * pl.width + idx % in_dim, xs[idx]);
        return;
    }
    // every CTA of the cluster is running (its shared memory may be written) past this point
    asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
    // ---- FC1 + BatchNorm + LeakyReLU: this CTA's slice of the hidden features ----
    {
        const int per = (m + CSIZE - 1) / CSIZE;
        const int j_hi = min(m, (rank + 1) * per);
        const T *w1 = reinterpret_cast<const T *>(pl.w1r);
        const int my_row = lane & 7, peer0 = lane >> 3;  // lane -> (row, two of the eight CTAs)
        for (int j = rank * per + warp; j < j_hi; j += NW) {
            float acc[CR];
            warp_dots<T>(w1 + (int64_t)j * in_dim, xs, in_dim, lane, acc);
            float mine = 0.f;
#pragma unroll
            for (int r = 0; r < CR; ++r) mine = (my_row == r) ? acc[r] : mine;
            float h = fmaf(mine, pl.s1[j], pl.t1[j]);
            h = h > 0.f ? h : h * pl.slope;
            const uint32_t local = smem_addr(hs + my_row * m + j);
#pragma unroll
            for (int pp = 0; pp < 2; ++pp) {
                uint32_t remote;
                asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(peer0 + 4 * pp));
                asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(h) : "memory");
            }
        }
    }
    asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
    // ---- FC2: this CTA's slice of the latent features, rounded and appended ----
    {
        const int per = (d + CSIZE - 1) / CSIZE;
        const int o_hi = min(d, (rank + 1) * per);
        const T *w2 = reinterpret_cast<const T *>(pl.w2r);
        for (int o = rank * per + warp; o < o_hi; o += NW) {
            float acc[CR];
            warp_dots<T>(w2 + (int64_t)o * m, hs, m, lane, acc);
            float mine = 0.f;
#pragma unroll
            for (int r = 0; r < CR; ++r) mine = (lane == r) ? acc[r] : mine;
            if (lane < CR && rows[lane] >= 0) Ld16<T>::store(pool + rows[lane] * pl.width + o, mine + pl.b2[o]);
        }
    }
}

}  // namespace

cudaError_t launch_encode_cluster(const EncodeArgs &a, const SeqList &seqs, int dtype, int max_in, int max_m,
                                  cudaStream_t st) {
    dim3 grid(CSIZE * ((seqs.n + CR - 1) / CR), 2);
    const size_t smem = (size_t)CR * (max_in + max_m) * sizeof(float);
    cudaError_t e;
    if (dtype == KVCAR_F32) {
        e = cudaFuncSetAttribute(encode_cluster_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        encode_cluster_kernel<float><<<grid, NW * 32, smem, st>>>(a, seqs);
    } else {
        e = cudaFuncSetAttribute(encode_cluster_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem);
        if (e != cudaSuccess) return e;
        encode_cluster_kernel<__nv_bfloat16><<<grid, NW * 32, smem, st>>>(a, seqs);
    }
    return cudaGetLastError();
}

}  // namespace kvcar
