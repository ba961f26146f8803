// Decode-time encoder + append (one new token per sequence).
//
// A batch of B rows meets weights that are far larger than the rows (GPT-2 shape:
// 0.9 MB per K or V encoder), so the cost is streaming the weights once, and that
// needs the whole machine: each of the two fully connected layers is its own launch
// whose grid spreads the layer's output features over all SMs (one warp per feature:
// the lanes stream that feature's weight row in 16-byte loads and hold it against a
// block of up to 16 input rows staged in shared memory).  The hidden activations
// travel between the two launches through a small fp32 scratch in the workspace.
// Both launches use programmatic dependent launch: a kernel starts while its
// predecessor in the stream drains, fetches its first weights, and only then waits
// for the predecessor's results.
#include <algorithm>

#include "kvcar_internal.h"

namespace kvcar {

namespace {

constexpr int RB = 16;  // input rows per CTA
constexpr int NW = 8;   // warps (= output features) per CTA

template <typename T>
struct Vec16;
template <>
struct Vec16<float> {
    static constexpr int N = 4;
    static __device__ __forceinline__ uint4 load(const float *p) { return __ldg(reinterpret_cast<const uint4 *>(p)); }
    static __device__ __forceinline__ void unpack(const uint4 &v, float *w) {
        w[0] = __uint_as_float(v.x); w[1] = __uint_as_float(v.y); w[2] = __uint_as_float(v.z); w[3] = __uint_as_float(v.w);
    }
    static __device__ __forceinline__ float one(const float *p) { return __ldg(p); }
    static __device__ __forceinline__ void store(float *p, float v) { *p = v; }
};
template <>
struct Vec16<__nv_bfloat16> {
    static constexpr int N = 8;
    static __device__ __forceinline__ uint4 load(const __nv_bfloat16 *p) {
        return __ldg(reinterpret_cast<const uint4 *>(p));
    }
    static __device__ __forceinline__ void unpack(const uint4 &v, float *w) {
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

__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// acc[r] += sum over this lane's share of w[0..n) * x[r][0..n); `pre` holds the lane's first vector already
template <typename T>
__device__ __forceinline__ void lane_dots(const T *wrow, const uint4 &pre, const float *x, int n, int lane, float *acc) {
    constexpr int VL = Vec16<T>::N;
    uint4 cur = pre;
    for (int k0 = lane * VL; k0 < n; k0 += 32 * VL) {
        const int kn = k0 + 32 * VL;
        uint4 nxt = cur;
        if (kn < n) nxt = Vec16<T>::load(wrow + kn);
        float w[VL];
        Vec16<T>::unpack(cur, w);
#pragma unroll
        for (int r = 0; r < RB; ++r) {
            const float4 *xr = reinterpret_cast<const float4 *>(x + r * n + k0);
#pragma unroll
            for (int i = 0; i < VL / 4; ++i) {
                const float4 xv = xr[i];
                acc[r] = fmaf(w[4 * i + 0], xv.x, acc[r]);
                acc[r] = fmaf(w[4 * i + 1], xv.y, acc[r]);
                acc[r] = fmaf(w[4 * i + 2], xv.z, acc[r]);
                acc[r] = fmaf(w[4 * i + 3], xv.w, acc[r]);
            }
        }
        cur = nxt;
    }
}

// after the call lane r (r < RB) holds the warp-wide sum of acc[r]
__device__ __forceinline__ float reduce_rows(float *acc, int lane) {
    // fold 16 accumulators over 32 lanes: halve the accumulator count while halving the lane distance
#pragma unroll
    for (int r = 0; r < 8; ++r) {  // distance 16: lanes < 16 keep rows 0..7, lanes >= 16 keep rows 8..15
        const float keep = (lane & 16) ? acc[r + 8] : acc[r];
        const float give = (lane & 16) ? acc[r] : acc[r + 8];
        acc[r] = keep + __shfl_xor_sync(0xffffffffu, give, 16);
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const float keep = (lane & 8) ? acc[r + 4] : acc[r];
        const float give = (lane & 8) ? acc[r] : acc[r + 4];
        acc[r] = keep + __shfl_xor_sync(0xffffffffu, give, 8);
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const float keep = (lane & 4) ? acc[r + 2] : acc[r];
        const float give = (lane & 4) ? acc[r] : acc[r + 2];
        acc[r] = keep + __shfl_xor_sync(0xffffffffu, give, 4);
    }
    {
        const float keep = (lane & 2) ? acc[1] : acc[0];
        const float give = (lane & 2) ? acc[0] : acc[1];
        acc[0] = keep + __shfl_xor_sync(0xffffffffu, give, 2);
    }
    acc[0] += __shfl_xor_sync(0xffffffffu, acc[0], 1);
    // lane l now holds row ((l>>4)&1)*8 + ((l>>3)&1)*4 + ((l>>2)&1)*2 + ((l>>1)&1)
    return acc[0];
}
__device__ __forceinline__ int row_of_lane(int lane) {
    return ((lane >> 4) & 1) * 8 + ((lane >> 3) & 1) * 4 + ((lane >> 2) & 1) * 2 + ((lane >> 1) & 1);
}

// STAGE 1: hidden = LeakyReLU(BN(W1 x + b1)) -> scratch.  STAGE 2: latent = W2 hidden + b2 -> cache rows.
// grid = (ceil(features / NW), ceil(rows / RB), 2 [K, V]); block = NW warps.
template <typename T, int STAGE>
__global__ void __launch_bounds__(NW * 32)
    encode_fc_kernel(const __grid_constant__ EncodeArgs a, const __grid_constant__ SeqList seqs, float *hid, int hid_pitch,
                     int max_batch) {
    extern __shared__ __align__(16) float xs[];  // [RB][n_in]
    const int which = blockIdx.z;
    const EncPlan &pl = a.plan[which];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_rows = seqs.n, r0 = blockIdx.y * RB;
    const int in_dim = pl.in_dim, m = pl.m, d = pl.d;
    const int n_in = STAGE == 1 ? in_dim : m, n_out = STAGE == 1 ? m : d;
    const int j = blockIdx.x * NW + warp;  // this warp's output feature
    const T *src = reinterpret_cast<const T *>(which == 0 ? a.k : a.v);
    const bool compressed = pl.compressed != 0;

    // weights do not depend on anything earlier in the stream: start fetching them right away
    constexpr int VL = Vec16<T>::N;
    const T *wrow = reinterpret_cast<const T *>(STAGE == 1 ? pl.w1r : pl.w2r) + (int64_t)j * n_in;
    uint4 pre = make_uint4(0, 0, 0, 0);
    const bool active = compressed && j < n_out;
    float p0 = 0.f, p1 = 0.f;  // stage 1: fused BatchNorm scale, shift; stage 2: bias
    if (active) {
        if (lane * VL < n_in) pre = Vec16<T>::load(wrow + lane * VL);
        if (STAGE == 1) {
            p0 = pl.s1[j];
            p1 = pl.t1[j];
        } else {
            p0 = pl.b2[j];
        }
    }
    launch_dependents();
    grid_dependency_wait();  // inputs, page table and (stage 2) the hidden scratch are final from here on

    const int rows_here = min(RB, n_rows - r0);
    const int my_row = row_of_lane(lane);
    int64_t prow = -1;  // stage 2: cache row of the input row this lane will write
    if (STAGE == 2 && active && !(lane & 1) && my_row < rows_here) {
        const int seq = seqs.id[r0 + my_row], t = a.seq_len[seq];
        const int page = a.block_table[(int64_t)seq * a.max_pages_per_seq + t / a.page_tokens];
        prow = (int64_t)page * a.page_tokens + t % a.page_tokens;
    }
    if (STAGE == 1) {
        const int wv = a.kv_width / VL;  // 16-byte vectors per input row (head_dim is a multiple of the vector)
        if (blockIdx.x == 0) {  // exact current-token rows (all heads)
            for (int idx = threadIdx.x; idx < rows_here * wv; idx += blockDim.x) {
                const int rr = idx / wv, cv = idx % wv, r = r0 + rr;
                reinterpret_cast<uint4 *>(reinterpret_cast<T *>(pl.cur) + (int64_t)seqs.id[r] * a.kv_width)[cv] =
                    reinterpret_cast<const uint4 *>(src + (int64_t)r * a.kv_width)[cv];
            }
        }
        if (!compressed) {  // raw layer: copy the stored heads' slices into the cache rows, 16 bytes at a time
            T *pool = reinterpret_cast<T *>(pl.pool);
            const int nv = in_dim / VL;
            for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < rows_here * nv; idx += gridDim.x * blockDim.x) {
                const int rr = idx / nv, c = (idx % nv) * VL, r = r0 + rr;
                const int seq = seqs.id[r], t = a.seq_len[seq];
                const int page = a.block_table[(int64_t)seq * a.max_pages_per_seq + t / a.page_tokens];
                const int64_t pr = (int64_t)page * a.page_tokens + t % a.page_tokens;
                *reinterpret_cast<uint4 *>(pool + pr * pl.width + c) =
                    Vec16<T>::load(src + (int64_t)r * a.kv_width + pl.heads[c / a.hd] * a.hd + c % a.hd);
            }
            return;
        }
        if (blockIdx.x * NW >= n_out) return;
        // stage the stored heads' slices of this block's rows as fp32, 16 bytes per load, four loads in flight
        const int nv = in_dim / VL, total = rows_here * nv;
        for (int base = threadIdx.x; base < total; base += 4 * blockDim.x) {
            uint4 v[4];
            int dst[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int idx = base + u * blockDim.x;
                dst[u] = -1;
                if (idx < total) {
                    const int rr = idx / nv, c = (idx % nv) * VL;
                    v[u] = Vec16<T>::load(src + (int64_t)(r0 + rr) * a.kv_width + pl.heads[c / a.hd] * a.hd + c % a.hd);
                    dst[u] = rr * in_dim + c;
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (dst[u] >= 0) {
                    float w[VL];
                    Vec16<T>::unpack(v[u], w);
#pragma unroll
                    for (int i = 0; i < VL; i += 4)
                        *reinterpret_cast<float4 *>(xs + dst[u] + i) = make_float4(w[i], w[i + 1], w[i + 2], w[i + 3]);
                }
        }
        for (int idx = rows_here * in_dim + threadIdx.x; idx < RB * in_dim; idx += blockDim.x) xs[idx] = 0.f;
    } else {
        if (!compressed || blockIdx.x * NW >= n_out) return;
        const float *h = hid + ((int64_t)which * max_batch + r0) * hid_pitch;
        const int nv = m / 4, total = rows_here * nv;
        for (int base = threadIdx.x; base < total; base += 4 * blockDim.x) {
            float4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int idx = base + u * blockDim.x;
                if (idx < total) v[u] = *reinterpret_cast<const float4 *>(h + (int64_t)(idx / nv) * hid_pitch + (idx % nv) * 4);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int idx = base + u * blockDim.x;
                if (idx < total) *reinterpret_cast<float4 *>(xs + (idx / nv) * m + (idx % nv) * 4) = v[u];
            }
        }
        for (int idx = rows_here * m + threadIdx.x; idx < RB * m; idx += blockDim.x) xs[idx] = 0.f;
    }
    __syncthreads();
    if (!active) return;
    float acc[RB];
#pragma unroll
    for (int r = 0; r < RB; ++r) acc[r] = 0.f;
    lane_dots<T>(wrow, pre, xs, n_in, lane, acc);
    const float sum = reduce_rows(acc, lane);
    if ((lane & 1) || my_row >= rows_here) return;
    if (STAGE == 1) {
        float hv = fmaf(sum, p0, p1);
        hv = hv > 0.f ? hv : hv * pl.slope;
        hid[((int64_t)which * max_batch + r0 + my_row) * hid_pitch + j] = hv;
    } else {
        Vec16<T>::store(reinterpret_cast<T *>(pl.pool) + prow * pl.width + j, sum + p0);
    }
}

template <typename T, int STAGE>
cudaError_t launch_stage(const EncodeArgs &a, const SeqList &seqs, float *hid, int hid_pitch, int max_batch, int n_out_max,
                         int n_in_max, cudaStream_t st) {
    const size_t smem = (size_t)RB * n_in_max * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(encode_fc_kernel<T, STAGE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((n_out_max + NW - 1) / NW, (seqs.n + RB - 1) / RB, 2);
    cfg.blockDim = dim3(NW * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, encode_fc_kernel<T, STAGE>, a, seqs, hid, hid_pitch, max_batch);
}

}  // namespace

size_t encode_split_smem(int max_in, int max_m) { return (size_t)RB * std::max(max_in, max_m) * sizeof(float); }

cudaError_t launch_encode_split(const EncodeArgs &a, const SeqList &seqs, int dtype, int max_in, int max_m, int max_d,
                                float *hid, int max_batch, cudaStream_t st) {
    cudaError_t e;
    const int n_hidden = std::max(max_m, NW);  // raw layers still need one block column for the copy
    if (dtype == KVCAR_F32) {
        e = launch_stage<float, 1>(a, seqs, hid, max_m, max_batch, n_hidden, max_in, st);
        if (e == cudaSuccess && max_m > 0) e = launch_stage<float, 2>(a, seqs, hid, max_m, max_batch, max_d, max_m, st);
    } else {
        e = launch_stage<__nv_bfloat16, 1>(a, seqs, hid, max_m, max_batch, n_hidden, max_in, st);
        if (e == cudaSuccess && max_m > 0)
            e = launch_stage<__nv_bfloat16, 2>(a, seqs, hid, max_m, max_batch, max_d, max_m, st);
    }
    return e;
}

}  // namespace kvcar
