// Which heads may reuse the layer below (Alg. 2, first steps): the mean absolute difference between every KV head's
// recorded rows and the same head's rows one layer down, and the choice of the closest heads from it.
//
// The distance is a pure streaming reduction over [n_layers][n_rows][n_kv_heads * head_dim] activations: HBM-bound,
// every element read once from HBM (a CTA walks the layers for its block of rows, so the layer just read is the
// "layer below" of the next step and comes out of L1).  Sums are formed in a fixed order - a thread per (row, head)
// slice, the rows of a CTA added in order, the CTAs added in order - so the result does not depend on scheduling.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <numeric>
#include <vector>

#include "kvcar_internal.h"

namespace kvcar {

namespace {

constexpr int ST_THREADS = 256;

template <typename T>
struct Chunk16;  // sum of |a - b| over the elements of two 16-byte chunks
template <>
struct Chunk16<float> {
    static constexpr int N = 4;
    static __device__ __forceinline__ float absdiff(const uint4 &a, const uint4 &b) {
        return (fabsf(__uint_as_float(a.x) - __uint_as_float(b.x)) + fabsf(__uint_as_float(a.y) - __uint_as_float(b.y))) +
               (fabsf(__uint_as_float(a.z) - __uint_as_float(b.z)) + fabsf(__uint_as_float(a.w) - __uint_as_float(b.w)));
    }
};
template <>
struct Chunk16<__nv_bfloat16> {
    static constexpr int N = 8;
    static __device__ __forceinline__ float pair(uint32_t a, uint32_t b) {
        return fabsf(__uint_as_float(a << 16) - __uint_as_float(b << 16)) +
               fabsf(__uint_as_float(a & 0xFFFF0000u) - __uint_as_float(b & 0xFFFF0000u));
    }
    static __device__ __forceinline__ float absdiff(const uint4 &a, const uint4 &b) {
        return (pair(a.x, b.x) + pair(a.y, b.y)) + (pair(a.z, b.z) + pair(a.w, b.w));
    }
};

// grid = ceil(n_rows / rows_per_cta) with rows_per_cta = ST_THREADS / hkv; thread = (row of the block, head).
// partial[cta][(l-1) * hkv + h] = sum over the CTA's rows and head h's channels of |x[l] - x[l-1]|.
constexpr int ST_LB = 8;  // layer steps between two block-wide reductions

template <typename T>
__global__ void __launch_bounds__(ST_THREADS) head_l1_kernel(const T *x, int n_layers, int64_t n_rows, int hkv, int hd,
                                                             float *partial) {
    __shared__ float val[ST_LB][ST_THREADS];
    const int rows_per_cta = ST_THREADS / hkv;
    const int tid = threadIdx.x, rl = tid / hkv, h = tid % hkv;
    const int64_t row = (int64_t)blockIdx.x * rows_per_cta + rl;
    const bool active = rl < rows_per_cta && row < n_rows;
    const int64_t width = (int64_t)hkv * hd, layer_stride = n_rows * width;
    const int nv = hd / Chunk16<T>::N;
    const uint4 *lo = reinterpret_cast<const uint4 *>(x + row * width + (int64_t)h * hd);  // layer l-1, this slice
    float *out = partial + (int64_t)blockIdx.x * (n_layers - 1) * hkv;
    for (int l0 = 1; l0 < n_layers; l0 += ST_LB) {
        const int nl = min(ST_LB, n_layers - l0);
        // ST_LB layer steps with nothing but loads and adds: the loads of consecutive steps overlap
        for (int j = 0; j < nl; ++j) {
            const uint4 *hi = reinterpret_cast<const uint4 *>(reinterpret_cast<const T *>(lo) + layer_stride);
            float s0 = 0.f, s1 = 0.f;
            if (active) {
                int v = 0;
                for (; v + 1 < nv; v += 2) {
                    const uint4 a0 = hi[v], b0 = lo[v], a1 = hi[v + 1], b1 = lo[v + 1];
                    s0 += Chunk16<T>::absdiff(a0, b0);
                    s1 += Chunk16<T>::absdiff(a1, b1);
                }
                if (v < nv) s0 += Chunk16<T>::absdiff(hi[v], lo[v]);
            }
            val[j][tid] = s0 + s1;
            lo = hi;
        }
        __syncthreads();
        // one thread per (layer step, head): the CTA's rows in order
        for (int i = tid; i < nl * hkv; i += ST_THREADS) {
            const int j = i / hkv, hh = i % hkv;
            float s = 0.f;
            for (int r = 0; r < rows_per_cta; ++r) s += val[j][r * hkv + hh];
            out[(l0 - 1 + j) * hkv + hh] = s;
        }
        __syncthreads();
    }
}

// The same sums with threads laid along a row (thread = one 16-byte chunk column, ST_RI rows each): every load
// instruction of a warp reads 512 contiguous bytes, and a thread keeps its chunks of the layer below in registers,
// so each element is loaded exactly once.  For rows of at most ST_THREADS chunks (4 KB).
constexpr int ST_RI = 8;  // rows per thread

template <typename T>
__global__ void __launch_bounds__(ST_THREADS) head_l1_rows_kernel(const T *x, int n_layers, int64_t n_rows, int hkv, int hd,
                                                                  float *partial) {
    __shared__ float val[ST_LB][ST_THREADS];
    const int cph = hd / Chunk16<T>::N, nvw = hkv * cph;  // chunks per head, per row
    const int rl_n = ST_THREADS / nvw;                    // rows side by side in the CTA
    const int tid = threadIdx.x, vcol = tid % nvw, rlane = tid / nvw;
    const int64_t row0 = (int64_t)blockIdx.x * rl_n * ST_RI + rlane;
    const bool lane_on = rlane < rl_n;
    const int64_t chunks_per_layer = n_rows * nvw;
    const uint4 *base = reinterpret_cast<const uint4 *>(x);
    float *out = partial + (int64_t)blockIdx.x * (n_layers - 1) * hkv;
    uint4 prev[ST_RI];
#pragma unroll
    for (int it = 0; it < ST_RI; ++it) {
        const int64_t row = row0 + (int64_t)it * rl_n;
        prev[it] = (lane_on && row < n_rows) ? __ldg(base + row * nvw + vcol) : make_uint4(0, 0, 0, 0);
    }
    for (int l0 = 1; l0 < n_layers; l0 += ST_LB) {
        const int nl = min(ST_LB, n_layers - l0);
        for (int j = 0; j < nl; ++j) {
            const uint4 *layer = base + (int64_t)(l0 + j) * chunks_per_layer;
            uint4 cur[ST_RI];
#pragma unroll
            for (int it = 0; it < ST_RI; ++it) {
                const int64_t row = row0 + (int64_t)it * rl_n;
                cur[it] = (lane_on && row < n_rows) ? __ldg(layer + row * nvw + vcol) : make_uint4(0, 0, 0, 0);
            }
            float s = 0.f;
#pragma unroll
            for (int it = 0; it < ST_RI; ++it) {  // rows past the end hold zeros in both layers
                s += Chunk16<T>::absdiff(cur[it], prev[it]);
                prev[it] = cur[it];
            }
            val[j][tid] = s;
        }
        __syncthreads();
        // one thread per (layer step, head): the head's chunk columns of every row lane, in order
        for (int i = tid; i < nl * hkv; i += ST_THREADS) {
            const int j = i / hkv, hh = i % hkv;
            float s = 0.f;
            for (int r = 0; r < rl_n; ++r)
                for (int k = 0; k < cph; ++k) s += val[j][r * nvw + hh * cph + k];
            out[(l0 - 1 + j) * hkv + hh] = s;
        }
        __syncthreads();
    }
}

// dist[i] = (sum over CTAs of partial[cta][i]) / count, one CTA per output: thread t adds CTAs t, t + 256, ... in
// order, then a fixed tree over the threads (the same association on every run)
__global__ void __launch_bounds__(ST_THREADS) head_l1_finish_kernel(const float *partial, int n_ctas, int n_out,
                                                                    float inv_count, float *dist) {
    __shared__ float red[ST_THREADS];
    const int i = blockIdx.x, tid = threadIdx.x;
    float s = 0.f;
    for (int c = tid; c < n_ctas; c += ST_THREADS) s += partial[(int64_t)c * n_out + i];
    red[tid] = s;
    __syncthreads();
    for (int w = ST_THREADS / 2; w > 0; w >>= 1) {
        if (tid < w) red[tid] += red[tid + w];
        __syncthreads();
    }
    if (tid == 0) dist[i] = red[0] * inv_count;
}

// CTAs the scratch is sized for: neither kernel takes fewer than ST_RI rows per CTA (row-wise: ST_RI rows per
// thread; slice per thread: ST_THREADS / n_kv_heads >= 16 rows)
int64_t l1_ctas(int, int64_t n_rows) { return (n_rows + ST_RI - 1) / ST_RI; }

bool l1_dims_ok(int n_layers, int n_kv_heads, int64_t n_rows) {
    return n_layers >= 2 && n_kv_heads >= 1 && n_kv_heads <= KVCAR_MAX_KV_HEADS && n_rows >= 1 &&
           l1_ctas(n_kv_heads, n_rows) <= 0x7fffffff;
}

}  // namespace

}  // namespace kvcar

using namespace kvcar;

extern "C" {

kvcar_status kvcar_head_l1_scratch_bytes(int32_t n_layers, int32_t n_kv_heads, int64_t n_rows, size_t *bytes) {
    if (!bytes || !l1_dims_ok(n_layers, n_kv_heads, n_rows)) return KVCAR_ERR_INVALID_ARG;
    *bytes = (size_t)l1_ctas(n_kv_heads, n_rows) * (size_t)(n_layers - 1) * (size_t)n_kv_heads * sizeof(float);
    return KVCAR_OK;
}

kvcar_status kvcar_head_l1_distance(int32_t n_layers, int32_t n_kv_heads, int32_t head_dim, int32_t storage, const void *x,
                                    int64_t n_rows, void *scratch, size_t scratch_bytes, float *dist, void *stream) {
    if (!x || !scratch || !dist || !l1_dims_ok(n_layers, n_kv_heads, n_rows)) return KVCAR_ERR_INVALID_ARG;
    if (storage != KVCAR_F32 && storage != KVCAR_BF16) return KVCAR_ERR_INVALID_ARG;
    const int per16 = storage == KVCAR_F32 ? 4 : 8;
    if (head_dim <= 0 || head_dim % per16) return KVCAR_ERR_INVALID_ARG;  // a head's slice is whole 16-byte chunks
    if (((uintptr_t)x | (uintptr_t)scratch) & 15 || ((uintptr_t)dist & 3)) return KVCAR_ERR_INVALID_ARG;
    size_t need = 0;
    kvcar_head_l1_scratch_bytes(n_layers, n_kv_heads, n_rows, &need);
    if (scratch_bytes < need) return KVCAR_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    int n_ctas = (int)((n_rows + ST_THREADS / n_kv_heads - 1) / (ST_THREADS / n_kv_heads));
    const int n_out = (n_layers - 1) * n_kv_heads;
    float *partial = reinterpret_cast<float *>(scratch);
    const int nvw = n_kv_heads * (head_dim / per16);  // 16-byte chunks per row
    const int rows_fast = nvw <= ST_THREADS ? ST_THREADS / nvw * ST_RI : 0;
    if (rows_fast > 0) {  // rows of at most 256 chunks: threads along the rows
        n_ctas = (int)((n_rows + rows_fast - 1) / rows_fast);
        if (storage == KVCAR_F32)
            head_l1_rows_kernel<float><<<n_ctas, ST_THREADS, 0, st>>>(reinterpret_cast<const float *>(x), n_layers, n_rows,
                                                                      n_kv_heads, head_dim, partial);
        else
            head_l1_rows_kernel<__nv_bfloat16><<<n_ctas, ST_THREADS, 0, st>>>(reinterpret_cast<const __nv_bfloat16 *>(x),
                                                                              n_layers, n_rows, n_kv_heads, head_dim,
                                                                              partial);
    } else if (storage == KVCAR_F32)
        head_l1_kernel<float><<<n_ctas, ST_THREADS, 0, st>>>(reinterpret_cast<const float *>(x), n_layers, n_rows,
                                                             n_kv_heads, head_dim, partial);
    else
        head_l1_kernel<__nv_bfloat16><<<n_ctas, ST_THREADS, 0, st>>>(reinterpret_cast<const __nv_bfloat16 *>(x), n_layers,
                                                                     n_rows, n_kv_heads, head_dim, partial);
    if (cudaGetLastError() != cudaSuccess) return KVCAR_ERR_CUDA;
    head_l1_finish_kernel<<<n_out, ST_THREADS, 0, st>>>(partial, n_ctas, n_out, 1.0f / ((float)n_rows * (float)head_dim),
                                                        dist);
    return cudaGetLastError() == cudaSuccess ? KVCAR_OK : KVCAR_ERR_CUDA;
}

kvcar_status kvcar_reuse_map_from_l1(const float *dist, int32_t n_layers, int32_t n_kv_heads, int32_t n_reuse,
                                     int32_t *src) {
    if (!dist || !src || n_layers < 1 || n_kv_heads < 1 || n_reuse < 0) return KVCAR_ERR_INVALID_ARG;
    const int n = (n_layers - 1) * n_kv_heads;
    if (n_reuse > n) return KVCAR_ERR_INVALID_ARG;
    for (int i = 0; i < n; ++i)
        if (std::isnan(dist[i])) return KVCAR_ERR_INVALID_ARG;
    std::vector<int> order(n);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return dist[a] < dist[b]; });
    for (int i = 0; i < n_layers * n_kv_heads; ++i) src[i] = -1;
    for (int i = 0; i < n_reuse; ++i) src[n_kv_heads + order[i]] = order[i] % n_kv_heads;
    return KVCAR_OK;
}

}  // extern "C"
