// Generic (fp32 FMA) kernels of the KV-CAR decode path: table maintenance,
// encoder + append, decoder + attention over one chunk of cached tokens, and the
// split-KV combine.  They handle every supported shape in both storage types and
// are the fp32-mode path; the bf16 tensor-core kernel lives in kvcar_tc.cu.
#include "kvcar_internal.h"

namespace kvcar {

namespace {

template <typename T>
__device__ __forceinline__ float ld(const T *p);
template <>
__device__ __forceinline__ float ld<float>(const float *p) {
    return __ldg(p);
}
template <>
__device__ __forceinline__ float ld<__nv_bfloat16>(const __nv_bfloat16 *p) {
    return __bfloat162float(*p);
}
template <typename T>
__device__ __forceinline__ void st(T *p, float v);
template <>
__device__ __forceinline__ void st<float>(float *p, float v) {
    *p = v;
}
template <>
__device__ __forceinline__ void st<__nv_bfloat16>(__nv_bfloat16 *p, float v) {
    *p = __float2bfloat16_rn(v);
}

__device__ __forceinline__ float lrelu(float a, float slope) { return a > 0.f ? a : a * slope; }

// logical token -> pool row
__device__ __forceinline__ int64_t pool_row(const int32_t *block_table, int max_pages_per_seq, int P, int seq,
                                            int token) {
    int page = block_table[(int64_t)seq * max_pages_per_seq + token / P];
    return (int64_t)page * P + token % P;
}

// ---------------------------------------------------------------------------
__global__ void table_update_kernel(int32_t *block_table, int32_t *seq_len, const __grid_constant__ TableUpdates u) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= u.n) return;
    int4 e = u.e[i];
    if (e.x == 0)
        block_table[(int64_t)e.y * u.max_pages_per_seq + e.z] = e.w;
    else
        seq_len[e.y] = e.w;
}

// ---------------------------------------------------------------------------
// Encoder + append.  grid = (ceil(rows/ER), 2 [K,V]); block = 256.
// Each block pushes ER rows through FC -> (BN as scale/shift) -> LeakyReLU -> FC
// and writes the rounded latent rows into the page pool.
constexpr int ER = 8;

template <typename T>
__global__ void __launch_bounds__(256) encode_generic_kernel(const __grid_constant__ EncodeArgs a,
                                                             const __grid_constant__ SeqList seqs) {
    extern __shared__ float smem[];
    const int which = blockIdx.y;
    const EncPlan &pl = a.plan[which];
    const int n_rows = seqs.n * a.n_tokens;
    const int r0 = blockIdx.x * ER;
    const int in_dim = pl.in_dim, m = pl.m, d = pl.d;
    float *xs = smem;                 // [ER][in_dim]
    float *hs = smem + ER * in_dim;   // [ER][m]
    __shared__ int64_t rows[ER];
    const T *src = reinterpret_cast<const T *>(which == 0 ? a.k : a.v);

    if (threadIdx.x < ER) {
        int r = r0 + threadIdx.x;
        int64_t row = -1;
        if (r < n_rows) {
            int si = r / a.n_tokens, t = r % a.n_tokens;
            int seq = seqs.id[si];
            row = pool_row(a.block_table, a.max_pages_per_seq, a.page_tokens, seq, a.seq_len[seq] + t);
        }
        rows[threadIdx.x] = row;
    }
    // gather the stored heads' slices; keep the last token's full exact row as the current token
    for (int idx = threadIdx.x; idx < ER * a.kv_width; idx += blockDim.x) {
        int rr = idx / a.kv_width, c = idx % a.kv_width;
        int r = r0 + rr;
        if (r >= n_rows) continue;
        int si = r / a.n_tokens, t = r % a.n_tokens;
        if (t == a.n_tokens - 1) {
            T *cur = reinterpret_cast<T *>(pl.cur) + (int64_t)seqs.id[si] * a.kv_width;
            cur[c] = src[(int64_t)r * a.kv_width + c];
        }
    }
    for (int idx = threadIdx.x; idx < ER * in_dim; idx += blockDim.x) {
        int rr = idx / in_dim, c = idx % in_dim;
        int r = r0 + rr;
        float v = 0.f;
        if (r < n_rows) {
            int head = pl.heads[c / a.hd];
            v = ld(src + (int64_t)r * a.kv_width + head * a.hd + c % a.hd);
        }
        xs[rr * in_dim + c] = v;
    }
    __syncthreads();
    T *pool = reinterpret_cast<T *>(pl.pool);
    if (!pl.compressed) {
        for (int idx = threadIdx.x; idx < ER * in_dim; idx += blockDim.x) {
            int rr = idx / in_dim, c = idx % in_dim;
            if (rows[rr] >= 0) st(pool + rows[rr] * pl.width + c, xs[idx]);
        }
        return;
    }
    const T *w1t = reinterpret_cast<const T *>(pl.w1t);
    for (int j = threadIdx.x; j < m; j += blockDim.x) {
        float acc[ER];
#pragma unroll
        for (int r = 0; r < ER; ++r) acc[r] = 0.f;
        for (int k = 0; k < in_dim; ++k) {
            float w = ld(w1t + (int64_t)k * m + j);
#pragma unroll
            for (int r = 0; r < ER; ++r) acc[r] = fmaf(xs[r * in_dim + k], w, acc[r]);
        }
        float s = pl.s1[j], t = pl.t1[j];
#pragma unroll
        for (int r = 0; r < ER; ++r) hs[r * m + j] = lrelu(fmaf(acc[r], s, t), pl.slope);
    }
    __syncthreads();
    const T *w2t = reinterpret_cast<const T *>(pl.w2t);
    for (int j = threadIdx.x; j < d; j += blockDim.x) {
        float acc[ER];
#pragma unroll
        for (int r = 0; r < ER; ++r) acc[r] = 0.f;
        for (int k = 0; k < m; ++k) {
            float w = ld(w2t + (int64_t)k * d + j);
#pragma unroll
            for (int r = 0; r < ER; ++r) acc[r] = fmaf(hs[r * m + k], w, acc[r]);
        }
        float b = pl.b2[j];
        if (pl.qparam) {  // int8 rows: the whole row is needed before any code can be written
#pragma unroll
            for (int r = 0; r < ER; ++r) xs[r * in_dim + j] = acc[r] + b;  // d <= in_dim (checked at bind time)
        } else {
#pragma unroll
            for (int r = 0; r < ER; ++r)
                if (rows[r] >= 0) st(pool + rows[r] * pl.width + j, acc[r] + b);
        }
    }
    if (!pl.qparam) return;
    // Eq. 4 per cached row: scale = 255/(max-min), zero-point = -round(scale*min) - 128,
    // code = round(scale*x + zero-point) kept inside int8.  One warp per row (ER = warps per block).
    __syncthreads();
    const int r = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (rows[r] < 0) return;
    const float *z = xs + r * in_dim;
    float lo = INFINITY, hi = -INFINITY;
    for (int j = lane; j < d; j += 32) {
        lo = fminf(lo, z[j]);
        hi = fmaxf(hi, z[j]);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
        hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    float scale, zp;
    if (hi > lo) {
        scale = 255.f / (hi - lo);
        zp = -rintf(scale * lo) - 128.f;
    } else {  // a row of equal values has no range: code 0 with zero-point -x restores it exactly
        scale = 1.f;
        zp = -lo;
    }
    int8_t *codes = reinterpret_cast<int8_t *>(pl.pool) + rows[r] * pl.width;
    for (int j = lane; j < d; j += 32) {
        float q = hi > lo ? fminf(fmaxf(rintf(fmaf(scale, z[j], zp)), -128.f), 127.f) : 0.f;
        codes[j] = (int8_t)(int)q;
    }
    if (lane == 0) {
        pl.qparam[rows[r] * 2] = scale;
        pl.qparam[rows[r] * 2 + 1] = zp;
    }
}

// ---------------------------------------------------------------------------
// Decoder + attention over one chunk of cached tokens.
// grid = (max_chunks, n_seqs); block = 256.  The chunk is walked in sub-tiles of
// TOK tokens with an online softmax; the chunk's (max, sum, acc) per query head
// goes to `partials` for the combine kernel.
constexpr int TOK = 32;
constexpr int NT = 256;

struct GenSmem {
    float *zT;    // [max_d][TOK]   latent sub-tile, transposed
    float *hT;    // [max_m][TOK]   activated hidden sub-tile, transposed
    float *kh;    // [TOK][hd+1]    one restored head slice
    float *q;     // [hq][hd]
    float *S;     // [hq][TOK]      scores, then probabilities
    float *acc;   // [hq][hd]
    float *mx;    // [hq]
    float *sum;   // [hq]
    float *corr;  // [hq]
};

__host__ __device__ inline size_t gen_smem_floats(int hq, int hd, int max_d, int max_m) {
    return (size_t)max_d * TOK + (size_t)max_m * TOK + (size_t)TOK * (hd + 1) + (size_t)hq * hd + (size_t)hq * TOK +
           (size_t)hq * hd + 3 * (size_t)hq;
}

// restore head `slot` of a compressed source from hT, or fetch it from a raw source, into kh[TOK][hd+1]
template <typename T>
__device__ void restore_head(const SourcePlan &sp, const GenSmem &sm, int slot, int hd, const int64_t *rows,
                             int valid) {
    const int tid = threadIdx.x;
    if (sp.compressed) {
        const T *w2t = reinterpret_cast<const T *>(sp.w2t);
        // thread -> (column c, token group of 8)
        for (int o = tid; o < hd * (TOK / 8); o += NT) {
            int c = o % hd, tg = o / hd;
            float acc[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] = 0.f;
            const T *wp = w2t + slot * hd + c;
            for (int j = 0; j < sp.m; ++j) {
                float w = ld(wp + (int64_t)j * sp.in_dim);
                const float4 *h4 = reinterpret_cast<const float4 *>(sm.hT + j * TOK + tg * 8);
                float4 h0 = h4[0], h1 = h4[1];
                acc[0] = fmaf(h0.x, w, acc[0]); acc[1] = fmaf(h0.y, w, acc[1]);
                acc[2] = fmaf(h0.z, w, acc[2]); acc[3] = fmaf(h0.w, w, acc[3]);
                acc[4] = fmaf(h1.x, w, acc[4]); acc[5] = fmaf(h1.y, w, acc[5]);
                acc[6] = fmaf(h1.z, w, acc[6]); acc[7] = fmaf(h1.w, w, acc[7]);
            }
            float b = sp.b2[slot * hd + c];
#pragma unroll
            for (int i = 0; i < 8; ++i) sm.kh[(tg * 8 + i) * (hd + 1) + c] = acc[i] + b;
        }
    } else {
        const T *pool = reinterpret_cast<const T *>(sp.pool);
        for (int o = tid; o < hd * TOK; o += NT) {
            int c = o % hd, t = o / hd;
            float v = 0.f;
            if (t < valid) v = ld(pool + rows[t] * sp.width + slot * hd + c);
            sm.kh[t * (hd + 1) + c] = v;
        }
    }
}

// load a compressed source's latent sub-tile and run decoder FC1 + BN + LeakyReLU into hT
template <typename T>
__device__ void hidden_tile(const SourcePlan &sp, const GenSmem &sm, const int64_t *rows, int valid) {
    const int tid = threadIdx.x;
    const T *pool = reinterpret_cast<const T *>(sp.pool);
    if (sp.qparam) {  // int8 rows (Eq. 4, last line): x = (code - zero-point) / scale
        const int8_t *codes = reinterpret_cast<const int8_t *>(sp.pool);
        for (int o = tid; o < sp.d * TOK; o += NT) {
            int k = o % sp.d, t = o / sp.d;
            float v = 0.f;
            if (t < valid) {
                const float scale = sp.qparam[rows[t] * 2], zp = sp.qparam[rows[t] * 2 + 1];
                v = ((float)codes[rows[t] * sp.width + k] - zp) / scale;
            }
            sm.zT[k * TOK + t] = v;
        }
    } else {
        for (int o = tid; o < sp.d * TOK; o += NT) {
            int k = o % sp.d, t = o / sp.d;
            float v = 0.f;
            if (t < valid) v = ld(pool + rows[t] * sp.width + k);
            sm.zT[k * TOK + t] = v;
        }
    }
    __syncthreads();
    const T *w1t = reinterpret_cast<const T *>(sp.w1t);
    for (int j = tid; j < sp.m; j += NT) {
        float acc[TOK];
#pragma unroll
        for (int i = 0; i < TOK; ++i) acc[i] = 0.f;
        for (int k = 0; k < sp.d; ++k) {
            float w = ld(w1t + (int64_t)k * sp.m + j);
            const float4 *z4 = reinterpret_cast<const float4 *>(sm.zT + k * TOK);
#pragma unroll
            for (int i = 0; i < TOK / 4; ++i) {
                float4 z = z4[i];
                acc[4 * i + 0] = fmaf(z.x, w, acc[4 * i + 0]);
                acc[4 * i + 1] = fmaf(z.y, w, acc[4 * i + 1]);
                acc[4 * i + 2] = fmaf(z.z, w, acc[4 * i + 2]);
                acc[4 * i + 3] = fmaf(z.w, w, acc[4 * i + 3]);
            }
        }
        float s = sp.s1[j], t = sp.t1[j];
#pragma unroll
        for (int i = 0; i < TOK; ++i) sm.hT[j * TOK + i] = lrelu(fmaf(acc[i], s, t), sp.slope);
    }
    __syncthreads();
}

template <typename T>
__global__ void __launch_bounds__(NT) decode_generic_kernel(const __grid_constant__ DecodeArgs a,
                                                            const __grid_constant__ SeqList seqs, int max_d,
                                                            int max_m) {
    extern __shared__ float smem[];
    const int tid = threadIdx.x;
    const int chunk = blockIdx.x, si = blockIdx.y;
    const int seq = seqs.id[si];
    const int L = a.seq_len[seq];
    const int t_begin = chunk * a.chunk_tokens;
    if (t_begin >= L) return;
    const int t_end = min(L, t_begin + a.chunk_tokens);
    const int hq = a.hq, hd = a.hd, group = a.hq / a.hkv;

    GenSmem sm;
    float *p = smem;
    sm.zT = p;   p += (size_t)max_d * TOK;
    sm.hT = p;   p += (size_t)max_m * TOK;
    sm.kh = p;   p += (size_t)TOK * (hd + 1);
    sm.q = p;    p += (size_t)hq * hd;
    sm.S = p;    p += (size_t)hq * TOK;
    sm.acc = p;  p += (size_t)hq * hd;
    sm.mx = p;   p += hq;
    sm.sum = p;  p += hq;
    sm.corr = p;
    __shared__ int64_t rows[TOK];

    const T *qg = reinterpret_cast<const T *>(a.q) + (int64_t)si * hq * hd;
    for (int i = tid; i < hq * hd; i += NT) {
        sm.q[i] = ld(qg + i);
        sm.acc[i] = 0.f;
    }
    for (int i = tid; i < hq; i += NT) {
        sm.mx[i] = -INFINITY;
        sm.sum[i] = 0.f;
    }
    const LayerPlan &lp = *a.plan;

    for (int t0 = t_begin; t0 < t_end; t0 += TOK) {
        const int valid = min(TOK, t_end - t0);
        __syncthreads();
        if (tid < TOK)
            rows[tid] = tid < valid ? pool_row(a.block_table, a.max_pages_per_seq, a.page_tokens, seq, t0 + tid) : 0;
        __syncthreads();

        // ---- K: scores for every query head ----
        const WhichPlan &wk = lp.w[0];
        for (int s = 0; s < wk.n_src; ++s) {
            const SourcePlan &sp = wk.src[s];
            if (sp.compressed) hidden_tile<T>(sp, sm, rows, valid);
            for (int i = 0; i < sp.n_need; ++i) {
                restore_head<T>(sp, sm, sp.slot[i], hd, rows, valid);
                __syncthreads();
                const int g = sp.kv_head[i];
                for (int o = tid; o < group * TOK; o += NT) {
                    int t = o % TOK, qh = g * group + o / TOK;
                    float sc = -INFINITY;
                    if (t < valid) {
                        float dot = 0.f;
                        const float *qq = sm.q + qh * hd, *kk = sm.kh + t * (hd + 1);
                        for (int c = 0; c < hd; ++c) dot = fmaf(qq[c], kk[c], dot);
                        sc = dot * a.scale;
                    }
                    sm.S[qh * TOK + t] = sc;
                }
                __syncthreads();
            }
        }
        // ---- online softmax update, one warp per query head ----
        for (int qh = tid / 32; qh < hq; qh += NT / 32) {
            const int lane = tid % 32;
            float sc = sm.S[qh * TOK + lane];
            float mx = sc;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            float m_old = sm.mx[qh];
            float m_new = fmaxf(m_old, mx);
            float pr = (lane < valid) ? expf(sc - m_new) : 0.f;
            float ps = pr;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
            sm.S[qh * TOK + lane] = pr;
            if (lane == 0) {
                float corr = (m_old == -INFINITY) ? 0.f : expf(m_old - m_new);
                sm.corr[qh] = corr;
                sm.mx[qh] = m_new;
                sm.sum[qh] = sm.sum[qh] * corr + ps;
            }
        }
        __syncthreads();
        for (int i = tid; i < hq * hd; i += NT) sm.acc[i] *= sm.corr[i / hd];
        __syncthreads();

        // ---- V: weighted sum ----
        const WhichPlan &wv = lp.w[1];
        for (int s = 0; s < wv.n_src; ++s) {
            const SourcePlan &sp = wv.src[s];
            if (sp.compressed) hidden_tile<T>(sp, sm, rows, valid);
            for (int i = 0; i < sp.n_need; ++i) {
                restore_head<T>(sp, sm, sp.slot[i], hd, rows, valid);
                __syncthreads();
                const int g = sp.kv_head[i];
                for (int o = tid; o < group * hd; o += NT) {
                    int c = o % hd, qh = g * group + o / hd;
                    float acc = 0.f;
                    const float *pp = sm.S + qh * TOK;
                    for (int t = 0; t < valid; ++t) acc = fmaf(pp[t], sm.kh[t * (hd + 1) + c], acc);
                    sm.acc[qh * hd + c] += acc;
                }
                __syncthreads();
            }
        }
    }
    __syncthreads();
    float *part = a.partials + ((int64_t)si * a.max_chunks + chunk) * hq * (hd + 2);
    for (int i = tid; i < hq * hd; i += NT) part[(i / hd) * (hd + 2) + 2 + i % hd] = sm.acc[i];
    for (int i = tid; i < hq; i += NT) {
        part[i * (hd + 2) + 0] = sm.mx[i];
        part[i * (hd + 2) + 1] = sm.sum[i];
    }
}

// ---------------------------------------------------------------------------
// Combine the tile partials of one (sequence, query head) and, if asked, the
// exact current token.  grid = (hq, n_seqs); block = 256.  A long sequence has
// hundreds of tiles, so nothing walks them one after the other: three passes of
// independent loads (largest maximum; sum of the sums scaled to it; weighted
// values, one warp per tile in turns, lanes over the channels), each closed by a
// block reduction.
constexpr int CB_WARPS = 8;

__device__ __forceinline__ float block_reduce(float v, bool is_max, float *red) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float u = __shfl_xor_sync(0xffffffffu, v, o);
        v = is_max ? fmaxf(v, u) : v + u;
    }
    __syncthreads();  // red may still be read from the previous reduction
    if (lane == 0) red[warp] = v;
    __syncthreads();
    v = red[0];
#pragma unroll
    for (int w = 1; w < CB_WARPS; ++w) v = is_max ? fmaxf(v, red[w]) : v + red[w];
    return v;
}

template <typename T>
__global__ void __launch_bounds__(32 * CB_WARPS) combine_kernel(const __grid_constant__ DecodeArgs a,
                                                                const __grid_constant__ SeqList seqs) {
    const int qh = blockIdx.x, si = blockIdx.y, c = threadIdx.x, lane = c & 31, warp = c >> 5;
    const int seq = seqs.id[si];
    const int L = a.seq_len[seq];
    const int hd = a.hd, hq = a.hq;  // hd <= 128
    const int n_chunks = (L + a.chunk_tokens - 1) / a.chunk_tokens;
    const bool on = c < hd;
    const int64_t stride = (int64_t)hq * (hd + 2);  // floats from one tile's partial to the next
    const float *base = a.partials + ((int64_t)si * a.max_chunks * hq + qh) * (hd + 2);
    __shared__ float red[CB_WARPS];
    __shared__ float accs[CB_WARPS][128];

    // One pass: warp w folds tiles w, w + CB_WARPS, ... into a running (maximum, sum, weighted values), the loads of eight
    // tiles in flight at a time (they do not depend on one another; only the fold does), then the
    // warps' results are folded in shared memory.
    constexpr int U = 8;
    float Mw = -INFINITY, Sw = 0.f;
    float av[4] = {0.f, 0.f, 0.f, 0.f};  // channels lane, lane + 32, lane + 64, lane + 96
    for (int ch0 = warp; ch0 < n_chunks; ch0 += U * CB_WARPS) {
        float m[U], s_[U], v[U][4];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int ch = ch0 + u * CB_WARPS;
            const float *part = base + (int64_t)ch * stride;
            const bool in = ch < n_chunks;
            m[u] = in ? part[0] : -INFINITY;
            s_[u] = in ? part[1] : 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) v[u][j] = (in && lane + 32 * j < hd) ? part[2 + lane + 32 * j] : 0.f;
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (m[u] == -INFINITY) continue;  // an empty tile (or none)
            const float Mn = fmaxf(Mw, m[u]);
            const float cw = (Mw == -INFINITY) ? 0.f : expf(Mw - Mn), cn = expf(m[u] - Mn);
            Sw = Sw * cw + s_[u] * cn;
#pragma unroll
            for (int j = 0; j < 4; ++j) av[j] = av[j] * cw + v[u][j] * cn;
            Mw = Mn;
        }
    }
    __shared__ float wM[CB_WARPS], wS[CB_WARPS];
    if (lane == 0) {
        wM[warp] = Mw;
        wS[warp] = Sw;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) accs[warp][lane + 32 * j] = av[j];
    __syncthreads();
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < CB_WARPS; ++w) M = fmaxf(M, wM[w]);
    float S = 0.f, acc = 0.f;
#pragma unroll
    for (int w = 0; w < CB_WARPS; ++w) {
        const float f = (wM[w] == -INFINITY) ? 0.f : expf(wM[w] - M);
        S += wS[w] * f;
        if (on) acc += accs[w][c] * f;
    }

    if (a.flags & KVCAR_INCLUDE_CURRENT_EXACT) {
        const int g = qh / (hq / a.hkv);
        const int W = a.hkv * hd;
        const T *kc = reinterpret_cast<const T *>(a.plan->cur[0][g]) + (int64_t)seq * W + a.plan->cur_head[0][g] * hd;
        const T *vc = reinterpret_cast<const T *>(a.plan->cur[1][g]) + (int64_t)seq * W + a.plan->cur_head[1][g] * hd;
        const T *qg = reinterpret_cast<const T *>(a.q) + ((int64_t)si * hq + qh) * hd;
        const float vcur = on ? ld(vc + c) : 0.f;
        const float sc = block_reduce(on ? ld(qg + c) * ld(kc + c) : 0.f, false, red) * a.scale;
        const float Mn = fmaxf(M, sc);
        const float c0 = (M == -INFINITY) ? 0.f : expf(M - Mn);
        const float c1 = expf(sc - Mn);
        S = S * c0 + c1;
        acc = acc * c0 + vcur * c1;
    }
    if (on) {
        T *o = reinterpret_cast<T *>(a.out) + ((int64_t)si * hq + qh) * hd;
        st(o + c, S > 0.f ? acc / S : 0.f);
    }
}

// The same merge with one warp per (sequence, query head), for sequences of at most 32 tiles: lane c owns tile c's
// (maximum, sum); the weighted values of all tiles are fetched in one batch of independent loads, and the current
// token's operands are requested before anything else, so the whole merge is about two memory round trips.
// grid = ceil(hq * n_seqs / CB_WARPS); block = 32 * CB_WARPS.
template <typename T>
__global__ void __launch_bounds__(32 * CB_WARPS) combine_warp_kernel(const __grid_constant__ DecodeArgs a,
                                                                     const __grid_constant__ SeqList seqs) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int hd = a.hd, hq = a.hq;  // hd <= 128
    const int item = blockIdx.x * CB_WARPS + warp;
    if (item >= hq * seqs.n) return;
    const int si = item / hq, qh = item % hq;
    const int seq = seqs.id[si];
    const bool with_cur = (a.flags & KVCAR_INCLUDE_CURRENT_EXACT) != 0;
    // current token: its operands do not depend on the partials
    float qv[4] = {0.f, 0.f, 0.f, 0.f}, kv[4] = {0.f, 0.f, 0.f, 0.f}, vv[4] = {0.f, 0.f, 0.f, 0.f};
    if (with_cur) {
        const int g = qh / (hq / a.hkv);
        const int W = a.hkv * hd;
        const T *kc = reinterpret_cast<const T *>(a.plan->cur[0][g]) + (int64_t)seq * W + a.plan->cur_head[0][g] * hd;
        const T *vc = reinterpret_cast<const T *>(a.plan->cur[1][g]) + (int64_t)seq * W + a.plan->cur_head[1][g] * hd;
        const T *qg = reinterpret_cast<const T *>(a.q) + ((int64_t)si * hq + qh) * hd;
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (lane + 32 * j < hd) {
                qv[j] = ld(qg + lane + 32 * j);
                kv[j] = ld(kc + lane + 32 * j);
                vv[j] = ld(vc + lane + 32 * j);
            }
    }
    const int L = a.seq_len[seq];
    const int n_chunks = (L + a.chunk_tokens - 1) / a.chunk_tokens;  // <= 32 (the launcher's choice)
    const int64_t stride = (int64_t)hq * (hd + 2);
    const float *base = a.partials + ((int64_t)si * a.max_chunks * hq + qh) * (hd + 2);
    // lane c: tile c
    float m_c = -INFINITY, s_c = 0.f;
    if (lane < n_chunks) {
        m_c = base[lane * stride];
        s_c = base[lane * stride + 1];
    }
    // all weighted values: tile c, channels lane + 32 j
    float pv[32][2];
    const bool wide = hd > 64;
#pragma unroll
    for (int c = 0; c < 32; ++c) {
        pv[c][0] = pv[c][1] = 0.f;
        if (c < n_chunks) {
            const float *part = base + c * stride + 2;
            if (lane < hd) pv[c][0] = part[lane];
            if (lane + 32 < hd) pv[c][1] = part[lane + 32];
        }
    }
    float M = m_c;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    const float w_c = (m_c == -INFINITY) ? 0.f : expf(m_c - M);
    float S = s_c * w_c;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) S += __shfl_xor_sync(0xffffffffu, S, o);
    float av[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int c = 0; c < 32; ++c) {
        const float w = __shfl_sync(0xffffffffu, w_c, c);
        av[0] = fmaf(w, pv[c][0], av[0]);
        av[1] = fmaf(w, pv[c][1], av[1]);
    }
    if (wide) {  // head_dim above 64: channels 64.. in a second, plain pass
        for (int c = 0; c < n_chunks; ++c) {
            const float w = __shfl_sync(0xffffffffu, w_c, c);
            const float *part = base + c * stride + 2;
            if (lane + 64 < hd) av[2] = fmaf(w, part[lane + 64], av[2]);
            if (lane + 96 < hd) av[3] = fmaf(w, part[lane + 96], av[3]);
        }
    }
    float c0 = 1.f, c1 = 0.f;
    if (with_cur) {
        float prod = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) prod = fmaf(qv[j], kv[j], prod);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) prod += __shfl_xor_sync(0xffffffffu, prod, o);
        const float sc = prod * a.scale;
        const float Mn = fmaxf(M, sc);
        c0 = (M == -INFINITY) ? 0.f : expf(M - Mn);
        c1 = expf(sc - Mn);
        S = S * c0 + c1;
    }
    T *o = reinterpret_cast<T *>(a.out) + ((int64_t)si * hq + qh) * hd;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int c = lane + 32 * j;
        if (c < hd) {
            const float acc = av[j] * c0 + vv[j] * c1;
            st(o + c, S > 0.f ? acc / S : 0.f);
        }
    }
}

}  // namespace

// ---------------------------------------------------------------------------
cudaError_t launch_table_updates(int32_t *block_table, int32_t *seq_len, const TableUpdates &u, cudaStream_t st) {
    table_update_kernel<<<1, 256, 0, st>>>(block_table, seq_len, u);
    return cudaGetLastError();
}

cudaError_t launch_encode_generic(const EncodeArgs &a, const SeqList &seqs, int dtype, int max_in, int max_m,
                                  cudaStream_t st) {
    const int n_rows = seqs.n * a.n_tokens;
    dim3 grid((n_rows + ER - 1) / ER, 2);
    size_t smem = (size_t)ER * (max_in + max_m) * sizeof(float);
    cudaError_t e;
    if (dtype == KVCAR_F32) {
        e = cudaFuncSetAttribute(encode_generic_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        encode_generic_kernel<float><<<grid, 256, smem, st>>>(a, seqs);
    } else {
        e = cudaFuncSetAttribute(encode_generic_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem);
        if (e != cudaSuccess) return e;
        encode_generic_kernel<__nv_bfloat16><<<grid, 256, smem, st>>>(a, seqs);
    }
    return cudaGetLastError();
}

size_t decode_generic_smem(int hq, int hd, int max_d, int max_m) {
    return gen_smem_floats(hq, hd, max_d, max_m) * sizeof(float);
}

cudaError_t launch_decode_generic(const DecodeArgs &a, const SeqList &seqs, int dtype, int max_d, int max_m,
                                  int grid_chunks, cudaStream_t st) {
    dim3 grid(grid_chunks, seqs.n);
    size_t smem = decode_generic_smem(a.hq, a.hd, max_d, max_m);
    cudaError_t e;
    if (dtype == KVCAR_F32) {
        e = cudaFuncSetAttribute(decode_generic_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        decode_generic_kernel<float><<<grid, NT, smem, st>>>(a, seqs, max_d, max_m);
    } else {
        e = cudaFuncSetAttribute(decode_generic_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem);
        if (e != cudaSuccess) return e;
        decode_generic_kernel<__nv_bfloat16><<<grid, NT, smem, st>>>(a, seqs, max_d, max_m);
    }
    return cudaGetLastError();
}

cudaError_t launch_combine(const DecodeArgs &a, const SeqList &seqs, int dtype, int n_chunks, cudaStream_t st) {
    // At most 32 tiles per sequence: one warp per (sequence, query head) row, everything in two round trips.
    // Longer sequences: a CTA per row, which walks a row's tiles in parallel.
    if (n_chunks <= 32) {
        const int grid = (a.hq * seqs.n + CB_WARPS - 1) / CB_WARPS;
        if (dtype == KVCAR_F32)
            combine_warp_kernel<float><<<grid, 32 * CB_WARPS, 0, st>>>(a, seqs);
        else
            combine_warp_kernel<__nv_bfloat16><<<grid, 32 * CB_WARPS, 0, st>>>(a, seqs);
        return cudaGetLastError();
    }
    dim3 grid(a.hq, seqs.n);
    if (dtype == KVCAR_F32)
        combine_kernel<float><<<grid, 32 * CB_WARPS, 0, st>>>(a, seqs);
    else
        combine_kernel<__nv_bfloat16><<<grid, 32 * CB_WARPS, 0, st>>>(a, seqs);
    return cudaGetLastError();
}

}  // namespace kvcar
