// Stand-alone measurements of the operations the tile kernel's producer and issuer threads are made of, on static
// operands: (1) how many tcgen05.mma (cta_group::2, M=256, K=16) one thread can have queued before the issue waits,
// and the time per product; (2) the sustained rate of those products on one cluster and on one cluster per SM pair;
// (3) shared-memory bytes per clock that 1, 2 or 4 threads of an SM get from tensor loads of L2-resident data;
// (4) what a completed mbarrier.try_wait, an expect-tx, a tensor load and a mapa cost their thread on an idle SM, and
// how long a 16-KB load takes to land; (5) the rate of tensor loads into shared memory while the pair's tensor pipe
// runs products out of the same shared memory, and the products' rate meanwhile; (6) the issuer's and a producer's loop
// while eight other warps of the CTA sleep, compute, use shared memory or read tensor memory.  Every wait is bounded;
// results go to stdout.
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -I ../csrc -o pair_ops pair_ops.cu -lcuda && ./pair_ops
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdio>
#include <algorithm>
#include <cstring>
#include <vector>

#include "kvcar_ptx.cuh"
using namespace kvcar::ptx;

constexpr int SLOT = 16384;
constexpr int NQ = 32;      // products issued back to back in test 1
constexpr int MAXD = 12;    // places per warp in test 3
constexpr int SPIN = 4000000;

__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity) {
    for (int i = 0; i < SPIN; ++i)
        if (mbar_try(bar, parity)) return true;
    return false;
}

struct PipeArgs {
    long long *out;
    int *err;
    int n, rounds;  // rounds == 0: test 1 (stamps), else test 2 (rounds of 8 products)
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(128, 1) pipe_kernel(PipeArgs P) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t tmem_slot;
    __shared__ __align__(8) uint64_t bar[2];
    const uint32_t rank = blockIdx.x & 1u;
    const int warp = threadIdx.x >> 5;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *g = smem_raw + (base - smem_u32(smem_raw));
    for (int i = threadIdx.x; i < 2 * SLOT / 4; i += blockDim.x) reinterpret_cast<uint32_t *>(g)[i] = 0x3c003c00u;
    fence_async_smem();
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar[0]), 1);
        mbar_init(smem_u32(&bar[1]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(256u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    if (rank == 0 && warp == 1 && elect_one()) {
        const uint32_t idesc = make_idesc(256, P.n);
        const uint64_t da = make_desc(base), db = make_desc(base + SLOT);
        long long *o = P.out + (blockIdx.x >> 1) * (NQ + 2);
        bool ok = true;
        if (P.rounds == 0) {
            long long t[NQ + 2];
            t[0] = clock64();
#pragma unroll
            for (int i = 0; i < NQ; ++i) {
                if (i == 0)
                    umma_pair<0>(tmem, da + 2u * (i & 3), db + 2u * (i & 3), idesc);
                else
                    umma_pair<1>(tmem, da + 2u * (i & 3), db + 2u * (i & 3), idesc);
                t[i + 1] = clock64();
            }
            umma_commit_pair(smem_u32(&bar[0]));
            ok = wait_bounded(smem_u32(&bar[0]), 0);
            t[NQ + 1] = clock64();
            for (int i = 0; i < NQ + 2; ++i) o[i] = t[i] - t[0];
        } else {
            const long long c0 = clock64();
            const uint64_t n0 = global_ns();
            uint32_t par[2] = {0, 0};
            for (int r = 0; r < P.rounds && ok; ++r) {
                const int b = r & 1;
                if (r >= 2) {  // the round before last on this barrier must be complete
                    ok = wait_bounded(smem_u32(&bar[b]), par[b]);
                    par[b] ^= 1u;
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) umma_pair<1>(tmem, da + 2u * (i & 3), db + 2u * (i & 3), idesc);
                umma_commit_pair(smem_u32(&bar[b]));
            }
            for (int b = 0; b < 2 && ok; ++b) {
                const int bb = (P.rounds + b) & 1;
                ok = wait_bounded(smem_u32(&bar[bb]), par[bb]);
                par[bb] ^= 1u;
            }
            o[0] = clock64() - c0;
            o[1] = (long long)(global_ns() - n0);
        }
        if (!ok) atomicExch(P.err, 1);
    } else if (P.rounds == 0) {
        if (!wait_bounded(smem_u32(&bar[0]), 0)) atomicExch(P.err, 2);
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(256u) : "memory");
    }
}

struct LoadArgs {
    long long *out;
    int *err;
    int depth, rounds, own_rows, rows, kslabs, warps;
};

// test 3: `warps` threads per CTA, each keeping `depth` 16-KB places (two 64x64 bf16 boxes) in flight
__global__ void __launch_bounds__(128, 1) load_kernel(const __grid_constant__ CUtensorMap map, LoadArgs P) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_all[4 * MAXD];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    if (threadIdx.x == 0) {
        for (int i = 0; i < 4 * MAXD; ++i) mbar_init(smem_u32(&bar_all[i]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const int wid = threadIdx.x >> 5;
    if (wid < P.warps && elect_one()) {
        uint64_t *bar = bar_all + wid * MAXD;
        const uint32_t wbase = base + wid * P.depth * SLOT;
        const long long c0 = clock64();
        bool ok = true;
        uint32_t par = 0;
        int s = 0;
        const int nblk = P.rows / 128;  // own_rows: every CTA and warp starts in its own row block, else all read the same
        int blk = P.own_rows ? (int)((blockIdx.x * 37u + wid * 11u) % nblk) : wid, ks = 0;
        for (int r = 0; r < P.rounds + P.depth && ok; ++r) {
            if (r >= P.depth) ok = wait_bounded(smem_u32(&bar[s]), par);
            if (r < P.rounds) {
                mbar_expect_tx(smem_u32(&bar[s]), SLOT);
                tma_load_2d(wbase + s * SLOT, &map, 64 * ks, 128 * blk, smem_u32(&bar[s]));
                tma_load_2d(wbase + s * SLOT + 8192, &map, 64 * ks, 128 * blk + 64, smem_u32(&bar[s]));
                if (++ks == P.kslabs) {
                    ks = 0;
                    if (++blk == nblk) blk = 0;
                }
            }
            if (++s == P.depth) {
                s = 0;
                if (r >= P.depth) par ^= 1u;
            }
        }
        if (!ok) atomicExch(P.err, 1);
        if (wid == 0) P.out[blockIdx.x] = clock64() - c0;
    }
    __syncthreads();
}

// test 4: instruction costs for the issuing thread on an idle SM
__global__ void __launch_bounds__(128, 1) ops_kernel(const __grid_constant__ CUtensorMap map, long long *out, int *err) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar[4];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    if (threadIdx.x == 0) {
        for (int i = 0; i < 4; ++i) mbar_init(smem_u32(&bar[i]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x < 32 && elect_one()) {
        uint32_t acc = 0;
        const long long t0 = clock64();
#pragma unroll 1
        for (int i = 0; i < 64; ++i) acc += mbar_try(smem_u32(&bar[1]) + (acc & 0u), 1);  // parity 1 of a fresh barrier: complete
        const long long t1 = clock64();
        bool ok = true;
        long long issue = 0, land = 0;
#pragma unroll 1
        for (int i = 0; i < 16 && ok; ++i) {
            const long long a0 = clock64();
            mbar_expect_tx(smem_u32(&bar[0]), SLOT);
            tma_load_2d(base, &map, 0, 128 * i, smem_u32(&bar[0]));
            tma_load_2d(base + 8192, &map, 0, 128 * i + 64, smem_u32(&bar[0]));
            const long long a1 = clock64();
            ok = wait_bounded(smem_u32(&bar[0]), i & 1);
            issue += a1 - a0;
            land += clock64() - a1;
        }
        const long long t2 = clock64();
        mbar_expect_tx(smem_u32(&bar[2]), 8 * 8192);
        mbar_expect_tx(smem_u32(&bar[3]), 8 * 8192);
#pragma unroll
        for (int i = 0; i < 16; ++i) tma_load_2d(base + 8192 * i, &map, 64 * (i & 7), 64 * i, smem_u32(&bar[2 + (i & 1)]));
        const long long t3 = clock64();
        ok = ok && wait_bounded(smem_u32(&bar[2]), 0) && wait_bounded(smem_u32(&bar[3]), 0);
        const long long t4 = clock64();
        uint32_t m = smem_u32(&bar[0]);
#pragma unroll 1
        for (int i = 0; i < 64; ++i) m = map_to_cta(m, 0) + (acc & 0u);
        const long long t5 = clock64();
        if (!ok) atomicExch(err, 1);
        out[0] = t1 - t0;
        out[1] = issue;
        out[2] = land;
        out[3] = t3 - t2;
        out[4] = t4 - t3;
        out[5] = t5 - t4;
        out[6] = acc + m;
    }
    __syncthreads();
}


// test 5: tensor loads into shared memory while the pair's tensor pipe runs products from other places of the same
// shared memory: warp 1 of the leader issues products (as in test 2) until the loading threads are done; warp 2 of each
// CTA keeps three 16-KB places in flight (as in test 3) for a fixed number of places.
struct MixArgs {
    long long *out;
    int *err;
    int n, with_products, places;
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(128, 1) mix_kernel(const __grid_constant__ CUtensorMap map, MixArgs P) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t tmem_slot;
    __shared__ __align__(8) uint64_t bar[2], lbar[3];
    __shared__ volatile int loads_done;
    const uint32_t rank = blockIdx.x & 1u;
    const int warp = threadIdx.x >> 5;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *g = smem_raw + (base - smem_u32(smem_raw));
    for (int i = threadIdx.x; i < 2 * SLOT / 4; i += blockDim.x) reinterpret_cast<uint32_t *>(g)[i] = 0x3c003c00u;
    fence_async_smem();
    if (threadIdx.x == 0) {
        loads_done = 0;
        mbar_init(smem_u32(&bar[0]), 1);
        mbar_init(smem_u32(&bar[1]), 1);
        for (int i = 0; i < 3; ++i) mbar_init(smem_u32(&lbar[i]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(256u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    if (rank == 0 && warp == 1 && P.with_products && elect_one()) {
        const uint32_t idesc = make_idesc(256, P.n);
        const uint64_t da = make_desc(base), db = make_desc(base + SLOT);
        bool ok = true;
        uint32_t par[2] = {0, 0};
        long long n = 0;
        const long long c0 = clock64();
        for (int r = 0; r < (1 << 20) && ok; ++r) {   // bounded: at most 2^20 rounds
            const int b = r & 1;
            if (r >= 2) {
                ok = wait_bounded(smem_u32(&bar[b]), par[b]);
                par[b] ^= 1u;
            }
            if (loads_done) {   // drain the other barrier's round and stop
                if (r >= 1) ok = ok && wait_bounded(smem_u32(&bar[b ^ 1]), par[b ^ 1]);
                break;
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) umma_pair<1>(tmem, da + 2u * (i & 3), db + 2u * (i & 3), idesc);
            umma_commit_pair(smem_u32(&bar[b]));
            n += 8;
        }
        if (!ok) atomicExch(P.err, 1);
        P.out[(blockIdx.x >> 1) * 4 + 2] = clock64() - c0;
        P.out[(blockIdx.x >> 1) * 4 + 3] = n;
    } else if (warp == 2 && elect_one()) {
        const uint32_t wbase = base + 2 * SLOT;
        bool ok = true;
        uint32_t par = 0;
        int s = 0, ks = 0, blk = (int)((blockIdx.x * 37u) % 64u);
        const long long c0 = clock64();
        for (int r = 0; r < P.places + 3 && ok; ++r) {
            if (r >= 3) ok = wait_bounded(smem_u32(&lbar[s]), par);
            if (r < P.places) {
                mbar_expect_tx(smem_u32(&lbar[s]), SLOT);
                tma_load_2d(wbase + s * SLOT, &map, 64 * ks, 128 * blk, smem_u32(&lbar[s]));
                tma_load_2d(wbase + s * SLOT + 8192, &map, 64 * ks, 128 * blk + 64, smem_u32(&lbar[s]));
                if (++ks == 9) {
                    ks = 0;
                    if (++blk == 64) blk = 0;
                }
            }
            if (++s == 3) {
                s = 0;
                if (r >= 3) par ^= 1u;
            }
        }
        if (!ok) atomicExch(P.err, 2);
        P.out[(blockIdx.x >> 1) * 4 + rank] = clock64() - c0;
        if (rank == 0) loads_done = 1;
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(256u) : "memory");
    }
}


// test 6: the issuer's and a producer's loop while eight other warps of each CTA do one kind of work.  Issuer: per
// round one try_wait, one fence, four short products (N = 64, so the pipe is never the limit) and a commit; producer:
// as in test 3, three places in flight.  Background (bounded, ends with the producer): 0 sleeping; 1 four dependent
// FMA chains per thread; 2 shared-memory load + store; 3 tcgen05.ld x32 + wait back to back; 4 tcgen05.ld x32 + wait,
// then 32 independent FMA chains, twice (an epilogue-like mix); 5 the same with 64 rounds of arithmetic per load.
struct BgArgs {
    long long *out;
    int *err;
    int mode, rounds, places;
    float *sink;
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(384, 1) bg_kernel(const __grid_constant__ CUtensorMap map, BgArgs P) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t tmem_slot;
    __shared__ __align__(8) uint64_t bar[2], lbar[3];
    __shared__ volatile int stop;
    __shared__ __align__(16) float scratch[8 * 32 * 8];
    const uint32_t rank = blockIdx.x & 1u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *g = smem_raw + (base - smem_u32(smem_raw));
    for (int i = threadIdx.x; i < 2 * SLOT / 4; i += blockDim.x) reinterpret_cast<uint32_t *>(g)[i] = 0x3c003c00u;
    fence_async_smem();
    if (threadIdx.x == 0) {
        stop = 0;
        mbar_init(smem_u32(&bar[0]), 1);
        mbar_init(smem_u32(&bar[1]), 1);
        for (int i = 0; i < 3; ++i) mbar_init(smem_u32(&lbar[i]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(256u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    if (warp == 1) {
        if (rank == 0 && elect_one()) {
            const uint32_t idesc = make_idesc(256, 64);
            bool ok = true;
            uint32_t par[2] = {0, 0};
            const long long c0 = clock64();
            for (int r = 0; r < P.rounds && ok; ++r) {
                const int b = r & 1;
                if (r >= 2) {
                    ok = wait_bounded(smem_u32(&bar[b]), par[b]);
                    par[b] ^= 1u;
                }
                tc_fence_after();
                const uint64_t da = make_desc(base), db = make_desc(base + SLOT);
#pragma unroll
                for (int i = 0; i < 4; ++i) umma_pair<1>(tmem, da + 2u * i, db + 2u * i, idesc);
                umma_commit_pair(smem_u32(&bar[b]));
            }
            for (int b = 0; b < 2 && ok; ++b) {
                const int bb = (P.rounds + b) & 1;
                ok = wait_bounded(smem_u32(&bar[bb]), par[bb]);
                par[bb] ^= 1u;
            }
            P.out[(blockIdx.x >> 1) * 4 + 2] = clock64() - c0;
            if (!ok) atomicExch(P.err, 1);
        }
    } else if (warp == 2) {
        if (elect_one()) {
            const uint32_t wbase = base + 2 * SLOT;
            bool ok = true;
            uint32_t par = 0;
            int s = 0, ks = 0, blk = (int)((blockIdx.x * 37u) % 64u);
            const long long c0 = clock64();
            for (int r = 0; r < P.places + 3 && ok; ++r) {
                if (r >= 3) ok = wait_bounded(smem_u32(&lbar[s]), par);
                if (r < P.places) {
                    mbar_expect_tx(smem_u32(&lbar[s]), SLOT);
                    tma_load_2d(wbase + s * SLOT, &map, 64 * ks, 128 * blk, smem_u32(&lbar[s]));
                    tma_load_2d(wbase + s * SLOT + 8192, &map, 64 * ks, 128 * blk + 64, smem_u32(&lbar[s]));
                    if (++ks == 9) {
                        ks = 0;
                        if (++blk == 64) blk = 0;
                    }
                }
                if (++s == 3) {
                    s = 0;
                    if (r >= 3) par ^= 1u;
                }
            }
            if (!ok) atomicExch(P.err, 2);
            P.out[(blockIdx.x >> 1) * 4 + rank] = clock64() - c0;
        }
        __syncwarp();
        if (lane == 0) stop = 1;  // the background warps of this CTA run until its producer is done
    } else if (warp >= 4) {
        float a0 = lane, a1 = lane + 1, a2 = lane + 2, a3 = lane + 3;
        float v[32];
        for (int it = 0; it < (1 << 22) && !stop; ++it) {
            if (P.mode == 1) {
#pragma unroll
                for (int u = 0; u < 16; ++u) {
                    a0 = fmaf(a0, 1.0001f, 0.5f);
                    a1 = fmaf(a1, 0.9999f, 0.25f);
                    a2 = fmaf(a2, 1.0002f, 0.125f);
                    a3 = fmaf(a3, 0.9998f, 0.75f);
                }
            } else if (P.mode == 2) {
                float4 *p4 = reinterpret_cast<float4 *>(scratch) + ((warp - 4) * 64 + lane);
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    float4 x = *p4;
                    x.x += 1.f;
                    *p4 = x;
                    p4 += 32 * ((u & 1) ? -1 : 1);
                }
            } else if (P.mode >= 3) {
                tmem_ld32(tmem + ((uint32_t)(32 * (warp & 3)) << 16) + 64u + 32u * (it & 3), v);
                tmem_ld_wait();
                const int reps = P.mode == 3 ? 0 : P.mode == 4 ? 2 : 64;
                for (int rr = 0; rr < reps; ++rr)
#pragma unroll
                    for (int u = 0; u < 32; ++u) v[u] = fmaf(v[u], 1.0001f, 0.5f);
#pragma unroll
                for (int u = 0; u < 32; ++u) a0 += v[u];
            } else {
                __nanosleep(200);
            }
        }
        if (a0 + a1 + a2 + a3 == 12345.f) P.sink[threadIdx.x] = a0;
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(256u) : "memory");
    }
}

static bool check(const char *what) {
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        printf("%s: CUDA error %s\n", what, cudaGetErrorString(e));
        return false;
    }
    return true;
}

int main() {
    int *err;
    long long *out;
    cudaMalloc(&err, 4);
    cudaMalloc(&out, 148 * (NQ + 2) * 8);
    int herr = 0;

    // ---- 1 and 2: the tensor pipe
    PipeArgs P{out, err, 256, 0};
    const int psmem = 2 * SLOT + 2048;
    cudaFuncSetAttribute(pipe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, psmem);
    for (int n : {256, 128, 64}) {
        P.n = n;
        P.rounds = 0;
        cudaMemset(err, 0, 4);
        for (int rep = 0; rep < 2; ++rep) pipe_kernel<<<2, 128, psmem>>>(P);
        if (!check("issue queue")) return 1;
        std::vector<long long> s(NQ + 2);
        cudaMemcpy(s.data(), out, s.size() * 8, cudaMemcpyDeviceToHost);
        cudaMemcpy(&herr, err, 4, cudaMemcpyDeviceToHost);
        printf("issue queue, N %3d (err %d): cycles between consecutive issues:", n, herr);
        for (int i = 1; i <= NQ; ++i) printf(" %lld", s[i] - s[i - 1]);
        printf(" | all %d complete %lld cycles after the first issue\n", NQ, s[NQ + 1]);
    }
    for (int clusters : {1, 74})
        for (int rounds : {512, 65536}) {
            P.n = 256;
            P.rounds = rounds;
            cudaMemset(err, 0, 4);
            pipe_kernel<<<2 * clusters, 128, psmem>>>(P);
            if (!check("sustained rate")) return 1;
            std::vector<long long> s((size_t)clusters * (NQ + 2));
            cudaMemcpy(s.data(), out, s.size() * 8, cudaMemcpyDeviceToHost);
            cudaMemcpy(&herr, err, 4, cudaMemcpyDeviceToHost);
            long long cmax = 0, nmax = 0;
            for (int c = 0; c < clusters; ++c) {
                cmax = s[(size_t)c * (NQ + 2)] > cmax ? s[(size_t)c * (NQ + 2)] : cmax;
                nmax = s[(size_t)c * (NQ + 2) + 1] > nmax ? s[(size_t)c * (NQ + 2) + 1] : nmax;
            }
            const double mm = 8.0 * rounds;
            printf("sustained, %2d clusters x %6.0f products of M256 N256 K16 (err %d): %.1f cycles per product, SM clock %.0f MHz, "
                   "%.0f TFLOP/s\n",
                   clusters, mm, herr, cmax / mm, 1e3 * cmax / (double)nmax, clusters * mm * 2.0 * 256 * 256 * 16 / (nmax * 1e-9) / 1e12);
        }

    // ---- 3 and 4: tensor loads
    const int rows = 8192, cols = 576;  // 9.4 MB: stays in L2
    __nv_bfloat16 *w;
    cudaMalloc(&w, (size_t)rows * cols * 2);
    cudaMemset(w, 0, (size_t)rows * cols * 2);
    kvcar::EncodeTiledFn fn = kvcar::tensor_map_encoder();
    CUtensorMap map;
    if (!fn || !kvcar::encode_bf16_map(fn, &map, w, rows, cols, cols)) {
        printf("tensor map encode failed\n");
        return 1;
    }
    LoadArgs L{out, err, 3, 4096, 0, rows, cols / 64, 1};
    const int lsmem = MAXD * SLOT + 2048;
    cudaFuncSetAttribute(load_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, lsmem);
    for (int own : {0, 1})
        for (int warps : {1, 2, 4}) {
            L.own_rows = own;
            L.warps = warps;
            cudaMemset(err, 0, 4);
            for (int rep = 0; rep < 2; ++rep) load_kernel<<<148, 128, lsmem>>>(map, L);
            if (!check("tensor loads")) return 1;
            std::vector<long long> s(148);
            cudaMemcpy(s.data(), out, s.size() * 8, cudaMemcpyDeviceToHost);
            cudaMemcpy(&herr, err, 4, cudaMemcpyDeviceToHost);
            long long mx = 0;
            for (auto v : s) mx = v > mx ? v : mx;
            printf("tensor loads, 148 CTAs, %d issuing thread(s) per SM, 3 places each, %s (err %d): %.0f cycles per 16-KB place "
                   "and thread, %.1f B/clk/SM\n",
                   warps, own ? "own rows per CTA" : "same rows in every CTA", herr, mx / 4096.0, warps * 16384.0 * 4096 / mx);
        }
    {   // ---- 5: loads while the pipe runs
        const int msmem = 5 * SLOT + 2048;
        cudaFuncSetAttribute(mix_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, msmem);
        MixArgs M{out, err, 256, 0, 2048};
        for (int clusters : {1, 74})
            for (int mode = 0; mode < 4; ++mode) {
                M.with_products = mode > 0;
                M.n = mode == 1 ? 256 : mode == 2 ? 128 : 64;
                cudaMemset(err, 0, 4);
                cudaMemset(out, 0, 148 * 4 * 8);
                mix_kernel<<<2 * clusters, 128, msmem>>>(map, M);
                if (!check("loads under products")) return 1;
                std::vector<long long> s((size_t)clusters * 4);
                cudaMemcpy(s.data(), out, s.size() * 8, cudaMemcpyDeviceToHost);
                cudaMemcpy(&herr, err, 4, cudaMemcpyDeviceToHost);
                long long lmax = 0;
                for (int c = 0; c < clusters; ++c) lmax = std::max(lmax, std::max(s[4 * c], s[4 * c + 1]));
                printf("loads under products, %2d clusters, %s (err %d): %.0f cycles per 16-KB place and CTA (%.1f B/clk/SM)", clusters,
                       mode == 0 ? "pipe idle" : mode == 1 ? "products N256" : mode == 2 ? "products N128" : "products N64", herr,
                       lmax / 2048.0, 16384.0 * 2048 / lmax);
                if (mode) printf(", %.1f cycles per product meanwhile", (double)s[2] / (double)std::max(1LL, s[3]));
                printf("\n");
            }
    }
    {   // ---- 6: the single-thread roles beside working warps
        const int bsmem = 5 * SLOT + 2048;
        cudaFuncSetAttribute(bg_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bsmem);
        float *sink;
        cudaMalloc(&sink, 4096);
        BgArgs G{out, err, 0, 8192, 4096, sink};
        const char *names[6] = {"sleeping", "4 dependent FMA chains", "shared-memory load + store", "tcgen05.ld x32 + wait",
                                "tcgen05.ld + 2 x 32 independent FMA", "tcgen05.ld + 64 x 32 independent FMA"};
        for (int mode = 0; mode < 6; ++mode) {
            G.mode = mode;
            cudaMemset(err, 0, 4);
            cudaMemset(out, 0, 74 * 4 * 8);
            bg_kernel<<<2 * 74, 384, bsmem>>>(map, G);
            if (!check("roles beside working warps")) return 1;
            long long o4[4];
            cudaMemcpy(o4, out, 32, cudaMemcpyDeviceToHost);
            cudaMemcpy(&herr, err, 4, cudaMemcpyDeviceToHost);
            printf("eight other warps %-38s (err %d): issuer %.0f cycles per round of 4 short products, producer %.0f cycles per place\n",
                   names[mode], herr, o4[2] / 8192.0, o4[0] / 4096.0);
        }
    }
    const int osmem = 16 * 8192 + 2048;
    cudaFuncSetAttribute(ops_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, osmem);
    cudaMemset(err, 0, 4);
    for (int rep = 0; rep < 2; ++rep) ops_kernel<<<1, 128, osmem>>>(map, out, err);
    if (!check("instruction costs")) return 1;
    long long o[8];
    cudaMemcpy(o, out, 56, cudaMemcpyDeviceToHost);
    cudaMemcpy(&herr, err, 4, cudaMemcpyDeviceToHost);
    printf("idle SM (err %d): try_wait on a complete phase %.0f cycles; expect-tx + two tensor loads %.0f cycles to issue, bytes seen "
           "%.0f cycles later; 16 tensor loads back to back %.0f cycles each to issue, all landed %lld cycles later; mapa %.0f cycles\n",
           herr, o[0] / 64.0, o[1] / 16.0, o[2] / 16.0, o[3] / 16.0, o[4], o[5] / 64.0);
    return 0;
}
