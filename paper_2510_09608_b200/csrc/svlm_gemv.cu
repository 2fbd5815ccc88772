// Projections of a few tokens at a time (decode): Y = X W^T for n <= 16 rows of X.  With so few rows the
// work is reading W once, so this is a bandwidth kernel, not a tensor-core one: a warp owns output rows
// (one row of W each, 16-byte loads, several in flight per lane), multiplies them with all n token vectors
// held in shared memory, accumulates in fp32 and reduces with shuffles (up to 4 tokens; more take the
// tensor-core form further down).  It serves svlm_out_proj for small n, on both sides of the decode step: [q | k | v] = W_qkv x before svlm_decode_step, W_o a after it.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "svlm_dev.h"
#include "svlm_launch.h"
#include "svlm_ptx.cuh"

namespace {

constexpr int GV_THREADS = 256;
// 16-byte chunks of a W row in flight per lane: the fewer token vectors share the registers, the more loads
template <int NX> __host__ __device__ constexpr int gv_unroll() { return NX == 1 ? 16 : (NX <= 4 ? 8 : 4); }

template <int NX>
__global__ void __launch_bounds__(GV_THREADS) gemv_kernel(const uint16_t* __restrict__ X, const uint16_t* __restrict__ W,
                                                         uint16_t* __restrict__ Y, int n, int in_dim, int out_dim) {
    constexpr int GV_UNROLL = gv_unroll<NX>();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint4* sx = reinterpret_cast<uint4*>(smem_raw);            // [NX][in_dim / 8] chunks of 8 bf16; rows >= n are zero
    const int chunks = in_dim / 8;
    const int lane = threadIdx.x & 31;
    const int warp = blockIdx.x * (GV_THREADS / 32) + (threadIdx.x >> 5), n_warps = gridDim.x * (GV_THREADS / 32);
    uint4 w[GV_UNROLL];
    auto load_w = [&](int row, int c0) {
        const uint4* wrow = reinterpret_cast<const uint4*>(W + (size_t)row * in_dim);
#pragma unroll
        for (int u = 0; u < GV_UNROLL; ++u) {
            const int c = c0 + 32 * u;
            w[u] = c < chunks ? __ldg(wrow + c) : make_uint4(0, 0, 0, 0);
        }
    };
    // The weights do not depend on anything earlier in the stream: the kernel is launched while its predecessor
    // may still run and fetches the first row of every warp at once; the token vectors wait for the predecessor.
    svlm_ptx::pdl_launch_dependents();
    if (warp < out_dim) load_w(warp, lane);
    svlm_ptx::pdl_wait();
    for (int i = threadIdx.x; i < NX * chunks; i += GV_THREADS) {
        const int t = i / chunks;
        sx[i] = t < n ? *reinterpret_cast<const uint4*>(X + (size_t)t * in_dim + (size_t)(i % chunks) * 8) : make_uint4(0, 0, 0, 0);
    }
    __syncthreads();
    for (int row = warp; row < out_dim; row += n_warps) {
        float acc[NX];
#pragma unroll
        for (int t = 0; t < NX; ++t) acc[t] = 0.f;
        for (int c0 = lane; c0 < chunks; c0 += 32 * GV_UNROLL) {
            if (row != warp || c0 != lane) load_w(row, c0);      // the first batch is already here
#pragma unroll
            for (int u = 0; u < GV_UNROLL; ++u) {
                const int c = c0 + 32 * u;
                if (c >= chunks) continue;
                const __nv_bfloat162* wp = reinterpret_cast<const __nv_bfloat162*>(&w[u]);
                float2 wf[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) wf[q] = __bfloat1622float2(wp[q]);
#pragma unroll
                for (int t = 0; t < NX; ++t) {
                    const uint4 xv = sx[t * chunks + c];
                    const __nv_bfloat162* xp = reinterpret_cast<const __nv_bfloat162*>(&xv);
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const float2 xf = __bfloat1622float2(xp[q]);
                        acc[t] = fmaf(wf[q].x, xf.x, acc[t]);
                        acc[t] = fmaf(wf[q].y, xf.y, acc[t]);
                    }
                }
            }
        }
#pragma unroll
        for (int t = 0; t < NX; ++t) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc[t] += __shfl_xor_sync(0xffffffffu, acc[t], o);
        }
        if (lane == 0) {
#pragma unroll
            for (int t = 0; t < NX; ++t)
                if (t < n) Y[(size_t)t * out_dim + row] = __bfloat16_as_ushort(__float2bfloat16_rn(acc[t]));
        }
    }
}

// 5 to 16 tokens: the tokens are the M = 16 rows of mma.sync.m16n8k16, eight rows of W the N.  A block owns
// eight output rows; its eight warps split K (k-blocks of 32, strided), every lane loading 16 bytes of one W
// row and of two token rows per k-block straight into the fragment registers (the dot product does not care
// in which order k is summed, so the eight consecutive elements a lane loads serve two MMAs), several k-blocks
// in flight; the warps' partial tiles meet in shared memory.
constexpr int GM_KB_IN_FLIGHT = 7;

__device__ __forceinline__ void mma_bf16_16816(float* c, unsigned a0, unsigned a1, unsigned a2, unsigned a3, unsigned b0, unsigned b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__global__ void __launch_bounds__(GV_THREADS) gemv_mma_kernel(const uint16_t* __restrict__ X, const uint16_t* __restrict__ W,
                                                             uint16_t* __restrict__ Y, int n, int in_dim, int out_dim) {
    __shared__ float part[GV_THREADS / 32][16][8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, kq = lane & 3;
    const int row0 = blockIdx.x * 8;
    const int wrow = min(row0 + g, out_dim - 1);
    const uint4* wp = reinterpret_cast<const uint4*>(W + (size_t)wrow * in_dim) + kq;          // + 4 per k-block of 32
    const uint4* xlo = reinterpret_cast<const uint4*>(X + (size_t)min(g, n - 1) * in_dim) + kq;
    const uint4* xhi = reinterpret_cast<const uint4*>(X + (size_t)min(g + 8, n - 1) * in_dim) + kq;
    const bool lo_live = g < n, hi_live = g + 8 < n;
    const int n_kb = in_dim / 32;
    float c[4] = {0.f, 0.f, 0.f, 0.f};
    uint4 w[GM_KB_IN_FLIGHT];
    auto load_w = [&](int kb0) {
#pragma unroll
        for (int u = 0; u < GM_KB_IN_FLIGHT; ++u) {
            const int kb = kb0 + u * (GV_THREADS / 32);
            w[u] = kb < n_kb ? __ldg(wp + 4 * kb) : make_uint4(0, 0, 0, 0);
        }
    };
    // as in the FMA form: the first batch of weights is fetched before the wait for the predecessor
    svlm_ptx::pdl_launch_dependents();
    load_w(warp);
    svlm_ptx::pdl_wait();
    for (int kb0 = warp; kb0 < n_kb; kb0 += (GV_THREADS / 32) * GM_KB_IN_FLIGHT) {
        uint4 a[GM_KB_IN_FLIGHT], bq[GM_KB_IN_FLIGHT];
        if (kb0 != warp) load_w(kb0);
#pragma unroll
        for (int u = 0; u < GM_KB_IN_FLIGHT; ++u) {
            const int kb = kb0 + u * (GV_THREADS / 32);
            const bool live = kb < n_kb;
            a[u] = live && lo_live ? __ldg(xlo + 4 * kb) : make_uint4(0, 0, 0, 0);
            bq[u] = live && hi_live ? __ldg(xhi + 4 * kb) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < GM_KB_IN_FLIGHT; ++u) {
            mma_bf16_16816(c, a[u].x, bq[u].x, a[u].y, bq[u].y, w[u].x, w[u].y);
            mma_bf16_16816(c, a[u].z, bq[u].z, a[u].w, bq[u].w, w[u].z, w[u].w);
        }
    }
    part[warp][g][2 * kq] = c[0];
    part[warp][g][2 * kq + 1] = c[1];
    part[warp][g + 8][2 * kq] = c[2];
    part[warp][g + 8][2 * kq + 1] = c[3];
    __syncthreads();
    if (threadIdx.x < 128) {
        const int t = threadIdx.x >> 3, r = threadIdx.x & 7;
        float s = 0.f;
#pragma unroll
        for (int w8 = 0; w8 < GV_THREADS / 32; ++w8) s += part[w8][t][r];
        if (t < n && row0 + r < out_dim) Y[(size_t)t * out_dim + row0 + r] = __bfloat16_as_ushort(__float2bfloat16_rn(s));
    }
}

template <int NX>
cudaError_t launch(const uint16_t* X, const uint16_t* W, uint16_t* Y, int n, int in_dim, int out_dim, cudaStream_t st) {
    const size_t smem = (size_t)NX * in_dim * 2;
    cudaError_t e = svlm_allow_smem<gemv_kernel<NX>>(smem);
    if (e != cudaSuccess) return e;
    const int rows_per_block = GV_THREADS / 32;
    int blocks = (out_dim + rows_per_block - 1) / rows_per_block;
    if (blocks > 2 * 148) blocks = 2 * 148;         // two resident blocks per SM, each warp walks a few rows
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(blocks);
    cfg.blockDim = dim3(GV_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // weights are fetched under the predecessor's tail
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, gemv_kernel<NX>, X, W, Y, n, in_dim, out_dim);
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

bool svlm_gemv_supported(int n, int in_dim) { return n >= 1 && n <= 16 && in_dim % 32 == 0 && (size_t)4 * in_dim * 2 <= 200 * 1024; }

cudaError_t svlm_launch_gemv(const void* X, const void* W, void* Y, int n, int in_dim, int out_dim, cudaStream_t st) {
    const uint16_t* x = static_cast<const uint16_t*>(X);
    const uint16_t* w = static_cast<const uint16_t*>(W);
    uint16_t* y = static_cast<uint16_t*>(Y);
    cudaError_t e;
    if (n == 1) e = launch<1>(x, w, y, n, in_dim, out_dim, st);
    else if (n <= 4) e = launch<4>(x, w, y, n, in_dim, out_dim, st);
    else {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((out_dim + 7) / 8);
        cfg.blockDim = dim3(GV_THREADS);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, gemv_mma_kernel, x, w, y, n, in_dim, out_dim);
        if (e == cudaSuccess) e = cudaGetLastError();
    }
    svlm_count_launch();
    return e;
}
