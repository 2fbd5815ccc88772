// Split-KV decode attention (n_q = 1): one query token per cache/layer attends over the whole
// retained cache (paper Section 3.3: per-token latency over a fixed-length context is the figure of
// merit).  The step streams every stored key and value exactly once, so it is bound by HBM
// bandwidth; the design is about keeping enough bytes in flight:
//   * grid = (splits, kv_heads, caches*layers); a CTA owns a contiguous run of active pages;
//   * each of its 4 warps owns the same 32-key quarter of every page and runs its own 3-stage
//     cp.async ring (16-byte copies into XOR-swizzled shared memory), so no CTA-wide barrier sits
//     in the streaming loop;
//   * the G <= 8 query heads that share a kv head ride in the N dimension of m16n8k16 tensor-core
//     MMAs (S^T = K Q^T, O^T += V^T P^T), so K and V are read once for the whole group;
//   * per-warp online softmax with warp-shuffle reductions; warps merge through shared memory;
//   * split partials (o, m, l) go to scratch; the last CTA of a (cache, layer, kv head) to arrive
//     combines them (arrival counter, no waiting).
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include "svlm_dev.h"
#include "svlm_launch.h"

namespace {

constexpr int DEC_WARPS = 4;
constexpr int DEC_THREADS = DEC_WARPS * 32;
constexpr int DEC_STAGES = 3;
constexpr int SUB = 32;            // keys per warp per page

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

__device__ __forceinline__ void ldmatrix_x4(unsigned& r0, unsigned& r1, unsigned& r2, unsigned& r3, const void* p) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(p);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(s));
}
__device__ __forceinline__ void ldmatrix_x4_trans(unsigned& r0, unsigned& r1, unsigned& r2, unsigned& r3,
                                                  const void* p) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(p);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(s));
}
__device__ __forceinline__ unsigned movmatrix_trans(unsigned a) {
    unsigned d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ void mma_bf16(float* c, unsigned a0, unsigned a1, unsigned a2, unsigned a3, unsigned b0,
                                         unsigned b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                 "{%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ unsigned pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<unsigned*>(&v);
}

// Scratch layout per cache: arrival counters [layers*kv_heads] (kept at zero between launches),
// then per (layer in launch, kv head): splits x { o[8][D], m[8], l[8] } floats.
template <int D>
__host__ __device__ constexpr int partial_floats() { return 8 * D + 16; }

template <int D>
__global__ void __launch_bounds__(DEC_THREADS, 1)
decode_kernel(SvlmAttendBatch b, int layer0, int n_layers, const uint16_t* __restrict__ Q,
              const int* __restrict__ q_pos, int q_heads, uint16_t* __restrict__ out, int splits) {
    constexpr int ROW_BYTES = D * 2;                 // one key row
    constexpr int CHUNKS = ROW_BYTES / 16;           // 16-byte chunks per row
    constexpr int STAGE_BYTES = 2 * SUB * ROW_BYTES; // K then V sub-tile
    constexpr int KSTEPS = D / 16;
    constexpr int DBLK = D / 16;
    extern __shared__ __align__(128) unsigned char smem[];
    // [warp][stage][K | V]  then  q rows [8][D] bf16
    unsigned char* my = smem + (size_t)(threadIdx.x >> 5) * DEC_STAGES * STAGE_BYTES;
    uint16_t* s_q = reinterpret_cast<uint16_t*>(smem + (size_t)DEC_WARPS * DEC_STAGES * STAGE_BYTES);
    __shared__ int s_last;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int split = blockIdx.x, hk = blockIdx.y;
    const int prob = blockIdx.z;
    const int ci = prob / n_layers, li = prob % n_layers;
    const int layer = layer0 + li;
    const SvlmAttendView& vw = b.view[ci];
    const int G = q_heads / b.kv_heads;

    const int n_tiles = vw.ctrl->n_tiles;
    const long long shift = vw.ctrl->shift_total;
    const int tps = (n_tiles + splits - 1) / splits;
    const int t0 = min(n_tiles, split * tps), t1 = min(n_tiles, t0 + tps);

    const uint16_t* Kb = vw.K + ((size_t)layer * b.kv_heads + hk) * b.n_slots * D;
    const uint16_t* Vb = vw.V + ((size_t)layer * b.kv_heads + hk) * b.n_slots * D;

    // ---- sub-tile loader (this warp's 32 keys of tile ti into its stage) ----------------------
    auto issue = [&](int it) {   // it = index into this warp's sequence of sub-tiles
        const int ti = t0 + it;
        if (ti < t1) {
            const SvlmTile tl = vw.tiles[ti];
            const int k0 = warp * SUB;
            if (k0 < tl.hi && k0 + SUB > tl.lo) {
                unsigned char* st = my + (it % DEC_STAGES) * STAGE_BYTES;
                const size_t row0 = (size_t)tl.page * SVLM_PAGE + k0;
                const unsigned char* gk = reinterpret_cast<const unsigned char*>(Kb + row0 * D);
                const unsigned char* gv = reinterpret_cast<const unsigned char*>(Vb + row0 * D);
#pragma unroll
                for (int j = 0; j < SUB * CHUNKS / 32; ++j) {
                    const int idx = j * 32 + lane;
                    const int r = idx / CHUNKS, c = idx % CHUNKS;
                    const int dst = r * ROW_BYTES + ((c ^ (r & 7)) << 4);
                    cp_async16(st + dst, gk + (size_t)idx * 16);
                    cp_async16(st + SUB * ROW_BYTES + dst, gv + (size_t)idx * 16);
                }
            }
        }
        cp_async_commit();
    };
    for (int s = 0; s < DEC_STAGES - 1; ++s) issue(s);

    // ---- query rows: rotate at q_pos - shift_total, round to bf16, park in shared memory -------
    {
        const int half = D / 2;
        for (int i = threadIdx.x; i < 8 * half; i += DEC_THREADS) {
            const int h = i / half, pair = i % half;
            float lo = 0.f, hi = 0.f;
            if (h < G) {
                const size_t off = (((size_t)prob) * q_heads + hk * G + h) * D;   // n_q = 1
                const float x = __bfloat162float(__ushort_as_bfloat16(Q[off + pair]));
                const float y = __bfloat162float(__ushort_as_bfloat16(Q[off + pair + half]));
                const int axis = b.rope_mode == 0 ? 0 : (pair < b.sec_t ? 0 : (pair < b.sec_th ? 1 : 2));
                const int* qp = q_pos + (size_t)ci * (b.rope_mode == 0 ? 1 : 3);
                const long long c = (long long)qp[b.rope_mode == 0 ? 0 : axis] - shift;
                double sn, cs;
                sincos((double)c * b.theta[pair], &sn, &cs);
                lo = x * (float)cs - y * (float)sn;
                hi = y * (float)cs + x * (float)sn;
            }
            s_q[h * D + pair] = __bfloat16_as_ushort(__float2bfloat16_rn(lo));
            s_q[h * D + pair + half] = __bfloat16_as_ushort(__float2bfloat16_rn(hi));
        }
    }
    __syncthreads();
    unsigned qf[KSTEPS][2];   // B fragments of Q^T: (d = ks*16 + 2t.., head g)
#pragma unroll
    for (int ks = 0; ks < KSTEPS; ++ks) {
        qf[ks][0] = *reinterpret_cast<const unsigned*>(s_q + g * D + ks * 16 + 2 * t);
        qf[ks][1] = *reinterpret_cast<const unsigned*>(s_q + g * D + ks * 16 + 2 * t + 8);
    }

    const float scale = 1.4426950408889634f * rsqrtf((float)D);
    float o[DBLK][4];
#pragma unroll
    for (int i = 0; i < DBLK; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};   // heads 2t, 2t+1 (l: this thread's share)

    // ---- streaming loop ----------------------------------------------------------------------
    const int n_it = t1 - t0;
    for (int it = 0; it < n_it; ++it) {
        __syncwarp();   // every lane has finished reading the stage that is refilled next
        issue(it + DEC_STAGES - 1);
        cp_async_wait<DEC_STAGES - 1>();
        __syncwarp();
        const SvlmTile tl = vw.tiles[t0 + it];
        const int k0 = warp * SUB;
        if (!(k0 < tl.hi && k0 + SUB > tl.lo)) continue;
        const unsigned char* sk = my + (it % DEC_STAGES) * STAGE_BYTES;
        const unsigned char* sv = sk + SUB * ROW_BYTES;

        // S^T[32 keys x 8 heads] = K Q^T
        float s[2][4];
#pragma unroll
        for (int mb = 0; mb < 2; ++mb) {
            s[mb][0] = s[mb][1] = s[mb][2] = s[mb][3] = 0.f;
#pragma unroll
            for (int ks = 0; ks < KSTEPS; ++ks) {
                const int i = lane >> 3, r = lane & 7;
                const int key = mb * 16 + (i & 1) * 8 + r;
                const int chunk = ks * 2 + (i >> 1);
                unsigned a0, a1, a2, a3;
                ldmatrix_x4(a0, a1, a2, a3, sk + key * ROW_BYTES + ((chunk ^ (key & 7)) << 4));
                mma_bf16(s[mb], a0, a1, a2, a3, qf[ks][0], qf[ks][1]);
            }
        }
        // scale, mask slots outside [lo, hi), column (head) maxima over the 32 keys
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int mb = 0; mb < 2; ++mb)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int key = k0 + mb * 16 + g + (e >> 1) * 8;
                const bool ok = key >= tl.lo && key < tl.hi;
                s[mb][e] = ok ? s[mb][e] * scale : -INFINITY;
                mx[e & 1] = fmaxf(mx[e & 1], s[mb][e]);
            }
#pragma unroll
        for (int sh = 4; sh < 32; sh <<= 1) {
            mx[0] = fmaxf(mx[0], __shfl_xor_sync(0xffffffffu, mx[0], sh));
            mx[1] = fmaxf(mx[1], __shfl_xor_sync(0xffffffffu, mx[1], sh));
        }
        float corr[2], mu[2];
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            const float mn = fmaxf(m[c], mx[c]);
            mu[c] = mn == -INFINITY ? 0.f : mn;
            corr[c] = exp2f(m[c] - mu[c]);      // m = -inf gives 0
            m[c] = mn;
            l[c] *= corr[c];
        }
        unsigned pb[2][2];   // P^T as B fragments: [key block of 16][k halves]
#pragma unroll
        for (int mb = 0; mb < 2; ++mb) {
            float p[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                p[e] = exp2f(s[mb][e] - mu[e & 1]);
                l[e & 1] += p[e];
            }
            pb[mb][0] = movmatrix_trans(pack_bf16(p[0], p[1]));
            pb[mb][1] = movmatrix_trans(pack_bf16(p[2], p[3]));
        }
        // O^T[D x 8 heads] = O^T * corr + V^T P^T
#pragma unroll
        for (int db = 0; db < DBLK; ++db) {
            o[db][0] *= corr[0]; o[db][2] *= corr[0];
            o[db][1] *= corr[1]; o[db][3] *= corr[1];
#pragma unroll
            for (int kb = 0; kb < 2; ++kb) {
                const int i = lane >> 3, r = lane & 7;
                const int key = kb * 16 + (i >> 1) * 8 + r;
                const int chunk = db * 2 + (i & 1);
                unsigned a0, a1, a2, a3;
                ldmatrix_x4_trans(a0, a1, a2, a3, sv + key * ROW_BYTES + ((chunk ^ (key & 7)) << 4));
                mma_bf16(o[db], a0, a1, a2, a3, pb[kb][0], pb[kb][1]);
            }
        }
    }
    cp_async_wait<0>();
    // l: sum the shares of the 8 lane groups that hold the same heads
#pragma unroll
    for (int sh = 4; sh < 32; sh <<= 1) {
        l[0] += __shfl_xor_sync(0xffffffffu, l[0], sh);
        l[1] += __shfl_xor_sync(0xffffffffu, l[1], sh);
    }
    __syncthreads();   // everyone is done with the staging memory: reuse it for the warp merge

    // ---- merge the 4 warps: s_o[warp][8 heads][D], s_m/s_l[warp][8] -----------------------------
    float* s_o = reinterpret_cast<float*>(smem);
    float* s_m = s_o + DEC_WARPS * 8 * D;
    float* s_l = s_m + DEC_WARPS * 8;
#pragma unroll
    for (int db = 0; db < DBLK; ++db) {
        float* base = s_o + (size_t)warp * 8 * D;
        base[(2 * t) * D + db * 16 + g] = o[db][0];
        base[(2 * t + 1) * D + db * 16 + g] = o[db][1];
        base[(2 * t) * D + db * 16 + g + 8] = o[db][2];
        base[(2 * t + 1) * D + db * 16 + g + 8] = o[db][3];
    }
    if (g == 0) {
        s_m[warp * 8 + 2 * t] = m[0]; s_m[warp * 8 + 2 * t + 1] = m[1];
        s_l[warp * 8 + 2 * t] = l[0]; s_l[warp * 8 + 2 * t + 1] = l[1];
    }
    __syncthreads();
    float* ws_parts = vw.ws + (size_t)b.layers * b.kv_heads;   // after the counters
    float* part = ws_parts + ((size_t)(li * b.kv_heads + hk) * splits + split) * partial_floats<D>();
    for (int i = threadIdx.x; i < 8 * D; i += DEC_THREADS) {
        const int h = i / D;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < DEC_WARPS; ++w) M = fmaxf(M, s_m[w * 8 + h]);
        float acc = 0.f;
        if (M > -INFINITY)
#pragma unroll
            for (int w = 0; w < DEC_WARPS; ++w) acc += s_o[(size_t)w * 8 * D + i] * exp2f(s_m[w * 8 + h] - M);
        part[i] = acc;
    }
    if (threadIdx.x < 8) {
        const int h = threadIdx.x;
        float M = -INFINITY, L = 0.f;
#pragma unroll
        for (int w = 0; w < DEC_WARPS; ++w) M = fmaxf(M, s_m[w * 8 + h]);
        if (M > -INFINITY)
#pragma unroll
            for (int w = 0; w < DEC_WARPS; ++w) L += s_l[w * 8 + h] * exp2f(s_m[w * 8 + h] - M);
        part[8 * D + h] = M;
        part[8 * D + 8 + h] = L;
    }

    // ---- last CTA of this (cache, layer, kv head) combines the splits -----------------------------
    __threadfence();
    __syncthreads();
    unsigned* counter = reinterpret_cast<unsigned*>(vw.ws) + li * b.kv_heads + hk;
    if (threadIdx.x == 0) {
        const unsigned prev = atomicAdd(counter, 1u);
        s_last = (prev == (unsigned)splits - 1);
        if (s_last) *counter = 0;   // ready for the next launch
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // Phase 1: per-split (m, l) into shared memory, then per-head global max, weights and 1/L.
    const float* parts = ws_parts + (size_t)(li * b.kv_heads + hk) * splits * partial_floats<D>();
    float* c_m = reinterpret_cast<float*>(smem);          // [splits][8] -> weights exp2(m - M)
    float* c_l = c_m + splits * 8;                        // [splits][8]
    float* c_inv = c_l + splits * 8;                      // [8]
    for (int i = threadIdx.x; i < splits * 16; i += DEC_THREADS) {
        const int sp = i >> 4, j = i & 15;
        const float v = __ldcg(parts + (size_t)sp * partial_floats<D>() + 8 * D + j);
        (j < 8 ? c_m : c_l)[sp * 8 + (j & 7)] = v;
    }
    __syncthreads();
    if (threadIdx.x < 8) {
        const int h = threadIdx.x;
        float M = -INFINITY, L = 0.f;
        for (int sp = 0; sp < splits; ++sp) M = fmaxf(M, c_m[sp * 8 + h]);
        for (int sp = 0; sp < splits; ++sp) {
            const float f = M > -INFINITY ? exp2f(c_m[sp * 8 + h] - M) : 0.f;
            c_m[sp * 8 + h] = f;
            L += c_l[sp * 8 + h] * f;
        }
        c_inv[h] = L > 0.f ? 1.f / L : 0.f;
    }
    __syncthreads();
    // Phase 2: weighted sum of the split outputs; all loads of a thread are independent.
    constexpr int PER = 8 * D / DEC_THREADS;
    float acc[PER];
#pragma unroll
    for (int e = 0; e < PER; ++e) acc[e] = 0.f;
    for (int sp = 0; sp < splits; ++sp) {
        const float* p = parts + (size_t)sp * partial_floats<D>();
#pragma unroll
        for (int e = 0; e < PER; ++e) {
            const int i = e * DEC_THREADS + threadIdx.x;
            acc[e] += __ldcg(p + i) * c_m[sp * 8 + i / D];
        }
    }
#pragma unroll
    for (int e = 0; e < PER; ++e) {
        const int i = e * DEC_THREADS + threadIdx.x;
        const int h = i / D;
        if (h < G)
            out[((size_t)prob * q_heads + hk * G + h) * D + (i % D)] =
                __bfloat16_as_ushort(__float2bfloat16_rn(acc[e] * c_inv[h]));
    }
}

template <int D>
constexpr size_t decode_smem() { return (size_t)DEC_WARPS * DEC_STAGES * 2 * SUB * D * 2 + 8 * D * 2; }

}  // namespace

// Scratch floats needed per cache for `splits` splits (all layers at once is the largest launch).
size_t svlm_decode_ws_floats(int layers, int kv_heads, int head_dim, int splits) {
    const size_t pf = head_dim == 128 ? partial_floats<128>() : partial_floats<64>();
    return (size_t)layers * kv_heads + (size_t)layers * kv_heads * splits * pf;
}

int svlm_decode_splits(int n_pages, int kv_heads, int problems) {
    // about two CTAs' worth of work items per SM, but at most 16 splits: the combine reads every
    // split's partial once, and beyond 16 that read costs more than the extra parallelism saves
    int splits = (2 * 148 + kv_heads * problems - 1) / (kv_heads * problems);
    splits = splits < 1 ? 1 : (splits > 16 ? 16 : splits);
    return splits > n_pages ? n_pages : splits;
}

cudaError_t svlm_launch_decode(const SvlmAttendBatch& b, int layer0, int n_layers, const void* Q, const int* q_pos,
                               int q_heads, void* out, int splits, cudaStream_t st) {
    dim3 grid(splits, b.kv_heads, b.n_caches * n_layers);
    cudaError_t e;
    if (b.head_dim == 128) {
        static bool once = false;
        if (!once) {
            e = cudaFuncSetAttribute(decode_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)decode_smem<128>());
            if (e != cudaSuccess) return e;
            once = true;
        }
        decode_kernel<128><<<grid, DEC_THREADS, decode_smem<128>(), st>>>(b, layer0, n_layers, (const uint16_t*)Q, q_pos,
                                                                       q_heads, (uint16_t*)out, splits);
    } else {
        static bool once = false;
        if (!once) {
            e = cudaFuncSetAttribute(decode_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)decode_smem<64>());
            if (e != cudaSuccess) return e;
            once = true;
        }
        decode_kernel<64><<<grid, DEC_THREADS, decode_smem<64>(), st>>>(b, layer0, n_layers, (const uint16_t*)Q, q_pos,
                                                                     q_heads, (uint16_t*)out, splits);
    }
    svlm_count_launch();
    return cudaGetLastError();
}
