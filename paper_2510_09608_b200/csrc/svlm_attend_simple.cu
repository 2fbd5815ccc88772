// Row-at-a-time attention on the CUDA cores: one CTA per (query row, query head, cache/layer).
// It is the general path for any n_q and both head sizes; the tensor-core chunk-prefill kernel and
// the split-KV decode kernel take over the shapes they are built for.
// out[r,h] = sum_j softmax_j(<R(c_q) q, K'_j> / sqrt(d)) V_j over stored j with gid_j <= gid_q(r).
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include "svlm_dev.h"
#include "svlm_launch.h"

namespace {

template <int D>
__global__ void __launch_bounds__(128) attend_simple_kernel(SvlmAttendBatch b, int layer0, int n_layers,
                                                            const uint16_t* __restrict__ Q,
                                                            const int* __restrict__ q_pos, int n_q, int q_heads,
                                                            uint16_t* __restrict__ out) {
    constexpr int E = D / 32;   // elements per lane
    const int r = blockIdx.x, hq = blockIdx.y;
    const int ci = blockIdx.z / n_layers, li = blockIdx.z % n_layers;
    const int layer = layer0 + li;
    const SvlmAttendView& vw = b.view[ci];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = hq / (q_heads / b.kv_heads);

    const long long gid_q = vw.ctrl->n_total - n_q + r;
    const long long shift = vw.ctrl->shift_total;
    const int n_tiles = vw.ctrl->n_tiles;

    // query row, rotated at q_pos - shift_total, pre-scaled by log2(e)/sqrt(d)
    const size_t qoff = ((((size_t)ci * n_layers + li) * n_q + r) * q_heads + hq) * D + lane * E;
    float q[E];
    {
        float x[E];
#pragma unroll
        for (int e = 0; e < E; ++e) x[e] = __bfloat162float(__ushort_as_bfloat16(Q[qoff + e]));
        const float scale = 1.4426950408889634f * rsqrtf((float)D);
#pragma unroll
        for (int e = 0; e < E; ++e) {
            const int pair = (lane & 15) * E + e;
            const int axis = b.rope_mode == 0 ? 0 : (pair < b.sec_t ? 0 : (pair < b.sec_th ? 1 : 2));
            const int* qp = q_pos + ((size_t)ci * n_q + r) * (b.rope_mode == 0 ? 1 : 3);
            const long long c = (long long)qp[b.rope_mode == 0 ? 0 : axis] - shift;
            double sn, cs;
            sincos((double)c * b.theta[pair], &sn, &cs);
            const float other = __shfl_xor_sync(0xffffffffu, x[e], 16);
            const float rot = lane < 16 ? x[e] * (float)cs - other * (float)sn : x[e] * (float)cs + other * (float)sn;
            q[e] = rot * scale;
        }
    }

    const uint16_t* Kb = vw.K + ((size_t)layer * b.kv_heads + g) * b.n_slots * D + lane * E;
    const uint16_t* Vb = vw.V + ((size_t)layer * b.kv_heads + g) * b.n_slots * D + lane * E;
    float m = -INFINITY, l = 0.f, o[E];
#pragma unroll
    for (int e = 0; e < E; ++e) o[e] = 0.f;

    for (int ti = warp; ti < n_tiles; ti += 4) {
        const SvlmTile tl = vw.tiles[ti];
        if (tl.min_gid > gid_q) continue;
        const bool masked = tl.max_gid > gid_q;
        for (int off = tl.lo; off < tl.hi; ++off) {
            const int slot = tl.page * SVLM_PAGE + off;
            if (masked && vw.slot_gid[slot] > gid_q) break;   // ordinals grow with the offset
            float k[E], v[E];
            if (E == 4) {
                const uint2 kk = *reinterpret_cast<const uint2*>(Kb + (size_t)slot * D);
                const uint2 vv = *reinterpret_cast<const uint2*>(Vb + (size_t)slot * D);
                k[0] = __uint_as_float(kk.x << 16); k[1] = __uint_as_float(kk.x & 0xffff0000u);
                k[2 % E] = __uint_as_float(kk.y << 16); k[3 % E] = __uint_as_float(kk.y & 0xffff0000u);
                v[0] = __uint_as_float(vv.x << 16); v[1] = __uint_as_float(vv.x & 0xffff0000u);
                v[2 % E] = __uint_as_float(vv.y << 16); v[3 % E] = __uint_as_float(vv.y & 0xffff0000u);
            } else {
                const unsigned kk = *reinterpret_cast<const unsigned*>(Kb + (size_t)slot * D);
                const unsigned vv = *reinterpret_cast<const unsigned*>(Vb + (size_t)slot * D);
                k[0] = __uint_as_float(kk << 16); k[1] = __uint_as_float(kk & 0xffff0000u);
                v[0] = __uint_as_float(vv << 16); v[1] = __uint_as_float(vv & 0xffff0000u);
            }
            float s = 0.f;
#pragma unroll
            for (int e = 0; e < E; ++e) s += q[e] * k[e];
#pragma unroll
            for (int sh = 16; sh; sh >>= 1) s += __shfl_xor_sync(0xffffffffu, s, sh);
            const float m_new = fmaxf(m, s);
            const float corr = exp2f(m - m_new);
            const float p = exp2f(s - m_new);
            l = l * corr + p;
#pragma unroll
            for (int e = 0; e < E; ++e) o[e] = o[e] * corr + p * v[e];
            m = m_new;
        }
    }

    __shared__ float s_m[4], s_l[4], s_o[4][D];
    if (lane == 0) { s_m[warp] = m; s_l[warp] = l; }
#pragma unroll
    for (int e = 0; e < E; ++e) s_o[warp][lane * E + e] = o[e];
    __syncthreads();
    if (warp == 0) {
        float M = fmaxf(fmaxf(s_m[0], s_m[1]), fmaxf(s_m[2], s_m[3]));
        float L = 0.f, acc[E];
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e] = 0.f;
        if (M > -INFINITY) {
            for (int w = 0; w < 4; ++w) {
                const float f = exp2f(s_m[w] - M);   // 0 for a warp that saw nothing
                L += s_l[w] * f;
#pragma unroll
                for (int e = 0; e < E; ++e) acc[e] += s_o[w][lane * E + e] * f;
            }
        }
        const float inv = L > 0.f ? 1.f / L : 0.f;
        uint16_t* dst = out + qoff;
#pragma unroll
        for (int e = 0; e < E; ++e) dst[e] = __bfloat16_as_ushort(__float2bfloat16_rn(acc[e] * inv));
    }
}

}  // namespace

void svlm_launch_attend_simple(const SvlmAttendBatch& b, int layer0, int n_layers, const void* Q, const int* q_pos,
                               int n_q, int q_heads, void* out, cudaStream_t st) {
    dim3 grid(n_q, q_heads, b.n_caches * n_layers);
    if (b.head_dim == 128)
        attend_simple_kernel<128><<<grid, 128, 0, st>>>(b, layer0, n_layers, (const uint16_t*)Q, q_pos, n_q, q_heads,
                                                       (uint16_t*)out);
    else
        attend_simple_kernel<64><<<grid, 128, 0, st>>>(b, layer0, n_layers, (const uint16_t*)Q, q_pos, n_q, q_heads,
                                                      (uint16_t*)out);
    svlm_count_launch();
}
