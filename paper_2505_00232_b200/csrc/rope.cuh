// Rotary embedding combined with the layout transformation of the Q, K and V projections (paper Section 3.6: the
// hand-written kernel of the attention block; query from (B, 1, S, h_q * d_h) to (B * h_kv, S * h_q / h_kv, d_h)).
//
//   token t = b * S + s reads q[t, h_q * d_h], k[t, h_kv * d_h], v[t, h_kv * d_h] (what the q / k / v projections wrote);
//   rotate-half pairs (i, i + d_h / 2), angle from the tables cos / sin [n_pos, d_h / 2] at row pos[t];
//   query head hq = hk * g + j (g = h_q / h_kv) goes to q_out[b * h_kv + hk, s * g + j, :], key and value head hk to
//   k_out / v_out[b * h_kv + hk, s, :]: one contiguous [rows, d_h] block per KV head, the rows the KV cache of
//   Section 3.8 and its score product take in.  V is only moved.
//
// One CTA per token; a work item is 8 elements of the low half of a head together with their partners in the high
// half (two 16-byte loads, two 16-byte stores, the 8 angles as two float4 per table).  Bound: HBM (every element is
// read once and written once).
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ql {

constexpr int kRopeThreads = 256;

struct RopeParams {
    const __half* q; const __half* k; const __half* v;
    const int32_t* pos;
    const float* cos_t; const float* sin_t;
    __half* q_out; __half* k_out; __half* v_out;
    int32_t B, S, h_q, h_kv, d_h, n_pos;
};

__device__ __forceinline__ void rope_unpack8(const uint4& u, float f[8])
{
    const __half2* h = reinterpret_cast<const __half2*>(&u);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 t = __half22float2(h[i]);
        f[2 * i] = t.x;
        f[2 * i + 1] = t.y;
    }
}
__device__ __forceinline__ uint4 rope_pack8(const float f[8])
{
    uint4 u;
    __half2* h = reinterpret_cast<__half2*>(&u);
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2half2_rn(f[2 * i], f[2 * i + 1]);
    return u;
}

__global__ void __launch_bounds__(kRopeThreads) rope_qkv_kernel(const RopeParams p)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel may set up; q, k, v may come from the previous one
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int t = blockIdx.x, b = t / p.S, s = t - b * p.S;
    const int g = p.h_q / p.h_kv, half = p.d_h >> 1, vec_half = half >> 3;
    const int pos = min(max(p.pos[t], 0), p.n_pos - 1);                  // (the caller keeps positions inside the tables)
    const float* cr = p.cos_t + (int64_t)pos * half;
    const float* sr = p.sin_t + (int64_t)pos * half;
    const int rot_items = (p.h_q + p.h_kv) * vec_half;
    const int items = rot_items + p.h_kv * 2 * vec_half;

    for (int it = threadIdx.x; it < items; it += blockDim.x) {
        if (it < rot_items) {
            const int head = it / vec_half, i0 = (it - head * vec_half) << 3;       // q heads first, then k heads
            const bool is_q = head < p.h_q;
            const int hk = is_q ? head / g : head - p.h_q;
            const __half* src = is_q ? p.q + ((int64_t)t * p.h_q + head) * p.d_h : p.k + ((int64_t)t * p.h_kv + hk) * p.d_h;
            __half* dst = is_q ? p.q_out + (((int64_t)(b * p.h_kv + hk) * p.S + s) * g + (head - hk * g)) * p.d_h
                               : p.k_out + ((int64_t)(b * p.h_kv + hk) * p.S + s) * p.d_h;
            float lo[8], hi[8], c[8], sn[8];
            rope_unpack8(*reinterpret_cast<const uint4*>(src + i0), lo);
            rope_unpack8(*reinterpret_cast<const uint4*>(src + half + i0), hi);
            *reinterpret_cast<float4*>(c) = __ldg(reinterpret_cast<const float4*>(cr + i0));
            *reinterpret_cast<float4*>(c + 4) = __ldg(reinterpret_cast<const float4*>(cr + i0 + 4));
            *reinterpret_cast<float4*>(sn) = __ldg(reinterpret_cast<const float4*>(sr + i0));
            *reinterpret_cast<float4*>(sn + 4) = __ldg(reinterpret_cast<const float4*>(sr + i0 + 4));
            float a[8], d[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                a[i] = lo[i] * c[i] - hi[i] * sn[i];
                d[i] = hi[i] * c[i] + lo[i] * sn[i];
            }
            *reinterpret_cast<uint4*>(dst + i0) = rope_pack8(a);
            *reinterpret_cast<uint4*>(dst + half + i0) = rope_pack8(d);
        } else {
            const int w = it - rot_items, hk = w / (2 * vec_half), i0 = (w - hk * 2 * vec_half) << 3;
            const uint4 u = *reinterpret_cast<const uint4*>(p.v + ((int64_t)t * p.h_kv + hk) * p.d_h + i0);
            *reinterpret_cast<uint4*>(p.v_out + ((int64_t)(b * p.h_kv + hk) * p.S + s) * p.d_h + i0) = u;
        }
    }
}

}  // namespace ql
