// Pieces shared by the kernels that keep a 128 x 128 fp32 state tile in the registers of 256 threads.
// Thread layout: warp w owns rows 16 w .. 16 w + 15 (rows = value components c, contiguous in memory along the key
// dimension); lane = 8 r4 + l8; a thread holds rows 16 w + 4 i + r4 (i = 0..3) and of each row the key positions
// 64 kh + 8 l8 + e (kh = 0,1; e = 0..7) as x[i][2 kh], x[i][2 kh + 1].  A warp instruction therefore covers four
// rows, the eight lanes of a row each owning 32 contiguous bytes of either half.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

namespace gdn {

constexpr int GDN_TILE_D = 128;

// 32-byte global accesses (one instruction per eight floats: half the load/store instructions of float4).
__device__ __forceinline__ void ldg_v8(const float *p, float4 &a, float4 &b)
{
    asm volatile("ld.global.L1::no_allocate.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(a.x), "=f"(a.y), "=f"(a.z), "=f"(a.w), "=f"(b.x), "=f"(b.y), "=f"(b.z), "=f"(b.w)
                 : "l"(p)
                 : "memory");
}
__device__ __forceinline__ void stg_v8(float *p, const float4 &a, const float4 &b)
{
    asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 ::"l"(p), "f"(a.x), "f"(a.y), "f"(a.z), "f"(a.w), "f"(b.x), "f"(b.y), "f"(b.z), "f"(b.w)
                 : "memory");
}

// Eq. 7 replayed along an accepted path of L >= 1 nodes on the tile x (Section 3.4: the delayed commit is a short
// recurrence).  Per row c: s_c <- alpha s_c + k beta (v_c - alpha k.s_c); the eight lanes that share a row reduce
// k.s_c by shuffles (the four rows of a thread folded into one butterfly), the four rows of a thread advance together.
//   pks, pvs : the path's k and v rows in shared memory, bf16 [L][128]
//   ab_path  : per step (A_t = decay of the path up to and including step t, beta_t, alpha_t, 1 / A_t)
__device__ __forceinline__ void replay_path_on_tile(float4 (&x)[4][4], int L, const uint16_t *pks, const uint16_t *pvs,
                                                    const float4 *ab_path, int warp, int r4, int l8)
{
    // Scaled form: with A_t = alpha_1 .. alpha_t and s~ = s / A_t a step is s~ += k beta_t (v / A_t - k.s~)
    // (the decay costs nothing), and s = A_L s~ at the end.  It is taken unless the path decays below 2^-80:
    // then 1 / A_t could overflow and the plain form alpha s + k w is used.
    const bool scaled = ab_path[L - 1].x > 8.3e-25f;
#pragma unroll 1
    for (int t = 0; t < L; ++t) {
        // this thread's sixteen key positions: 64*kh + 8*l8 + e
        float kf[16];
#pragma unroll
        for (int kh = 0; kh < 2; ++kh) {
            const uint4 kw = *reinterpret_cast<const uint4 *>(pks + t * GDN_TILE_D + kh * 64 + l8 * 8);
            const uint32_t w4[4] = {kw.x, kw.y, kw.z, kw.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                kf[kh * 8 + 2 * e] = __uint_as_float(w4[e] << 16);
                kf[kh * 8 + 2 * e + 1] = __uint_as_float(w4[e] & 0xFFFF0000u);
            }
        }
        const float4 ab = ab_path[t];   // (A_t, beta_t, alpha_t, 1 / A_t)
        // the four rows of this thread advance together: four independent FMA chains, then their
        // shuffle reductions back to back, then the four updates
        float dot[4];
        float2 kf2[8];   // the same values as packed pairs for the two-wide fp32 FMA
#pragma unroll
        for (int e = 0; e < 8; ++e) kf2[e] = make_float2(kf[2 * e], kf[2 * e + 1]);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float2 acc = make_float2(0.f, 0.f);
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
                acc = __ffma2_rn(kf2[q4 * 2 + 0], make_float2(x[i][q4].x, x[i][q4].y), acc);
                acc = __ffma2_rn(kf2[q4 * 2 + 1], make_float2(x[i][q4].z, x[i][q4].w), acc);
            }
            dot[i] = acc.x + acc.y;
        }
        // Reduction over the eight lanes of a row group with the four rows folded as it goes: after the exchange
        // with lane ^ 1 a lane keeps two rows, after lane ^ 2 one, after lane ^ 4 it holds the complete k.s of row
        // my_i (4 shuffles instead of 12); it forms w of that row alone and the four w come back by shuffles.
        const bool b0 = (l8 & 1) != 0, b1 = (l8 & 2) != 0;
        const int my_i = (b0 ? 2 : 0) + (b1 ? 1 : 0);
        float a0, a1;
        {
            const float s0 = b0 ? dot[0] : dot[2], s1 = b0 ? dot[1] : dot[3];
            const float r0 = __shfl_xor_sync(0xffffffffu, s0, 1), r1 = __shfl_xor_sync(0xffffffffu, s1, 1);
            a0 = (b0 ? dot[2] : dot[0]) + r0;
            a1 = (b0 ? dot[3] : dot[1]) + r1;
        }
        float d1 = (b1 ? a1 : a0) + __shfl_xor_sync(0xffffffffu, b1 ? a0 : a1, 2);
        d1 += __shfl_xor_sync(0xffffffffu, d1, 4);
        const int my_row = warp * 16 + my_i * 4 + r4;
        const float vc = __uint_as_float((uint32_t)pvs[t * GDN_TILE_D + my_row] << 16);
        // scaled form: x holds s / A_t and w = beta_t (v / A_t - k.s~); plain form: w = beta_t (v - alpha_t k.s)
        const float w_mine = scaled ? ab.y * fmaf(vc, ab.w, -d1) : ab.y * (vc - ab.z * d1);
        const int g8 = (r4 << 3);   // first lane of this row group
        float wv[4];
        wv[0] = __shfl_sync(0xffffffffu, w_mine, g8 | 0);
        wv[1] = __shfl_sync(0xffffffffu, w_mine, g8 | 2);
        wv[2] = __shfl_sync(0xffffffffu, w_mine, g8 | 1);
        wv[3] = __shfl_sync(0xffffffffu, w_mine, g8 | 3);
        if (scaled) {
            // s~ += k w, one packed FMA per pair
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 w2 = make_float2(wv[i], wv[i]);
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    const float2 lo = __ffma2_rn(kf2[q4 * 2 + 0], w2, make_float2(x[i][q4].x, x[i][q4].y));
                    const float2 hi = __ffma2_rn(kf2[q4 * 2 + 1], w2, make_float2(x[i][q4].z, x[i][q4].w));
                    x[i][q4] = make_float4(lo.x, lo.y, hi.x, hi.y);
                }
            }
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 w2 = make_float2(wv[i], wv[i]), a2 = make_float2(ab.z, ab.z);
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    const float2 lo = __ffma2_rn(kf2[q4 * 2 + 0], w2, __fmul2_rn(a2, make_float2(x[i][q4].x, x[i][q4].y)));
                    const float2 hi = __ffma2_rn(kf2[q4 * 2 + 1], w2, __fmul2_rn(a2, make_float2(x[i][q4].z, x[i][q4].w)));
                    x[i][q4] = make_float4(lo.x, lo.y, hi.x, hi.y);
                }
            }
        }
    }
    if (scaled) {   // back to s = A_L s~
        const float aL = ab_path[L - 1].x;
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4)
                x[i][q4] = make_float4(aL * x[i][q4].x, aL * x[i][q4].y, aL * x[i][q4].z, aL * x[i][q4].w);
    }
}

}  // namespace gdn
