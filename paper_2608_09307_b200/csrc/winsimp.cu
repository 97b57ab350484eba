// Exact windowed 2-simplicial attention (the comparison workload of Sec. 4.3 "Baselines": one joint softmax over a
// w1 x w2 pair plane, w1 = 512 keys k_j and w2 = 32 anchors r_c in the paper's runs):
//     s_ijc = sum_a q_i[a] k_j[a] r_c[a],   o_i = sum_{j,c} exp(s_ijc) (v_j * u_c) / sum_{j,c} exp(s_ijc)
// over j in [i - w1 + 1, i], c in [i - w2 + 1, i] (Eq. exact-window-app with a window on the key stream as well).
//
// Flash-style forward on warp-level tensor-core MMAs.  A CTA takes four consecutive queries; a query belongs to two warps
// (16 anchors each).  The composite queries X = q_i * r_c sit in registers as fp16 A-fragments for the whole walk over
// the key window (fp16: bf16 would lose too much in an exponent of this size); per block of 64 keys the warps form the
// scores S = X K^T, keep ONE running maximum per query (the normalisation is joint over the pair plane, so a query's
// maximum is a scalar shared by its two warps), exponentiate, and add P V to their accumulators O[c][e].  At the end
// o_i[e] = sum_c O[c][e] u_c[e] / l_i, the sum over the anchors by shuffles and one exchange through shared memory.
#include <cuda_fp16.h>

#include "../../include/linsimp.h"
#include "common.cuh"
#include "launch.cuh"

namespace linsimp {

static constexpr int WQ = 4;            // queries per CTA
static constexpr int WKB = 64;          // keys per block
static constexpr int WNT = WQ * 64;     // threads: two warps per query

__device__ __forceinline__ void mma_f16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float2 bf2_to_f2(uint32_t w) { return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u)); }
__device__ __forceinline__ uint32_t f2_to_h2(float2 x)
{
    __half2 h = __floats2half2_rn(x.x, x.y);
    return *(uint32_t *)&h;
}
__device__ __forceinline__ uint32_t f2_to_bf2(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *(uint32_t *)&v;
}
__device__ __forceinline__ float ex2w(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int D>
struct WinSmem {
    static constexpr int KP = D + 8;              // K block [64][D] fp16, padded rows
    static constexpr int VP = WKB + 8;            // V^T block [D][64] bf16, padded rows
    static constexpr int OFF_K = 0, OFF_V = OFF_K + WKB * KP * 2, OFF_X = OFF_V + D * VP * 2;
    static constexpr int TOTAL = OFF_X + 2 * 8 * 4 + WQ * 2 * D * 4 + WQ * 2 * 4;
};

// grid (ceil(T / 4), B*H), 256 threads
template <int D>
__global__ void __launch_bounds__(WNT) k_winsimp_fwd(const bf16 *__restrict__ q, const bf16 *__restrict__ k, const bf16 *__restrict__ v,
                                                     const bf16 *__restrict__ r, const bf16 *__restrict__ u, int T, int w1, int w2,
                                                     bf16 *__restrict__ o, float *__restrict__ lse)
{
    using S = WinSmem<D>;
    constexpr float LOG2E = 1.4426950408889634f;
    constexpr int KS = D / 16;                    // k-steps of the score product
    constexpr int NE = D / 8;                     // n-tiles of the value product
    extern __shared__ __align__(16) uint8_t sm[];
    __half *Ks = (__half *)(sm + S::OFF_K);
    bf16 *Vt = (bf16 *)(sm + S::OFF_V);
    float *mx_s = (float *)(sm + S::OFF_X);       // [2 block parities][8 warps] block maxima
    float *osum = mx_s + 16;                      // [4 queries][2 halves][D] partial outputs
    float *lsum = osum + WQ * 2 * D;              // [4 queries][2 halves] partial normalisers
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int qq = warp >> 1, hh = warp & 1;
    const int bh = blockIdx.y, i0 = blockIdx.x * WQ, i = i0 + qq;
    const long base = (long)bh * T * D;
    const bool q_live = i < T;
    // this thread's two anchor rows: steps back s0 = 16 hh + g and s0 + 8
    const int s0 = hh * 16 + g, s1 = s0 + 8;
    const bool row0 = q_live && s0 < w2 && i - s0 >= 0, row1 = q_live && s1 < w2 && i - s1 >= 0;
    // X = q_i * r_c as fp16 A-fragments
    uint32_t xa[KS][4];
    {
        const bf16 *qr = q + base + (long)(q_live ? i : 0) * D;
        const bf16 *r0 = r + base + (long)(row0 ? i - s0 : 0) * D, *r1 = r + base + (long)(row1 ? i - s1 : 0) * D;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                const int col = ks * 16 + hf * 8 + 2 * t;
                const float2 qv = bf2_to_f2(*(const uint32_t *)(qr + col));
                const float2 a = bf2_to_f2(*(const uint32_t *)(r0 + col)), b = bf2_to_f2(*(const uint32_t *)(r1 + col));
                xa[ks][hf * 2 + 0] = row0 ? f2_to_h2(make_float2(qv.x * a.x, qv.y * a.y)) : 0u;
                xa[ks][hf * 2 + 1] = row1 ? f2_to_h2(make_float2(qv.x * b.x, qv.y * b.y)) : 0u;
            }
        }
    }
    float oacc[NE][4];
#pragma unroll
    for (int nt = 0; nt < NE; ++nt) oacc[nt][0] = oacc[nt][1] = oacc[nt][2] = oacc[nt][3] = 0.f;
    float m_run = -INFINITY, l_run = 0.f;         // running maximum (in log2 units) and this warp's part of the normaliser
    const int j_lo = max(0, i0 - (w1 - 1)) / WKB * WKB;
    const int j_hi = min(T - 1, i0 + WQ - 1);
    int par = 0;
    for (int jb = j_lo; jb <= j_hi; jb += WKB, par ^= 1) {
        __syncthreads();                          // the previous block's operands are no longer read
        // stage K (fp16, row-major) and V^T (bf16) of the block
        for (int idx = tid; idx < WKB * (D / 8); idx += WNT) {
            const int row = idx / (D / 8), c8 = idx % (D / 8);
            const int j = jb + row;
            uint4 kv = make_uint4(0, 0, 0, 0), vv = kv;
            if (j < T) {
                kv = *(const uint4 *)(k + base + (long)j * D + c8 * 8);
                vv = *(const uint4 *)(v + base + (long)j * D + c8 * 8);
            }
            const uint32_t kw[4] = {kv.x, kv.y, kv.z, kv.w}, vw[4] = {vv.x, vv.y, vv.z, vv.w};
            uint32_t kh[4];
#pragma unroll
            for (int x = 0; x < 4; ++x) kh[x] = f2_to_h2(bf2_to_f2(kw[x]));
            *(uint4 *)(Ks + row * S::KP + c8 * 8) = make_uint4(kh[0], kh[1], kh[2], kh[3]);
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                Vt[(c8 * 8 + 2 * x) * S::VP + row] = __ushort_as_bfloat16((unsigned short)(vw[x] & 0xffffu));
                Vt[(c8 * 8 + 2 * x + 1) * S::VP + row] = __ushort_as_bfloat16((unsigned short)(vw[x] >> 16));
            }
        }
        __syncthreads();
        // S = X K^T for this warp's 16 rows x 64 keys
        float sc[WKB / 8][4];
#pragma unroll
        for (int nt = 0; nt < WKB / 8; ++nt) {
            sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
            const __half *krow = Ks + (nt * 8 + g) * S::KP + 2 * t;
#pragma unroll
            for (int ks = 0; ks < KS; ++ks)
                mma_f16(sc[nt], xa[ks], *(const uint32_t *)(krow + ks * 16), *(const uint32_t *)(krow + ks * 16 + 8));
        }
        // mask (j in the query's key window, the row's anchor inside the sequence) and the block maximum of the query
        float bm = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < WKB / 8; ++nt) {
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const int j = jb + nt * 8 + 2 * t + (x & 1);
                const bool ok = ((x & 2) ? row1 : row0) && j <= i && j > i - w1;
                sc[nt][x] = ok ? sc[nt][x] * LOG2E : -INFINITY;
                bm = fmaxf(bm, sc[nt][x]);
            }
        }
        bm = warp_max(bm);
        if (lane == 0) mx_s[par * 8 + warp] = bm;
        asm volatile("bar.sync %0, 64;" ::"r"(1 + qq) : "memory");      // the query's two warps
        const float m_new = fmaxf(m_run, fmaxf(mx_s[par * 8 + (warp & ~1)], mx_s[par * 8 + (warp | 1)]));
        if (m_new == -INFINITY) continue;         // nothing of this block is in the window (uniform over the query's warps)
        const float scale = ex2w(m_run - m_new);   // exp2(-inf) = 0 on the first block
        m_run = m_new;
        float ls = 0.f;
        uint32_t pa[WKB / 16][4];                 // P as bf16 A-fragments (two neighbouring score tiles per k-step)
#pragma unroll
        for (int nt = 0; nt < WKB / 8; ++nt) {
            const float p0 = ex2w(sc[nt][0] - m_new), p1 = ex2w(sc[nt][1] - m_new), p2 = ex2w(sc[nt][2] - m_new), p3 = ex2w(sc[nt][3] - m_new);
            ls += (p0 + p1) + (p2 + p3);
            pa[nt >> 1][(nt & 1) * 2 + 0] = f2_to_bf2(p0, p1);
            pa[nt >> 1][(nt & 1) * 2 + 1] = f2_to_bf2(p2, p3);
        }
        l_run = l_run * scale + ls;
        // O = O * scale + P V
#pragma unroll
        for (int nt = 0; nt < NE; ++nt) {
            oacc[nt][0] *= scale; oacc[nt][1] *= scale; oacc[nt][2] *= scale; oacc[nt][3] *= scale;
            const bf16 *vrow = Vt + (nt * 8 + g) * S::VP + 2 * t;
#pragma unroll
            for (int kk = 0; kk < WKB / 16; ++kk)
                mma_bf16(oacc[nt], pa[kk], *(const uint32_t *)(vrow + kk * 16), *(const uint32_t *)(vrow + kk * 16 + 8));
        }
    }
    // o_i[e] = sum_c O[c][e] u_c[e] / l_i : this thread's two rows, then the rows of the warp, then the query's two warps
    {
        const bf16 *u0 = u + base + (long)(row0 ? i - s0 : 0) * D, *u1 = u + base + (long)(row1 ? i - s1 : 0) * D;
#pragma unroll
        for (int nt = 0; nt < NE; ++nt) {
            const int e = nt * 8 + 2 * t;
            const float2 a = row0 ? bf2_to_f2(*(const uint32_t *)(u0 + e)) : make_float2(0.f, 0.f);
            const float2 b = row1 ? bf2_to_f2(*(const uint32_t *)(u1 + e)) : make_float2(0.f, 0.f);
            float x0 = oacc[nt][0] * a.x + oacc[nt][2] * b.x, x1 = oacc[nt][1] * a.y + oacc[nt][3] * b.y;
#pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
                x0 += __shfl_xor_sync(0xffffffffu, x0, off);
                x1 += __shfl_xor_sync(0xffffffffu, x1, off);
            }
            if (g == 0) {
                osum[(qq * 2 + hh) * D + e] = x0;
                osum[(qq * 2 + hh) * D + e + 1] = x1;
            }
        }
        // the normaliser: the rows' sums live in the lanes of equal t; every lane of a quad holds the same two rows' sums
        float lw = l_run;
#pragma unroll
        for (int off = 1; off < 4; off <<= 1) lw += __shfl_xor_sync(0xffffffffu, lw, off);     // over the quad: a row's columns
#pragma unroll
        for (int off = 4; off < 32; off <<= 1) lw += __shfl_xor_sync(0xffffffffu, lw, off);    // over the rows
        if (lane == 0) lsum[qq * 2 + hh] = lw;
    }
    __syncthreads();
    for (int idx = tid; idx < WQ * D; idx += WNT) {
        const int qi = idx / D, e = idx % D;
        const int iq = i0 + qi;
        if (iq >= T) continue;
        const float l = lsum[qi * 2] + lsum[qi * 2 + 1];
        const float val = (osum[(qi * 2) * D + e] + osum[(qi * 2 + 1) * D + e]) / l;
        o[base + (long)iq * D + e] = __float2bfloat16_rn(val);
    }
    if (lse && lane == 0 && hh == 0 && q_live) {
        // (the two warps of a query end with the same running maximum)
        lse[(long)bh * T + i] = (m_run + log2f(lsum[qq * 2] + lsum[qq * 2 + 1])) * 0.6931471805599453f;
    }
}

template <int D>
static int winsimp_launch(const linsimp_params *p, int w1, const void *q, const void *k, const void *v, const void *r, const void *u,
                          void *o, float *lse, cudaStream_t st)
{
    using S = WinSmem<D>;
    LaunchScope sc = {st, 0};
    sc.check(cudaFuncSetAttribute(k_winsimp_fwd<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, S::TOTAL));
    LS_LAUNCH(sc, "winsimp_fwd", k_winsimp_fwd<D><<<dim3((p->T + WQ - 1) / WQ, p->B * p->H), WNT, S::TOTAL, st>>>(
        (const bf16 *)q, (const bf16 *)k, (const bf16 *)v, (const bf16 *)r, (const bf16 *)u, p->T, w1, p->W, (bf16 *)o, lse));
    return sc.result();
}

int winsimp_run(const linsimp_params *p, int w1, const void *q, const void *k, const void *v, const void *r, const void *u, void *o,
                float *lse, cudaStream_t st)
{
    if (p->d == 64) return winsimp_launch<64>(p, w1, q, k, v, r, u, o, lse, st);
    if (p->d == 128) return winsimp_launch<128>(p, w1, q, k, v, r, u, o, lse, st);
    return -2;
}

}  // namespace linsimp
