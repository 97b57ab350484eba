// Single-token decode step (Theorem 1) for bf16 tokens, d and m in {64, 128} (figures below: d = m = 128):
// persistent CTAs, each a
// streaming warpgroup and a computing warpgroup working one (sequence, head) unit apart.
//
// The step is bandwidth-bound by design (fp32 state 64 KB read + written per unit), but its
// 4.3 MFLOP per unit exceed what the CUDA cores can do at HBM speed, so the two 64x128x128
// products run on warp-level tensor-core MMAs (m16n8k16, fp32 accumulate):
//   l[c][p]   = sum_a (q_a r_ca) Omega[a][p]          A = composite queries (fp16), B = Omega (fp16)
//   Dt[e][c]  = sum_p S[p][e] psi'[c][p]              A = state (bf16 from the fp32 copy in shared
//                                                     memory), B = psi' taken straight from the
//                                                     accumulator registers of the first product
// and a thread ends up owning output channels e, so the anchor sum against u_c[e] is a short FMA
// chain plus two shuffles.  The key feature exp(Omega k - |k|^2/2) needs an fp32-accurate
// exponent, so Omega is kept as an fp16 hi + lo pair; that one-row product runs on the tensor cores too.
// The state goes HBM -> shared (cp.async) -> rank-1 update -> HBM with 16-byte accesses.
#include <cuda_fp16.h>

#include "common.cuh"
#include "launch.cuh"
#include "simt_kernels.h"
#include "tc_common.cuh"

namespace linsimp {

static constexpr int DW = 64;

__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1, bool f16)
{
    if (f16)
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                     : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    else
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                     : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2d(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t w)
{
    const float lo = __uint_as_float(w << 16), hi = __uint_as_float(w & 0xffff0000u);
    __half2 h = __floats2half2_rn(lo, hi);
    return *(uint32_t *)&h;
}
__device__ __forceinline__ uint32_t packbf(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *(uint32_t *)&v;
}
// four 8x8 16-bit tiles from shared memory into the fragment layout of the warp-level MMAs (lane l gives the address
// of row l % 8 of tile l / 8); `trans` delivers the tiles transposed
__device__ __forceinline__ void ldsm4(uint32_t (&r)[4], const void *p)
{
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void ldsm4_trans(uint32_t (&r)[4], const void *p)
{
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ float2 unpackbf(uint32_t w)
{
    return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
__device__ __forceinline__ void wg_sync(int wg) { asm volatile("bar.sync %0, 128;" ::"r"(1 + wg) : "memory"); }

// DD: width of q, k, r, v, u (64 or 128); DM: feature rank (64 or 128)
template <int DD, int DM>
struct DecSmem {
    static constexpr int LDT = DD + 8;                             // Omega^T row stride in fp16 elements ([p][a], a contiguous)
    static constexpr int LDP = DD + 8;                             // bf16 state copy [p][e]: row stride in elements
    static constexpr int LDR = DD + 8;                             // ring row stride in bf16 elements
    static constexpr int OM = DM * LDT * 2;                        // one fp16 image of Omega^T
    static constexpr int STATE = DM * LDP * 2;                     // bf16 copy of the state [p][e]
    static constexpr int RING = DW * LDR * 2;
    static constexpr int SMALL = 1024;                             // qh [DD] half, a [DM] float, tpos
    static constexpr int STAGE = STATE + 2 * RING + SMALL;
    static constexpr int PRIV = 6144;                              // compute: red, scratch
    static constexpr int SPRIV = 4096;                             // per streaming warpgroup: two sets of k, v, chi, k (fp16)
    static constexpr int TOTAL = 2 * OM + 2 * STAGE + PRIV + 2 * SPRIV;
};

__device__ __forceinline__ void bar_sync_n(int id, int n) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory"); }
__device__ __forceinline__ void bar_arrive_n(int id, int n) { asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(n) : "memory"); }
__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gsrc)
{
    const uint32_t dst = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(gsrc) : "memory");
}

// Omega [a][p] fp32 -> Omega^T [p][a] as fp16 hi + lo (row stride LDT), by `nthreads` threads
template <int DD, int DM>
__device__ __forceinline__ void stage_omega(const float *__restrict__ omega, __half *omh, __half *oml, int tid, int nthreads)
{
    constexpr int LDT = DecSmem<DD, DM>::LDT;
    for (int idx = tid; idx < DD * DM; idx += nthreads) {
        const int a = idx / DM, p = idx - a * DM;                  // coalesced read of Omega [a][p]
        const float w = omega[idx];
        const __half hi = __float2half_rn(w);
        omh[p * LDT + a] = hi;
        oml[p * LDT + a] = __float2half_rn(w - __half2float(hi));
    }
}

// the image k_decode_mma copies when the caller has prepared it: the two parts back to back
// (one block per feature bank: a shared bank or one per head)
template <int DD, int DM>
__global__ void k_decode_prepare(const float *__restrict__ omega_all, uint8_t *__restrict__ image_all)
{
    using SM = DecSmem<DD, DM>;
    const float *omega = omega_all + (long)blockIdx.x * DD * DM;
    uint8_t *image = image_all + (long)blockIdx.x * 2 * SM::OM;
    for (int idx = threadIdx.x; idx < 2 * SM::OM / 4; idx += blockDim.x) ((uint32_t *)image)[idx] = 0u;   // row padding
    __syncthreads();
    stage_omega<DD, DM>(omega, (__half *)image, (__half *)(image + SM::OM), threadIdx.x, blockDim.x);
}

// 512 threads: warps 0-7 compute, warps 8-11 and 12-15 are two streaming warpgroups, one per
// stage.  A streamer fetches the token, computes the key feature, runs the fp32 state through
// registers (HBM -> update -> HBM) leaving a packed bf16 copy in shared memory, and pulls the
// anchor ring into shared memory with cp.async.  The compute warps do the two tensor-core
// products, the exponentials and the output of the staged unit (each warp 16 anchors x 64
// features).  Stages are handed over with named barriers (full[b] = 1 + b, empty[b] = 3 + b).
template <int DD, int DM>
__global__ void __launch_bounds__(512, 1)
k_decode_mma(const bf16 *__restrict__ q, const bf16 *__restrict__ k, const bf16 *__restrict__ v, const bf16 *__restrict__ r,
             const bf16 *__restrict__ u, const float *__restrict__ omega, int H, int W, int n_units,
             float log2_eps_m, float *__restrict__ S, float *__restrict__ z, bf16 *__restrict__ ring_r,
             bf16 *__restrict__ ring_u, const int *__restrict__ pos, bf16 *__restrict__ o,
             const uint8_t *__restrict__ om_image, int per_head)
{
    using SM = DecSmem<DD, DM>;
    constexpr int LDT = SM::LDT, LDP = SM::LDP, LDR = SM::LDR;
    constexpr int RP = DD / 8;                                     // 16-byte pieces per token row
    constexpr float LOG2E = 1.4426950408889634f;
    extern __shared__ __align__(128) uint8_t dsm[];
    __shared__ uint64_t om_bar;
    __half *omh = (__half *)dsm;                                   // Omega^T [p][a] fp16, hi part
    __half *oml = (__half *)(dsm + SM::OM);                   // lo part
    uint8_t *stages = dsm + 2 * SM::OM;
    uint8_t *priv = stages + 2 * SM::STAGE;
    const int tid = threadIdx.x;
    const bool streamer = tid >= 256;
    const int t128 = tid & 127;                                    // index inside a 128-thread group
    const int cw = tid >> 5;                                       // compute warp 0..7 (tid < 256)
    const int ab = cw & 3, fh = (cw >> 2) & 1;                     // anchor block of 16, feature half of 64
    const int lane = tid & 31, g = lane >> 2, t = lane & 3;

    // Unit schedule.  One bank for all heads: unit = itn * grid + cta.  A bank per head: the grid is a multiple of H,
    // a CTA serves one head (cta % H) for its whole life and walks that head's sequences, so the bank is staged once.
    const int head = per_head ? (int)blockIdx.x % H : 0;
    const int u_first = per_head ? ((int)blockIdx.x / H) * H + head : (int)blockIdx.x;
    const int u_step = per_head ? ((int)gridDim.x / H) * H : (int)gridDim.x;
    if (per_head) {
        omega += (long)head * DD * DM;
        if (om_image) om_image += (long)head * 2 * SM::OM;
    }
    if (om_image) {
        // the prepared image (both parts, laid out as below): two bulk copies behind one barrier
        if (tid == 0) {
            tc::mbar_init(&om_bar, 1);
            tc::fence_barrier_init();
        }
        __syncthreads();
        if (tid == 0) {
            tc::mbar_arrive_expect_tx(&om_bar, 2 * SM::OM);
            tc::bulk_g2s(dsm, om_image, SM::OM, &om_bar);
            tc::bulk_g2s(dsm + SM::OM, om_image + SM::OM, SM::OM, &om_bar);
        }
        tc::mbar_wait(&om_bar, 0, nullptr, 0);                     // bounded
    } else {
        stage_omega<DD, DM>(omega, omh, oml, tid, 512);
    }
    __syncthreads();
    const int n_mine = u_first < n_units ? (n_units - u_first + u_step - 1) / u_step : 0;   // units of this CTA

    if (streamer) {
        // ------------------------------------------------------------ streamer
        // two streaming warpgroups, one per stage: warpgroup sw serves the units with itn % 2 == sw
        const int sw = (tid - 256) >> 7;
        const int wq = t128 >> 5;                                  // warp inside the streaming warpgroup
        // The token of this warpgroup's next unit (k, v, q elements, position, normaliser entry, the new ring rows) is
        // fetched into registers one unit ahead, so that a unit starts without waiting on global memory.
        bf16 kq = __float2bfloat16_rn(0.f), vq = kq, qq = kq;
        int tpos_n = 0;
        float z_n = 0.f;
        uint4 rq = make_uint4(0, 0, 0, 0), uq = rq;
        auto fetch_token = [&](int itn_) {
            if (itn_ < n_mine) {
                const int un = itn_ * u_step + u_first;
                const long off = (long)un * DD;
                if (t128 < DD) {
                    kq = k[off + t128];
                    vq = v[off + t128];
                    qq = q[off + t128];
                }
                tpos_n = pos[un / H];
                if (t128 < DM) z_n = z[(long)un * DM + t128];
                if (t128 < RP) {
                    rq = ((const uint4 *)(r + off))[t128];
                    uq = ((const uint4 *)(u + off))[t128];
                }
            }
        };
        fetch_token(sw);
        for (int itn = sw; itn < n_mine; itn += 2) {
            const int b = sw;
            const int unit = itn * u_step + u_first;
            // per-unit scratch in two sets (by unit parity): a warp that runs ahead into the next unit must not
            // overwrite v and chi while another warp of the group still reads them in its rank-1 update
            float *ks = (float *)(priv + SM::PRIV + sw * SM::SPRIV + ((itn >> 1) & 1) * (SM::SPRIV / 2));   // [DD]
            float *vs = ks + DD;                                       // [DD]
            float *chis = vs + DD;                                     // [DM]
            __half *kh = (__half *)(chis + DM);                        // [DD] the key as fp16 (exact for bf16 values in range)
            uint8_t *st = stages + b * SM::STAGE;
            bf16 *sbf = (bf16 *)st;                                // bf16 copy of the updated state, [p][e]
            bf16 *rr_s = (bf16 *)(st + SM::STATE), *ru_s = rr_s + DW * LDR;
            __half *qh = (__half *)(st + SM::STATE + 2 * SM::RING);
            float *as_ = (float *)(qh + DD);
            int *tp = (int *)(as_ + DM);
            const int tpos = tpos_n;
            const int slot = tpos % W;
            const long tok_off = (long)unit * DD;
            bf16 *rr_g = ring_r + (long)unit * W * DD, *ru_g = ring_u + (long)unit * W * DD;
            float *Sg = S + (long)unit * DM * DD, *zg = z + (long)unit * DM;
            // Everything that does not touch the stage happens before the stage is waited for: the
            // token, the first half of the state (into registers) and the key feature.
            if (t128 < DD) {
                ks[t128] = __bfloat162float(kq);
                kh[t128] = __float2half_rn(ks[t128]);
                vs[t128] = __bfloat162float(vq);
            }
            const __half qv = __float2half_rn(__bfloat162float(qq));
            const float z_old = z_n;
            if (t128 < RP) {
                ((uint4 *)(rr_g + (long)slot * DD))[t128] = rq;
                ((uint4 *)(ru_g + (long)slot * DD))[t128] = uq;
            }
            // state rows (2*p2, 2*p2+1), 16 bytes of each per item
            constexpr int ITEMS = (DM / 2) * (DD / 4) / 128;       // items per thread (16 for d = m = 128)
            constexpr int RQ = DD / 4;                             // float4 pieces per state row
            float4 s0[ITEMS / 2], s1[ITEMS / 2];
#pragma unroll
            for (int i = 0; i < ITEMS / 2; ++i) {
                const int f = t128 + 128 * i, p2 = f / RQ, e4 = f % RQ;
                s0[i] = ((const float4 *)(Sg + (long)(2 * p2) * DD))[e4];
                s1[i] = ((const float4 *)(Sg + (long)(2 * p2 + 1) * DD))[e4];
            }
            fetch_token(itn + 2);
            bar_sync_n(5 + sw, 128);
            {
                // key feature exp(Omega k - |k|^2/2) with an fp32-accurate exponent: l = k . (Omega_hi + Omega_lo) as a
                // one-row product on the tensor cores (row 0 of the m16 tile holds the key; fp16 x fp16 products are
                // exact in the fp32 accumulator); this warp owns features [DM/4 wq, DM/4 wq + DM/4)
                float nrm = 0.f;
                {
                    if (lane * 4 < DD) {
                        const float4 k4 = *(const float4 *)(ks + lane * 4);
                        nrm = fmaf(k4.x, k4.x, fmaf(k4.y, k4.y, fmaf(k4.z, k4.z, k4.w * k4.w)));
                    }
#pragma unroll
                    for (int off = 16; off > 0; off >>= 1) nrm += __shfl_xor_sync(0xffffffffu, nrm, off);
                }
#pragma unroll
                for (int np = 0; np < DM / 64; ++np) {             // two feature blocks of 8 at a time (register budget)
                    float c[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
                    for (int ks_ = 0; ks_ < DD / 16; ++ks_) {
                        const int a = ks_ * 16 + 2 * t;
                        uint32_t af[4] = {0u, 0u, 0u, 0u};
                        if (g == 0) {
                            af[0] = *(const uint32_t *)(kh + a);
                            af[2] = *(const uint32_t *)(kh + a + 8);
                        }
                        {
                            // both feature blocks of 8 (and both halves of the k-step) per fragment load
                            const int i0 = ((wq * (DM / 32) + np * 2 + (lane >> 4)) * 8 + (lane & 7)) * LDT + ks_ * 16 + ((lane >> 3) & 1) * 8;
                            uint32_t bh_[4], bl_[4];
                            ldsm4(bh_, omh + i0);
                            ldsm4(bl_, oml + i0);
                            mma_16816(c[0], af, bh_[0], bh_[1], true);
                            mma_16816(c[0], af, bl_[0], bl_[1], true);
                            mma_16816(c[1], af, bh_[2], bh_[3], true);
                            mma_16816(c[1], af, bl_[2], bl_[3], true);
                        }
                    }
                    if (g == 0) {
#pragma unroll
                        for (int nt = 0; nt < 2; ++nt) {
                            const int p = wq * (DM / 4) + (np * 2 + nt) * 8 + 2 * t;
                            chis[p] = expf(c[nt][0] - 0.5f * nrm);
                            chis[p + 1] = expf(c[nt][1] - 0.5f * nrm);
                        }
                    }
                }
            }
            bar_sync_n(5 + sw, 128);                               // chis visible
            const float a_new = (t128 < DM) ? z_old + chis[t128] : 0.f;
            if (t128 < DM) zg[t128] = a_new;
            if (itn >= 2) bar_sync_n(3 + b, 384);                  // stage b consumed (128 streamers + 256 compute)
            // anchors: ring rows (the current token's row comes from r, u), 16 x 16-byte pieces per row
            for (int idx = t128; idx < DW * RP; idx += 128) {
                const int row = idx / RP, c16 = idx % RP;
                if (row < W) {
                    const bf16 *src_r = (row == slot) ? r + tok_off : rr_g + (long)row * DD;
                    const bf16 *src_u = (row == slot) ? u + tok_off : ru_g + (long)row * DD;
                    cp_async16(rr_s + row * LDR + c16 * 8, src_r + c16 * 8);
                    cp_async16(ru_s + row * LDR + c16 * 8, src_u + c16 * 8);
                }
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
            if (t128 < DD) qh[t128] = qv;
            if (t128 < DM) as_[t128] = a_new;
            if (t128 == 0) *tp = tpos;
            // rank-1 update, write back, packed bf16 copy (rows p, p+1) to shared
            const float4 v4 = *(const float4 *)(vs + (t128 % RQ) * 4);     // this thread's four channels in every piece
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                if (half == 1) {
#pragma unroll
                    for (int i = 0; i < ITEMS / 2; ++i) {
                        const int f = t128 + 128 * (i + ITEMS / 2), p2 = f / RQ, e4 = f % RQ;
                        s0[i] = ((const float4 *)(Sg + (long)(2 * p2) * DD))[e4];
                        s1[i] = ((const float4 *)(Sg + (long)(2 * p2 + 1) * DD))[e4];
                    }
                }
#pragma unroll
                for (int i = 0; i < ITEMS / 2; ++i) {
                    const int f = t128 + 128 * (i + half * (ITEMS / 2)), p2 = f / RQ, e4 = f % RQ;
                    float4 a0 = s0[i], a1 = s1[i];
                    const float2 c01 = *(const float2 *)(chis + 2 * p2);
                    const float c0 = c01.x, c1 = c01.y;
                    a0.x = fmaf(c0, v4.x, a0.x); a0.y = fmaf(c0, v4.y, a0.y); a0.z = fmaf(c0, v4.z, a0.z); a0.w = fmaf(c0, v4.w, a0.w);
                    a1.x = fmaf(c1, v4.x, a1.x); a1.y = fmaf(c1, v4.y, a1.y); a1.z = fmaf(c1, v4.z, a1.z); a1.w = fmaf(c1, v4.w, a1.w);
                    ((float4 *)(Sg + (long)(2 * p2) * DD))[e4] = a0;
                    ((float4 *)(Sg + (long)(2 * p2 + 1) * DD))[e4] = a1;
                    *(uint2 *)(sbf + (2 * p2) * LDP + e4 * 4) = make_uint2(packbf(a0.x, a0.y), packbf(a0.z, a0.w));
                    *(uint2 *)(sbf + (2 * p2 + 1) * LDP + e4 * 4) = make_uint2(packbf(a1.x, a1.y), packbf(a1.z, a1.w));
                }
            }
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            __threadfence_block();
            bar_arrive_n(1 + b, 384);                              // stage b full
        }
    } else {
        // ------------------------------------------------------------ compute
        float *red = (float *)priv;                                // [8][DD]
        float *scr = red + 8 * DD;                                 // [16]
        for (int itn = 0; itn < n_mine; ++itn) {
            const int b = itn & 1;
            const int unit = itn * u_step + u_first;
            const uint8_t *st = stages + b * SM::STAGE;
            const bf16 *sbf = (const bf16 *)st;
            const bf16 *rr_s = (const bf16 *)(st + SM::STATE), *ru_s = rr_s + DW * LDR;
            const __half *qh = (const __half *)(st + SM::STATE + 2 * SM::RING);
            const float *as_ = (const float *)(qh + DD);
            const int *tp = (const int *)(as_ + DM);
            bar_sync_n(1 + b, 384);                                // stage b full
            const int tpos = *tp;
            const long tok_off = (long)unit * DD;
            const int row0 = ab * 16 + g, row1 = row0 + 8;
            const bool ok0 = (row0 < W) && (tpos + 1 >= W || row0 <= tpos);
            const bool ok1 = (row1 < W) && (tpos + 1 >= W || row1 <= tpos);
            // fragment loads by ldmatrix: lane l addresses row l % 8 of tile l / 8
            const int lt = lane >> 3, lr = lane & 7;
            const bf16 *ra_lane = rr_s + min(ab * 16 + (lt & 1) * 8 + lr, W - 1) * LDR + (lt >> 1) * 8;   // anchors x a
            const __half *om_lane = omh + ((fh * (DM / 16) + (lt >> 1)) * 8 + lr) * LDT + (lt & 1) * 8;   // features x a
            const bf16 *st_lane = sbf + ((lt >> 1) * 8 + lr) * LDP + (lt & 1) * 8;                        // p x channels
            // ---- GEMM-1: l[c][p], 16 anchors x 64 features per warp
            constexpr int NTW = DM / 16;                           // feature blocks of 8 per warp
            float acc[NTW][4];
#pragma unroll
            for (int nt = 0; nt < NTW; ++nt)
#pragma unroll
                for (int x = 0; x < 4; ++x) acc[nt][x] = 0.f;
            float hn0 = 0.f, hn1 = 0.f;
#pragma unroll
            for (int ks_ = 0; ks_ < DD / 16; ++ks_) {
                const int a = ks_ * 16 + 2 * t;
                const uint32_t q0 = *(const uint32_t *)(qh + a), q1 = *(const uint32_t *)(qh + a + 8);
                uint32_t af[4];
                {
                    uint32_t rw[4];                                // r of anchors (g, g+8) x a (2t.., 2t+8..) as bf16 pairs
                    ldsm4(rw, ra_lane + ks_ * 16);
                    const uint32_t r0 = bf16x2_to_f16x2(rw[0]), r1 = bf16x2_to_f16x2(rw[1]);
                    const uint32_t r2 = bf16x2_to_f16x2(rw[2]), r3 = bf16x2_to_f16x2(rw[3]);
                    const __half2 x0 = __hmul2(*(const __half2 *)&q0, *(const __half2 *)&r0);
                    const __half2 x1 = __hmul2(*(const __half2 *)&q0, *(const __half2 *)&r1);
                    const __half2 x2 = __hmul2(*(const __half2 *)&q1, *(const __half2 *)&r2);
                    const __half2 x3 = __hmul2(*(const __half2 *)&q1, *(const __half2 *)&r3);
                    af[0] = *(const uint32_t *)&x0;
                    af[1] = *(const uint32_t *)&x1;
                    af[2] = *(const uint32_t *)&x2;
                    af[3] = *(const uint32_t *)&x3;
                    const float2 f0 = __half22float2(x0), f1 = __half22float2(x1), f2 = __half22float2(x2), f3 = __half22float2(x3);
                    hn0 = fmaf(f0.x, f0.x, fmaf(f0.y, f0.y, fmaf(f2.x, f2.x, fmaf(f2.y, f2.y, hn0))));
                    hn1 = fmaf(f1.x, f1.x, fmaf(f1.y, f1.y, fmaf(f3.x, f3.x, fmaf(f3.y, f3.y, hn1))));
                }
#pragma unroll
                for (int nt = 0; nt < NTW; nt += 2) {              // two feature blocks of 8 per fragment load
                    uint32_t bw[4];
                    ldsm4(bw, om_lane + nt * 8 * LDT + ks_ * 16);
                    mma_16816(acc[nt], af, bw[0], bw[1], true);
                    mma_16816(acc[nt + 1], af, bw[2], bw[3], true);
                }
            }
            hn0 += __shfl_xor_sync(0xffffffffu, hn0, 1);
            hn0 += __shfl_xor_sync(0xffffffffu, hn0, 2);
            hn1 += __shfl_xor_sync(0xffffffffu, hn1, 1);
            hn1 += __shfl_xor_sync(0xffffffffu, hn1, 2);
            hn0 *= 0.5f;
            hn1 *= 0.5f;
            // ---- shift L = max over valid anchors and features
            float mx = -INFINITY;
#pragma unroll
            for (int nt = 0; nt < NTW; ++nt) {
                if (ok0) mx = fmaxf(mx, fmaxf(acc[nt][0], acc[nt][1]) - hn0);
                if (ok1) mx = fmaxf(mx, fmaxf(acc[nt][2], acc[nt][3]) - hn1);
            }
            mx = warp_max(mx);
            if (lane == 0) scr[cw] = mx;
            bar_sync_n(7, 256);
            float L = scr[0];
#pragma unroll
            for (int x = 1; x < 8; ++x) L = fmaxf(L, scr[x]);
            // ---- psi' = exp(l - L) as B fragments of the second product; normaliser
            const float sh0 = ok0 ? (hn0 + L) * LOG2E : INFINITY, sh1 = ok1 ? (hn1 + L) * LOG2E : INFINITY;
            uint32_t pb[NTW][2];                                   // [feature block of 8][anchor g / g+8]
            float zeta = 0.f;
#pragma unroll
            for (int nt = 0; nt < NTW; ++nt) {
                const float2 a2 = *(const float2 *)(as_ + (fh * NTW + nt) * 8 + 2 * t);
                const float p0 = ex2d(fmaf(acc[nt][0], LOG2E, -sh0)), p1 = ex2d(fmaf(acc[nt][1], LOG2E, -sh0));
                const float p2 = ex2d(fmaf(acc[nt][2], LOG2E, -sh1)), p3 = ex2d(fmaf(acc[nt][3], LOG2E, -sh1));
                zeta = fmaf(p0, a2.x, fmaf(p1, a2.y, fmaf(p2, a2.x, fmaf(p3, a2.y, zeta))));
                pb[nt][0] = packbf(p0, p1);
                pb[nt][1] = packbf(p2, p3);
            }
            zeta = warp_sum(zeta);
            if (lane == 0) scr[8 + cw] = zeta;
            // ---- GEMM-2 (transposed), this warp's 64 features: Dt[e][c] partial; 128 channels x 16 anchors
            const int c_lo = ab * 16 + 2 * t;                      // anchors c_lo, c_lo+1 (first tile), +8, +9 (second)
            (void)c_lo;
            // u of this warp's 16 anchors x 16 channels, transposed: tiles (anchors 0-7 | 8-15) x (channels 0-7 | 8-15)
            const bf16 *u_lane = ru_s + min(ab * 16 + (lt & 1) * 8 + lr, W - 1) * LDR + (lt >> 1) * 8;
            float npart[DD / 16][2];
#pragma unroll
            for (int mt = 0; mt < DD / 16; ++mt) {
                float d0[4] = {0.f, 0.f, 0.f, 0.f}, d1[4] = {0.f, 0.f, 0.f, 0.f};
                const int e0 = mt * 16 + g;
#pragma unroll
                for (int j = 0; j < NTW / 2; ++j) {
                    uint32_t af[4];                                // state rows p (16 of them) x channels (16), transposed
                    ldsm4_trans(af, st_lane + (fh * (NTW / 2) + j) * 16 * LDP + mt * 16);
                    mma_16816(d0, af, pb[2 * j][0], pb[2 * j + 1][0], false);
                    mma_16816(d1, af, pb[2 * j][1], pb[2 * j + 1][1], false);
                }
                // rows e0 (x = 0, 1) and e0 + 8 (x = 2, 3); columns c_lo, c_lo + 1 of each anchor tile
                (void)e0;
                uint32_t uw[4];        // (anchors c_lo, c_lo+1 | c_lo+8, c_lo+9) of channel e0, then of channel e0 + 8
                ldsm4_trans(uw, u_lane + mt * 16);
                const float2 ua = unpackbf(uw[0]), ub = unpackbf(uw[1]), uc = unpackbf(uw[2]), ud = unpackbf(uw[3]);
                float n0 = d0[0] * ua.x + d0[1] * ua.y + d1[0] * ub.x + d1[1] * ub.y;
                float n1 = d0[2] * uc.x + d0[3] * uc.y + d1[2] * ud.x + d1[3] * ud.y;
                n0 += __shfl_xor_sync(0xffffffffu, n0, 1);
                n0 += __shfl_xor_sync(0xffffffffu, n0, 2);
                n1 += __shfl_xor_sync(0xffffffffu, n1, 1);
                n1 += __shfl_xor_sync(0xffffffffu, n1, 2);
                npart[mt][0] = n0;
                npart[mt][1] = n1;
            }
            if (t == 0) {
#pragma unroll
                for (int mt = 0; mt < DD / 16; ++mt) {
                    red[cw * DD + mt * 16 + g] = npart[mt][0];
                    red[cw * DD + mt * 16 + g + 8] = npart[mt][1];
                }
            }
            bar_sync_n(7, 256);
            bar_arrive_n(3 + b, 384);                              // stage b may be refilled
            if (tid < DD) {
                float Z = 0.f, N = 0.f;
#pragma unroll
                for (int x = 0; x < 8; ++x) {
                    Z += scr[8 + x];
                    N += red[x * DD + tid];
                }
                const float den = fmaxf(Z + ex2d(log2_eps_m - L * LOG2E), 1e-37f);
                o[tok_off + tid] = __float2bfloat16_rn(N / den);
            }
            bar_sync_n(7, 256);                                    // red, scr free for the next unit
        }
    }
}

// banks: 1 (one Omega for all heads) or H (one per head; every CTA then serves one head, which needs H <= the SM count)
int decode_mma_supported(int d, int m, int W, int banks)
{
    return (d == 64 || d == 128) && (m == 64 || m == 128) && W <= DW && W >= 1 && banks <= sm_count();
}

size_t decode_mma_image_bytes(int d, int m, int banks) { return 2 * (size_t)m * (d + 8) * 2 * banks; }

template <int DD, int DM>
static int decode_prepare_t(const float *omega, int banks, void *image, cudaStream_t st)
{
    LaunchScope sc = {st, 0};
    LS_LAUNCH(sc, "decode_prepare", k_decode_prepare<DD, DM><<<banks, 1024, 0, st>>>(omega, (uint8_t *)image));
    return sc.result();
}

int decode_mma_prepare(const float *omega, int d, int m, int banks, void *image, cudaStream_t st)
{
    if (d == 128 && m == 128) return decode_prepare_t<128, 128>(omega, banks, image, st);
    if (d == 128 && m == 64) return decode_prepare_t<128, 64>(omega, banks, image, st);
    if (d == 64 && m == 128) return decode_prepare_t<64, 128>(omega, banks, image, st);
    if (d == 64 && m == 64) return decode_prepare_t<64, 64>(omega, banks, image, st);
    return -2;
}

template <int DD, int DM>
static int decode_run_t(const SimtArgs &a, const void *omega_image, cudaStream_t st)
{
    using SM = DecSmem<DD, DM>;
    const int n_units = a.B * a.H;
    LaunchScope sc = {st, 0};
    sc.check(cudaFuncSetAttribute(k_decode_mma<DD, DM>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM::TOTAL));
    const int per_head = a.omega_stride != 0 && a.H > 1;
    const int sms = sm_count();
    int grid = n_units < sms ? n_units : sms;
    if (per_head) grid = (grid / a.H) * a.H;               // a multiple of H (n_units is one, and H <= the SM count)
    const float log2_eps_m = a.log_eps_m * 1.4426950408889634f;
    LS_LAUNCH(sc, "decode_mma", k_decode_mma<DD, DM><<<grid, 512, SM::TOTAL, st>>>(
        (const bf16 *)a.q, (const bf16 *)a.k, (const bf16 *)a.v, (const bf16 *)a.r, (const bf16 *)a.u, a.omega, a.H, a.W,
        n_units, log2_eps_m, a.S_final, a.z_final, (bf16 *)a.ring_r, (bf16 *)a.ring_u, a.pos,
        (bf16 *)a.o, (const uint8_t *)omega_image, per_head));
    return sc.result();
}

int decode_mma_run(const SimtArgs &a, const void *omega_image, cudaStream_t st)
{
    if (a.d == 128 && a.m == 128) return decode_run_t<128, 128>(a, omega_image, st);
    if (a.d == 128 && a.m == 64) return decode_run_t<128, 64>(a, omega_image, st);
    if (a.d == 64 && a.m == 128) return decode_run_t<64, 128>(a, omega_image, st);
    if (a.d == 64 && a.m == 64) return decode_run_t<64, 64>(a, omega_image, st);
    return -2;
}

}  // namespace linsimp
