// Tensor-core (tcgen05 / TMEM) forward of the LinSimp hot path for bf16 I/O.
//
// Pre-pass (k_prep_tc5, k_state_tc): key features chi' = exp(l(k)) in fp32, the boundary
// states as an exclusive prefix over chunks in fp32 (all on tcgen05), and the operand
// "images" the main kernel bulk-copies: the boundary state as bf16 [e][p] (K-major,
// 128-byte swizzle), the chunk's key features as bf16 [j][p], and the chunk's values
// transposed as bf16 [e][j] (32-byte swizzle).
//
// Main kernel (k_fwd_tc): a CTA walks consecutive chunks of one (batch, head).  A tile is
// 128 composite-query rows = 2 queries x 64 anchors.  Per tile, on tcgen05:
//   GEMM-1  l_raw[(i,c), p]  = X[(i,c), :] . OmegaT[p, :]      (X = q_i*r_c in fp16, A from TMEM)
//   GEMM-P  P[(i,c), j]      = psi'[(i,c), :] . chi'[j, :]      (intra-chunk pair weights)
//   GEMM-2  Dt[e, (i,c)]     = MbT[e, :] . psi'[(i,c), :] + Vt[e, :] . Pm[(i,c), :]
// with psi' = exp(l - L_i) written to shared memory as bf16 between GEMM-1 and GEMM-2.
// GEMM-2 is computed transposed so that a thread owns one output channel e and sums the
// anchors with plain FMAs against u_c[e]; only the scalar normaliser needs a warp-shuffle
// reduction.  Each of the two warpgroups owns a private TMEM region and runs its tiles
// start to finish; the two overlap each other's tensor and SFU phases.
#include "common.cuh"
#include "launch.cuh"
#include "tc_common.cuh"
#include "tc_kernels.h"

#include <cuda_fp16.h>

namespace linsimp {
using namespace tc;

static constexpr int TC_C = kTcChunk;       // tokens per chunk
static constexpr int TC_SLOTS = 2;          // tiles in flight per CTA
static constexpr int TC_NT = TC_SLOTS * 256;

// ------------------------------------------------------------------ image geometry
// all byte sizes; MF in {64,128}, D in {64,128}
template <int D, int MF>
struct TcGeom {
    static constexpr int KB_M = MF / 64;                        // 64-wide feature blocks
    static constexpr int KB_D = D / 64;
    static constexpr int IMG_M = 128 * MF * 2;                  // [e (padded to 128)][p] bf16, per feature block [128][128B]
    static constexpr int IMG_CHI = TC_C * MF * 2;               // [j][p] bf16, per feature block [16][128B]
    static constexpr int IMG_VT = 128 * 32;                     // [e (padded to 128)][j] bf16, rows of 32 B
    static constexpr int IMG_CHUNK = IMG_M + IMG_CHI + IMG_VT;  // contiguous per chunk, bulk-copied in one go
    static constexpr int IMG_OM = MF * D * 2;                   // OmegaT [p][a] fp16, per a-block [MF][128B]
};

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *(uint32_t *)&v;
}

// ------------------------------------------------------------------ pre-pass 1: key features, chunk images
// Tiles of 128 tokens (8 chunks), on tcgen05:
//   l[tok][p] = sum_a k[tok][a] Omega[a][p]     A = the k rows as they are (bf16, exact), B = Omega^T in three bf16 terms
// (24 mantissa bits: the exponent argument stays fp32-accurate), accumulator in tensor memory; chi' = exp(l - |k|^2/2)
// in fp32 goes through a shared-memory tile from which all outputs are written with coalesced stores: each chunk's chi'
// operand image (bf16), the two further bf16 terms of chi' the state products use (chi_ml), fp32 rows for the backward
// (chi32, optional) and the chunk's V^T operand image.  Tokens at or beyond a padded sequence's own length have no key
// feature, hence add nothing to the state.
// grid (ceil(tiles / P5_TILES), BH), 256 threads, one CTA per SM.
static constexpr int P5_TILES = 4;
template <int D, int MF>
struct Prep5Smem {
    static constexpr int BIMG = MF * D * 2;                    // one term of Omega^T [p][a], per 64-wide a block [MF][128 B]
    static constexpr int AIMG = 128 * D * 2;                   // k tile [tok][a], per 64-wide a block [128][128 B]; later the v tile
    static constexpr int LC = MF + 4;                          // chi' row stride in floats
    static constexpr int OFF_B = 0, OFF_A = 3 * BIMG, OFF_CHI = OFF_A + AIMG, OFF_N = OFF_CHI + 128 * LC * 4;
    static constexpr int TOTAL = OFF_N + 128 * 4;
};

template <int D, int MF>
__global__ void __launch_bounds__(256, 1)
k_prep_tc5(const bf16 *__restrict__ k, const bf16 *__restrict__ v, const float *__restrict__ omega, long omega_stride, int m_real,
           int omega_ld, int H, int T, int NC, uint8_t *__restrict__ chi_ml, uint8_t *__restrict__ images,
           float *__restrict__ chi32, const int *__restrict__ seq_lens, int *__restrict__ status)
{
    using G = TcGeom<D, MF>;
    using S = Prep5Smem<D, MF>;
    constexpr int LC = S::LC;
    extern __shared__ __align__(1024) uint8_t smem_dyn[];
    uint8_t *smem = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
    __shared__ uint64_t bar_mma;
    __shared__ uint32_t tmem_base_s;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.y;
    const long seq_off = (long)bh * T * D;
    const float *om = omega + (long)(bh % H) * omega_stride;
    const int Tl = seq_lens ? min(T, max(0, seq_lens[bh / H])) : T;      // padded batches: no key feature beyond the length
    if (warp == 0) {
        tmem_alloc(&tmem_base_s, 128);
        tmem_relinquish();
    }
    if (tid == 0) {
        mbar_init(&bar_mma, 1);
        fence_barrier_init();
    }
    // Omega [a][p] -> Omega^T [p][a] in three bf16 terms (features beyond m_real: zero rows)
    for (int idx = tid; idx < D * MF; idx += 256) {
        const int a = idx / MF, p = idx % MF;                    // coalesced read along p
        const float w = (p < m_real) ? om[(long)a * omega_ld + p] : 0.f;
        const bf16 h0 = __float2bfloat16_rn(w);
        const float r1 = w - __bfloat162float(h0);
        const bf16 h1 = __float2bfloat16_rn(r1);
        const bf16 h2 = __float2bfloat16_rn(r1 - __bfloat162float(h1));
        const uint32_t off = (a >> 6) * (MF * 128) + sw_off<128>(p, (a & 63) >> 3) + (a & 7) * 2;
        *(bf16 *)(smem + S::OFF_B + off) = h0;
        *(bf16 *)(smem + S::OFF_B + S::BIMG + off) = h1;
        *(bf16 *)(smem + S::OFF_B + 2 * S::BIMG + off) = h2;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = tmem_base_s;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t idesc = make_idesc_f16(128, MF, 1, 0, 0);
    float *chi = (float *)(smem + S::OFF_CHI);
    float *nrm = (float *)(smem + S::OFF_N);
    const int n_tiles = (NC * TC_C + 127) / 128;
    constexpr int KPT = 128 * (D / 8) / 256;                     // 16-byte pieces of a [128][D] bf16 tile per thread
    uint32_t phase = 0;
    for (int tile = blockIdx.x * P5_TILES; tile < min(n_tiles, (int)(blockIdx.x + 1) * P5_TILES); ++tile) {
        const int tok0 = tile * 128;
        // the next tile's rows are read with plain loads: have them in L2 by then
        if (tid == 0 && tile + 1 < min(n_tiles, (int)(blockIdx.x + 1) * P5_TILES) && tok0 + 128 < T) {
            const int rows_n = min(128, T - tok0 - 128);
            bulk_prefetch_l2(k + seq_off + (long)(tok0 + 128) * D, rows_n * D * 2);
            bulk_prefetch_l2(v + seq_off + (long)(tok0 + 128) * D, rows_n * D * 2);
        }
        // k rows -> operand image (as they are) and |k|^2 per row
        uint4 kreg[KPT];
#pragma unroll
        for (int y = 0; y < KPT; ++y) {
            const int idx = tid + 256 * y, row = idx / (D / 8), c = idx % (D / 8);
            kreg[y] = make_uint4(0, 0, 0, 0);
            if (tok0 + row < T) kreg[y] = *(const uint4 *)(k + seq_off + (long)(tok0 + row) * D + c * 8);
        }
#pragma unroll
        for (int y = 0; y < KPT; ++y) {
            const int idx = tid + 256 * y, row = idx / (D / 8), c = idx % (D / 8);
            *(uint4 *)(smem + S::OFF_A + (c >> 3) * (128 * 128) + sw_off<128>(row, c & 7)) = kreg[y];
            const uint32_t w4[4] = {kreg[y].x, kreg[y].y, kreg[y].z, kreg[y].w};
            float s2 = 0.f;
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const float lo = __uint_as_float(w4[x] << 16), hi = __uint_as_float(w4[x] & 0xffff0000u);
                s2 = fmaf(lo, lo, fmaf(hi, hi, s2));
            }
#pragma unroll
            for (int o_ = (D / 8) / 2; o_ > 0; o_ >>= 1) s2 += __shfl_xor_sync(0xffffffffu, s2, o_);
            if (c == 0) nrm[row] = s2;
        }
        fence_proxy_async_smem();
        tc_fence_before();
        __syncthreads();
        if (tid == 0) {
            tc_fence_after();
            const uint64_t da = make_smem_desc(smem_u32(smem + S::OFF_A), 0, 1024, kSw128);
#pragma unroll
            for (int term = 2; term >= 0; --term) {                  // smallest term first
                const uint64_t db = make_smem_desc(smem_u32(smem + S::OFF_B + term * S::BIMG), 0, 1024, kSw128);
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks)
                    mma_f16_ss(tm, desc_adv(da, (ks >> 2) * (128 * 128) + (ks & 3) * 32), desc_adv(db, (ks >> 2) * (MF * 128) + (ks & 3) * 32),
                               idesc, (term < 2) || (ks > 0));
            }
            tc_commit(&bar_mma);
        }
        // the v rows of the tile, while the products run (into registers; the k image is still being read)
        uint4 vreg[KPT];
#pragma unroll
        for (int y = 0; y < KPT; ++y) {
            const int idx = tid + 256 * y, row = idx / (D / 8), c = idx % (D / 8);
            vreg[y] = make_uint4(0, 0, 0, 0);
            if (tok0 + row < T) vreg[y] = *(const uint4 *)(v + seq_off + (long)(tok0 + row) * D + c * 8);
        }
        mbar_wait(&bar_mma, phase, status, 36);
        phase ^= 1;
        tc_fence_after();
        // chi' = exp(l - |k|^2/2): thread = token row, half of the features
        {
            const int row = (warp & 3) * 32 + lane, half = warp >> 2;
            const float hn = 0.5f * nrm[row];
            const bool live = tok0 + row < Tl;
#pragma unroll
            for (int c0 = 0; c0 < MF / 2; c0 += 32) {
                uint32_t lv[32];
                tmem_ld32(tm + lane_off + half * (MF / 2) + c0, lv);
                tmem_ld_wait();
#pragma unroll
                for (int x = 0; x < 32; x += 4) {
                    const int p = half * (MF / 2) + c0 + x;
                    float4 w;
                    w.x = (live && p < m_real) ? expf(__uint_as_float(lv[x]) - hn) : 0.f;
                    w.y = (live && p + 1 < m_real) ? expf(__uint_as_float(lv[x + 1]) - hn) : 0.f;
                    w.z = (live && p + 2 < m_real) ? expf(__uint_as_float(lv[x + 2]) - hn) : 0.f;
                    w.w = (live && p + 3 < m_real) ? expf(__uint_as_float(lv[x + 3]) - hn) : 0.f;
                    *(float4 *)(chi + row * LC + p) = w;
                }
            }
        }
        // the v tile over the k image (its products are done), plain rows
#pragma unroll
        for (int y = 0; y < KPT; ++y) {
            const int idx = tid + 256 * y;
            *(uint4 *)(smem + S::OFF_A + idx * 16) = vreg[y];
        }
        tc_fence_before();
        __syncthreads();
        const int rows = min(128, NC * TC_C - tok0);             // rows of the tile that exist in the chunked buffers
        if (chi32) {
            float4 *dst = (float4 *)(chi32 + ((long)bh * NC * TC_C + tok0) * MF);
            for (int idx = tid; idx < rows * (MF / 4); idx += 256) {
                const int r_ = idx / (MF / 4), p4 = idx % (MF / 4);
                dst[idx] = *(const float4 *)(chi + r_ * LC + p4 * 4);
            }
        }
        // chi' images (three bf16 terms) of the tile's chunks
        for (int idx = tid; idx < rows * (MF / 8); idx += 256) {
            const int r_ = idx / (MF / 8), c8 = idx % (MF / 8);
            const int n = (tok0 + r_) / TC_C, j = (tok0 + r_) % TC_C;
            const int kb = c8 >> 3, ch = c8 & 7;
            __align__(16) bf16 pk[8], pm[8], pl[8];
#pragma unroll
            for (int x = 0; x < 8; ++x) {
                const float w = chi[r_ * LC + c8 * 8 + x];
                pk[x] = __float2bfloat16_rn(w);
                const float r1 = w - __bfloat162float(pk[x]);
                pm[x] = __float2bfloat16_rn(r1);
                pl[x] = __float2bfloat16_rn(r1 - __bfloat162float(pm[x]));
            }
            const uint32_t off = kb * (TC_C * 128) + sw_off<128>(j, ch);
            *(uint4 *)(images + ((long)bh * NC + n) * G::IMG_CHUNK + G::IMG_M + off) = *(const uint4 *)pk;
            uint8_t *ml = chi_ml + ((long)bh * NC + n) * 2 * G::IMG_CHI;
            *(uint4 *)(ml + off) = *(const uint4 *)pm;
            *(uint4 *)(ml + G::IMG_CHI + off) = *(const uint4 *)pl;
        }
        // V^T images of the tile's chunks: row e (padded to 128), 16 tokens = 2 pieces of 8
        {
            const bf16 *vt = (const bf16 *)(smem + S::OFF_A);    // [128 tok][D]
            for (int idx = tid; idx < (rows / TC_C) * 128 * 2; idx += 256) {
                const int cn = idx / 256, e = (idx >> 1) & 127, ch = idx & 1;
                __align__(16) bf16 pk[8];
#pragma unroll
                for (int x = 0; x < 8; ++x) pk[x] = (e < D) ? vt[(cn * TC_C + ch * 8 + x) * D + e] : __float2bfloat16_rn(0.f);
                *(uint4 *)(images + ((long)bh * NC + tok0 / TC_C + cn) * G::IMG_CHUNK + G::IMG_M + G::IMG_CHI + sw_off<32>(e, ch)) =
                    *(const uint4 *)pk;
            }
        }
        __syncthreads();                       // chi', the v tile and |k|^2 are free for the next tile
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base_s, 128);
}

// ------------------------------------------------------------------ pre-pass 2: running state in TMEM + state images
// grid (MF / 64, BH), 256 threads.  A CTA owns one 64-feature block of the state of one (batch, head), all 128
// (padded) channel rows, as an fp32 accumulator in tensor memory, and walks the chunks: per chunk
//   S[e][p] += sum_j V^T[e][j] (chi'_hi + chi'_mid + chi'_lo)[j][p]        three tcgen05 products, K = 16 tokens
// (A = the chunk's V^T operand image, B = the chi' images read MN-major), after the state before the chunk has been
// read from tensor memory, rounded to bf16 and written as the chunk's state operand image (exclusive prefix).  The
// operands arrive through a ring of bulk-copy stages; reading, converting and storing the image of chunk n overlaps
// the products of chunk n.  Threads 0..63 carry the normaliser's prefix of the block's features.
static constexpr int ST_STAGES = 6;
template <int D, int MF>
struct StateSmem {
    static constexpr int VT = 128 * 32, CB = TC_C * 128;       // V^T image; one 64-feature block of a chi' image
    static constexpr int STAGE = VT + 3 * CB;
    static constexpr int OBUF = 128 * 128;                     // one 64-feature block of a state image, as it lies in global memory
    static constexpr int TOTAL = ST_STAGES * STAGE + 2 * OBUF;
};

// The walk over a long sequence is cut into segments (blockIdx.z) so that enough CTAs run: a first launch (TOTALS)
// only accumulates each segment's sum of increments (no state is read back per chunk) into segtot
// [BH][segments][MF/64][128*64 + 64] fp32; the second launch starts every segment from the sums of the segments before it.
static constexpr int kStateSegMax = 8;
static constexpr int kSegTot = 128 * 64 + 64;                  // floats per (unit, segment, feature block)
template <int D, int MF, bool TOTALS>
__global__ void __launch_bounds__(256, 1)
k_state_tc(uint8_t *__restrict__ images, const uint8_t *__restrict__ chi_ml, int NC, float *__restrict__ ab,
           float *__restrict__ S_final, float *__restrict__ z_final, int m_real, const float *__restrict__ S_init,
           const float *__restrict__ z_init, int state_m, int p_off, int *__restrict__ status, int seg_len,
           float *__restrict__ segtot, int n_seg)
{
    using G = TcGeom<D, MF>;
    using SS = StateSmem<D, MF>;
    extern __shared__ __align__(1024) uint8_t smem_dyn[];
    uint8_t *smem = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
    __shared__ uint64_t full[ST_STAGES], bar_mma;
    __shared__ uint32_t tmem_base_s;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int kb = blockIdx.x, bh = blockIdx.y, seg = blockIdx.z;
    const int n_begin = seg * seg_len, n_end = min(NC, n_begin + seg_len);
    const bool last_seg = seg == n_seg - 1;
    float *tot_bh = segtot + ((long)bh * kStateSegMax * (MF / 64) + kb) * kSegTot;     // + s * (MF / 64) * kSegTot per segment
    if (warp == 0) {
        tmem_alloc(&tmem_base_s, 64);
        tmem_relinquish();
    }
    if (tid == 0) {
        for (int x = 0; x < ST_STAGES; ++x) mbar_init(&full[x], 1);
        mbar_init(&bar_mma, 1);
        fence_barrier_init();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = tmem_base_s;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const int e = (warp & 3) * 32 + lane;                       // state row (channel) = TMEM lane
    const int ch = warp >> 2;                                   // this thread's features: [32 ch, 32 ch + 32) of the block
    uint32_t v[32];
#pragma unroll
    for (int x = 0; x < 32; ++x) {
        const int p = kb * 64 + ch * 32 + x;
        float s0 = (!TOTALS && S_init && e < D && p < m_real) ? S_init[((long)bh * state_m + p_off + p) * D + e] : 0.f;
        if (!TOTALS)
            for (int s2 = 0; s2 < seg; ++s2) s0 += tot_bh[(long)s2 * (MF / 64) * kSegTot + e * 64 + ch * 32 + x];
        v[x] = __float_as_uint(s0);
    }
    tmem_st32(tm + lane_off + ch * 32, v);
    tmem_st_wait();
    // (the normaliser sits in warps 4 and 5, away from the thread that issues the copies and the products)
    const int na = tid - 128;
    const bool norm_thread = na >= 0 && na < 64;
    float arun = 0.f;
    if (!TOTALS && norm_thread) {
        if (z_init && kb * 64 + na < m_real) arun = z_init[(long)bh * state_m + p_off + kb * 64 + na];
        for (int s2 = 0; s2 < seg; ++s2) arun += tot_bh[(long)s2 * (MF / 64) * kSegTot + 128 * 64 + na];
    }
    uint8_t *obuf = smem + ST_STAGES * SS::STAGE;
    uint8_t *img_bh = images + (long)bh * NC * G::IMG_CHUNK;
    const uint8_t *ml_bh = chi_ml + (long)bh * NC * 2 * G::IMG_CHI;
    auto load = [&](int n) {                                     // (stages and barrier phases count from the segment's first chunk)
        uint8_t *st = smem + ((n - n_begin) % ST_STAGES) * SS::STAGE;
        uint64_t *bar = &full[(n - n_begin) % ST_STAGES];
        const uint8_t *img = img_bh + (long)n * G::IMG_CHUNK;
        const uint8_t *ml = ml_bh + (long)n * 2 * G::IMG_CHI;
        mbar_arrive_expect_tx(bar, SS::STAGE);
        bulk_g2s(st, img + G::IMG_M + G::IMG_CHI, SS::VT, bar);
        bulk_g2s(st + SS::VT, img + G::IMG_M + kb * SS::CB, SS::CB, bar);
        bulk_g2s(st + SS::VT + SS::CB, ml + kb * SS::CB, SS::CB, bar);
        bulk_g2s(st + SS::VT + 2 * SS::CB, ml + G::IMG_CHI + kb * SS::CB, SS::CB, bar);
    };
    if (tid == 0)
        for (int n = n_begin; n < n_begin + ST_STAGES && n < n_end; ++n) load(n);
    const uint32_t idesc = make_idesc_f16(128, 64, 1, 0, 1);     // bf16; A K-major (V^T rows of 16 tokens), B MN-major
    tc_fence_before();
    __syncthreads();                                             // initial state in tensor memory before the first product
    tc_fence_after();
    uint32_t mma_phase = 0;
    for (int n = n_begin; n < n_end; ++n) {
        const int sidx = (n - n_begin) % ST_STAGES;
        uint8_t *st = smem + sidx * SS::STAGE;
        // the state before chunk n
        if (!TOTALS) {
            tmem_ld32(tm + lane_off + ch * 32, v);
            tmem_ld_wait();
        }
        mbar_wait(&full[sidx], ((n - n_begin) / ST_STAGES) & 1, status, 30);
        // the image buffer about to be rewritten was handed to a bulk store an iteration ago: its reads must be over
        if (!TOTALS && tid == 0) bulk_wait_read<0>();
        tc_fence_before();
        __syncthreads();                       // every thread holds its part of the state; stage n is in shared memory
        if (tid == 0) {
            // the image of the chunk before is complete in shared memory (written before the barrier): one bulk store
            if (!TOTALS && n > n_begin)
                bulk_s2g(img_bh + (long)(n - 1) * G::IMG_CHUNK + kb * SS::OBUF, obuf + ((n - 1 - n_begin) & 1) * SS::OBUF, SS::OBUF);
            tc_fence_after();
            const uint64_t da = make_smem_desc(smem_u32(st), 0, 256, kSw32);
#pragma unroll
            for (int term = 0; term < 3; ++term)
                mma_f16_ss(tm, da, make_smem_desc(smem_u32(st + SS::VT + term * SS::CB), TC_C * 128, 1024, kSw128), idesc, 1);
            tc_commit(&bar_mma);
            // the stage of chunk n - 1 is free: its products have completed (waited for at the end of the iteration
            // before) and its reads for the normaliser lie before the barrier above
            if (n > n_begin && n - 1 + ST_STAGES < n_end) load(n - 1 + ST_STAGES);
        }
        // the chunk's state operand image: row e, features [64 kb + 32 ch, + 32) = four 16-byte pieces
        // (assembled in shared memory in its final layout and stored as one contiguous 16 KB block: a row per thread
        // straight to global memory would be 32 separate lines per store instruction)
        if (!TOTALS) {
            uint8_t *dst = obuf + ((n - n_begin) & 1) * SS::OBUF;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint32_t pk[4];
#pragma unroll
                for (int x = 0; x < 4; ++x) pk[x] = pack_bf16(__uint_as_float(v[i * 8 + 2 * x]), __uint_as_float(v[i * 8 + 2 * x + 1]));
                *(uint4 *)(dst + sw_off<128>(e, ch * 4 + i)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
            fence_proxy_async_smem();
        }
        if (norm_thread) {
            // normaliser: exclusive prefix out, then the chunk's sum of chi' (three bf16 terms) over its 16 tokens
            if (!TOTALS) ab[((long)bh * NC + n) * MF + kb * 64 + na] = arun;
            float acc = 0.f;
#pragma unroll
            for (int j = 0; j < TC_C; ++j) {
                const uint32_t off = sw_off<128>(j, na >> 3) + (na & 7) * 2;
#pragma unroll
                for (int term = 0; term < 3; ++term)
                    acc += __uint_as_float((uint32_t)(*(const uint16_t *)(st + SS::VT + term * SS::CB + off)) << 16);
            }
            arun += acc;
        }
        mbar_wait(&bar_mma, mma_phase, status, 31);
        mma_phase ^= 1;
        tc_fence_after();
    }
    if (!TOTALS) {
        __syncthreads();                       // the last chunk's image is complete in shared memory
        if (tid == 0) {
            if (n_end > n_begin)
                bulk_s2g(img_bh + (long)(n_end - 1) * G::IMG_CHUNK + kb * SS::OBUF, obuf + ((n_end - 1 - n_begin) & 1) * SS::OBUF, SS::OBUF);
            bulk_wait_all<0>();
        }
    }
    if (TOTALS) {
        tmem_ld32(tm + lane_off + ch * 32, v);
        tmem_ld_wait();
        float *dst = tot_bh + (long)seg * (MF / 64) * kSegTot;
#pragma unroll
        for (int x = 0; x < 32; x += 4)
            *(float4 *)(dst + e * 64 + ch * 32 + x) = make_float4(__uint_as_float(v[x]), __uint_as_float(v[x + 1]),
                                                                  __uint_as_float(v[x + 2]), __uint_as_float(v[x + 3]));
        if (norm_thread) dst[128 * 64 + na] = arun;
    } else if (S_final && last_seg && e < D) {
        tmem_ld32(tm + lane_off + ch * 32, v);
        tmem_ld_wait();
#pragma unroll
        for (int x = 0; x < 32; ++x) {
            const int p = kb * 64 + ch * 32 + x;
            if (p < m_real) S_final[((long)bh * state_m + p_off + p) * D + e] = __uint_as_float(v[x]);
        }
    }
    if (!TOTALS && z_final && last_seg && norm_thread && kb * 64 + na < m_real) z_final[(long)bh * state_m + p_off + kb * 64 + na] = arun;
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base_s, 64);
}

// OmegaT image: fp16 [p][a], per 64-wide a-block a [MF][128 B] tile with the 128-byte swizzle.  grid (n_omega).
template <int D, int MF>
__global__ void k_omega_image_tc(const float *__restrict__ omega, int m_real, int omega_ld, long bank_stride,
                                 uint8_t *__restrict__ img)
{
    using G = TcGeom<D, MF>;
    const float *om = omega + (long)blockIdx.x * bank_stride;
    uint8_t *out = img + (long)blockIdx.x * G::IMG_OM;
    for (int idx = threadIdx.x; idx < MF * D / 8; idx += blockDim.x) {
        const int p = idx / (D / 8), c8 = idx - p * (D / 8);
        const int kb = c8 >> 3, ch = c8 & 7;
        __align__(16) __half pk[8];
#pragma unroll
        for (int x = 0; x < 8; ++x) pk[x] = __float2half_rn(p < m_real ? om[(long)(c8 * 8 + x) * omega_ld + p] : 0.f);
        *(uint4 *)(out + kb * (MF * 128) + sw_off<128>(p, ch)) = *(const uint4 *)pk;
    }
}

// ------------------------------------------------------------------ main forward kernel
__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi)
{
    __half2 v = __floats2half2_rn(lo, hi);
    return *(uint32_t *)&v;
}
__device__ __forceinline__ uint32_t bf2h_(uint32_t w)
{
    __half2 h = __floats2half2_rn(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
    return *(uint32_t *)&h;
}
__device__ __forceinline__ float2 unpack_bf16(uint32_t w)
{
    __nv_bfloat162 v = *(__nv_bfloat162 *)&w;
    return __bfloat1622float2(v);
}

template <int D, int MF>
struct FwdTcSmem {
    using G = TcGeom<D, MF>;
    static constexpr int WROWS = 5 * TC_C;                        // anchor window: ring of 5 groups of 16 tokens
    static constexpr int ROWB = D * 2;                            // bytes per token row
    static constexpr int PITCH = ROWB + 16;                       // window row pitch (conflict-free 16-byte row reads)
    static constexpr int OFF_OM = 0;
    static constexpr int OFF_CHUNK0 = OFF_OM + G::IMG_OM;
    static constexpr int OFF_CHUNK1 = OFF_CHUNK0 + G::IMG_CHUNK;
    static constexpr int OFF_PSI = OFF_CHUNK1 + G::IMG_CHUNK;     // per tile slot: [128][MF] bf16
    static constexpr int PSI_BYTES = 128 * MF * 2;
    static constexpr int OFF_PM = OFF_PSI + TC_SLOTS * PSI_BYTES; // per tile slot: [128][16] bf16 (32-byte rows)
    static constexpr int PM_BYTES = 128 * 32;
    static constexpr int OFF_RWIN = OFF_PM + TC_SLOTS * PM_BYTES; // [WROWS][D] fp16, padded rows
    static constexpr int OFF_Q = OFF_RWIN + ((WROWS * PITCH + 1023) / 1024) * 1024;
    static constexpr int OFF_AB = OFF_Q + TC_C * ROWB;            // [MF] fp32
    static constexpr int OFF_HN = OFF_AB + MF * 4;                // per slot: [2 halves][128] fp32 partial |x|^2/2
    static constexpr int OFF_ACC = OFF_HN + TC_SLOTS * 2 * 128 * 4;   // per slot: [2 halves][2 queries][128] fp32 partial N
    static constexpr int OFF_MISC = OFF_ACC + TC_SLOTS * 4 * 128 * 4; // per slot: 8 warp maxima, 8 warp sums, 2 L, 2 den
    static constexpr int TOTAL = OFF_MISC + TC_SLOTS * 128;
};

// grid (ceil(NC / chunks_per_cta), B*H), 512 threads = 2 tile slots x 2 column halves x 128 rows.
// A tile is 128 composite rows = 2 queries x 64 steps back; each slot works through every second tile of the
// chunk, so that the products of one slot run under the CUDA-core phases of the other.  The two threads of a
// row own half of the feature columns each (rows side) and half of the steps back each (channel side).
// MODE 1 (HIST): the segment continues a sequence (anchors of the n_hist tokens before it come from hist_r, hist_u);
// the plain instance carries no trace of it.  MODE 2 (O32): `o` points to an fp32 buffer (the output of one feature
// block, to be combined with the other blocks' in full precision).
template <int D, int MF, int MODE>
__global__ void __launch_bounds__(TC_NT, 1)
k_fwd_tc(const bf16 *__restrict__ q, const bf16 *__restrict__ r, const bf16 *__restrict__ u,
         const uint8_t *__restrict__ om_img, int om_per_head, int H, int T, int W, int NC, int chunks_per_cta,
         float log2_eps_m, const uint8_t *__restrict__ images, const float *__restrict__ ab_g, bf16 *__restrict__ o,
         float *__restrict__ Lout, float *__restrict__ lse, int *__restrict__ status, int m_real,
         const bf16 *__restrict__ hist_r, const bf16 *__restrict__ hist_u, int n_hist_arg)
{
    constexpr bool HIST = MODE == 1, O32 = MODE == 2;
    const int n_hist = HIST ? n_hist_arg : 0;
    using G = TcGeom<D, MF>;
    using S = FwdTcSmem<D, MF>;
    constexpr float LOG2E = 1.4426950408889634f, LN2 = 0.6931471805599453f;
    constexpr int CH = D / 8;                     // 16-byte chunks per token row
    constexpr int XW = D / 4;                     // packed fp16 words of X per thread (half a row)
    constexpr int FH = MF / 2;                    // feature columns per thread
    extern __shared__ __align__(1024) uint8_t smem_dyn[];
    // 1024-byte alignment by an offset into the array (not by pointer casts), so that accesses stay shared-space loads/stores
    uint8_t *smem = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
    __shared__ uint64_t bar_full[2], bar_om, bar_mma[TC_SLOTS][3];
    __shared__ uint32_t tmem_base_s;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int slot = tid >> 8, hf = (tid >> 7) & 1, t = tid & 127;   // t = tile row (rows side) / channel (epilogue)
    const int wis = (warp & 3) + 4 * hf;                             // warp index inside the slot
    const int bh = blockIdx.y;
    const int n_begin = blockIdx.x * chunks_per_cta;
    const int n_end = min(NC, n_begin + chunks_per_cta);
    const long seq_off = (long)bh * T * D;

    if (warp == 0) {
        tmem_alloc(&tmem_base_s, 512);
        tmem_relinquish();
    }
    if (tid == 0) {
        mbar_init(&bar_full[0], 1);
        mbar_init(&bar_full[1], 1);
        mbar_init(&bar_om, 1);
        for (int g = 0; g < TC_SLOTS; ++g)
            for (int x = 0; x < 3; ++x) mbar_init(&bar_mma[g][x], 1);
        fence_barrier_init();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_sl = tmem_base_s + slot * 256;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    constexpr uint32_t TM_X = 0, TM_L = 64, TM_P = 192;     // column offsets inside the slot's region

    const uint8_t *img_bh = images + (long)bh * NC * G::IMG_CHUNK;
    if (tid == 0) {
        mbar_arrive_expect_tx(&bar_om, G::IMG_OM);
        bulk_g2s(smem + S::OFF_OM, om_img + (long)(om_per_head ? bh % H : 0) * G::IMG_OM, G::IMG_OM, &bar_om);
        mbar_arrive_expect_tx(&bar_full[0], G::IMG_CHUNK);
        bulk_g2s(smem + S::OFF_CHUNK0, img_bh + (long)n_begin * G::IMG_CHUNK, G::IMG_CHUNK, &bar_full[0]);
    }
    mbar_wait(&bar_om, 0, status, 10);

    uint8_t *psi_s = smem + S::OFF_PSI + slot * S::PSI_BYTES;
    uint8_t *pm_s = smem + S::OFF_PM + slot * S::PM_BYTES;
    uint8_t *rwin = smem + S::OFF_RWIN;
    uint8_t *qs = smem + S::OFF_Q;
    float *abs_ = (float *)(smem + S::OFF_AB);
    float *hnp = (float *)(smem + S::OFF_HN) + slot * 256;           // [2][128]
    float *accp = (float *)(smem + S::OFF_ACC) + slot * 512;         // [2 halves][2 queries][128]
    float *misc = (float *)(smem + S::OFF_MISC) + slot * 32;         // [0..7] warp max, [8..15] warp sums, [16..17] L, [18..19] den

    const uint32_t idesc_1 = make_idesc_f16(128, MF, 0, 0, 0);        // fp16: X . OmegaT
    const uint32_t idesc_p = make_idesc_f16(128, TC_C, 1, 0, 0);      // bf16: psi . chi'
    const uint32_t idesc_2 = make_idesc_f16(128, 128, 1, 0, 0);       // bf16: MbT . psi, Vt . Pm
    uint32_t mma_phase = 0;                                           // flips once per tile (each barrier used once per tile)
    const bool issuer = (hf == 0) && (t == 0);                        // the slot's product-issuing thread

    for (int n = n_begin; n < n_end; ++n) {
        const int it = n - n_begin, buf = it & 1;
        uint8_t *chunk_s = smem + (buf ? S::OFF_CHUNK1 : S::OFF_CHUNK0);
        if (tid == 0 && n + 1 < n_end) {
            mbar_arrive_expect_tx(&bar_full[buf ^ 1], G::IMG_CHUNK);
            bulk_g2s(smem + (buf ? S::OFF_CHUNK0 : S::OFF_CHUNK1), img_bh + (long)(n + 1) * G::IMG_CHUNK, G::IMG_CHUNK,
                     &bar_full[buf ^ 1]);
            // the next chunk's token rows are read with plain loads at its start: have them in L2 by then
            const int rows = min(TC_C, T - (n + 1) * TC_C);
            bulk_prefetch_l2(r + seq_off + (long)(n + 1) * TC_C * D, rows * D * 2);
            bulk_prefetch_l2(q + seq_off + (long)(n + 1) * TC_C * D, rows * D * 2);
            bulk_prefetch_l2(u + seq_off + (long)(n + 1) * TC_C * D, rows * D * 2);      // (the epilogues read u from global memory)
        }
        // anchor window (a ring of five 16-token groups: group g of the sequence sits in ring slot g mod 5; the
        // chunk needs groups n-4 .. n, of which all but group n are still there), query rows, boundary normaliser
        const int b5 = (n + 1) % 5;                          // ring slot of group n - 4
        auto ring_row = [&](int c) {                         // ring row of token c, c in groups n-4 .. n
            int sl = (c >> 4) - (n - 4) + b5;
            sl -= (sl >= 5) ? 5 : 0;
            return sl * TC_C + (c & 15);
        };
        {
            const int g_lo = (it == 0) ? n - 4 : n;
            const int nitem = (n - g_lo + 1) * TC_C * CH;
            for (int idx = tid; idx < nitem; idx += TC_NT) {
                const int row = idx / CH, ch = idx - row * CH;
                const int tok = g_lo * TC_C + row;
                uint4 val = make_uint4(0, 0, 0, 0);
                if (tok >= 0 && tok < T) val = *(const uint4 *)(r + seq_off + (long)tok * D + ch * 8);
                else if (HIST && tok < 0 && tok >= -n_hist)      // anchors from before the segment
                    val = *(const uint4 *)(hist_r + ((long)bh * n_hist + n_hist + tok) * D + ch * 8);
                // fp16 copies (exact for bf16 values in the fp16 range): X = q * r is then one packed multiply
                *(uint4 *)(rwin + ring_row(tok) * S::PITCH + (ch << 4)) = make_uint4(bf2h_(val.x), bf2h_(val.y), bf2h_(val.z), bf2h_(val.w));
            }
        }
        {
            const int j = (tid + TC_NT / 2) & (TC_NT - 1);   // the other half of the CTA
            if (j < TC_C * CH) {
                const int row = j / CH, ch = j - row * CH;
                const int tok = n * TC_C + row;
                uint4 val = make_uint4(0, 0, 0, 0);
                if (tok < T) val = *(const uint4 *)(q + seq_off + (long)tok * D + ch * 8);
                *(uint4 *)(qs + row * S::ROWB + (ch << 4)) = make_uint4(bf2h_(val.x), bf2h_(val.y), bf2h_(val.z), bf2h_(val.w));
            }
        }
        for (int p = tid; p < MF; p += TC_NT) abs_[p] = ab_g[((long)bh * NC + n) * MF + p];
        mbar_wait(&bar_full[buf], (it >> 1) & 1, status, 11);
        __syncthreads();

        const uint32_t mbt_addr = smem_u32(chunk_s);
        const uint32_t chi_addr = mbt_addr + G::IMG_M;
        const uint32_t vt_addr = chi_addr + G::IMG_CHI;

        for (int tile = slot; tile < TC_C / 2; tile += TC_SLOTS) {
            const int il = tile * 2 + (t >> 6);           // query index inside the chunk
            const int i = n * TC_C + il;                  // query token
            const int s = t & 63;                         // steps back
            const bool valid = (s < W) && (i - s >= -n_hist) && (i < T);
            // ---- X = q_i * r_c (fp16) into TMEM (this thread's half of the row), |x|^2/2 in fp32
            {
                float2 hn2 = make_float2(0.f, 0.f);
                const int wrow = ring_row(i - s);                        // always inside the window
                const uint8_t *rrow = rwin + wrow * S::PITCH;
                const uint8_t *qrow = qs + il * S::ROWB;
                uint32_t xr[XW];
#pragma unroll
                for (int c8 = 0; c8 < CH / 2; ++c8) {
                    const int ch = hf * (CH / 2) + c8;
                    const uint4 rv = *(const uint4 *)(rrow + (ch << 4));
                    const uint4 qv = *(const uint4 *)(qrow + (ch << 4));
                    const uint32_t rw[4] = {rv.x, rv.y, rv.z, rv.w}, qw[4] = {qv.x, qv.y, qv.z, qv.w};
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        const __half2 xv = __hmul2(*(const __half2 *)&rw[x], *(const __half2 *)&qw[x]);
                        const float2 xf = __half22float2(xv);
                        hn2 = ffma2(xf, xf, hn2);
                        xr[c8 * 4 + x] = *(const uint32_t *)&xv;
                    }
                }
                if (XW == 32) tmem_st32(tmem_sl + lane_off + TM_X + hf * XW, (const uint32_t(&)[32])xr);
                else tmem_st16(tmem_sl + lane_off + TM_X + hf * XW, (const uint32_t(&)[16])xr);
                hnp[hf * 128 + t] = 0.5f * (hn2.x + hn2.y);
            }
            tmem_st_wait();
            tc_fence_before();
            bar_sync(1 + slot, 256);
            if (issuer) {
                tc_fence_after();
                const uint64_t dom = make_smem_desc(smem_u32(smem + S::OFF_OM), 0, 1024, kSw128);
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks)
                    mma_f16_ts(tmem_sl + TM_L, tmem_sl + TM_X + ks * 8, desc_adv(dom, (ks >> 2) * (MF * 128) + (ks & 3) * 32), idesc_1,
                               ks > 0);
                tc_commit(&bar_mma[slot][0]);
            }
            const float hn = hnp[t] + hnp[128 + t];
            mbar_wait(&bar_mma[slot][0], mma_phase, status, 12);
            tc_fence_after();
            // ---- max of l = l_raw - |x|^2/2 over this thread's columns, then the query's max over its 64 rows
            // (this thread's FH columns are read once and kept in registers for the exponentials below)
            float mx = -INFINITY;
            uint32_t lv[FH];
#pragma unroll
            for (int c0 = 0; c0 < FH; c0 += 32) tmem_ld32(tmem_sl + lane_off + TM_L + hf * FH + c0, (uint32_t(&)[32])lv[c0]);
            tmem_ld_wait();
            if (m_real == MF) {
#pragma unroll
                for (int x = 0; x < FH; ++x) mx = fmaxf(mx, __uint_as_float(lv[x]));
            } else {                                              // zero-padded features take no part in L_i
#pragma unroll
                for (int x = 0; x < FH; ++x)
                    if (hf * FH + x < m_real) mx = fmaxf(mx, __uint_as_float(lv[x]));
            }
            mx = valid ? mx - hn : -INFINITY;
            mx = warp_max(mx);
            if (lane == 0) misc[wis] = mx;
            bar_sync(1 + slot, 256);
            const int qi = t >> 6;
            float L = fmaxf(fmaxf(misc[2 * qi], misc[2 * qi + 1]), fmaxf(misc[4 + 2 * qi], misc[5 + 2 * qi]));
            if (!(L > -INFINITY)) L = 0.f;                        // query beyond T: nothing valid
            // ---- psi' = exp(l - L) -> bf16 tile in shared memory; zeta = psi' . a_b
            const float shift = valid ? (hn + L) * LOG2E : INFINITY;   // invalid rows: exp2(-inf) = 0
            float2 zeta2 = make_float2(0.f, 0.f);
            const float2 l2e = make_float2(LOG2E, LOG2E), nshift = make_float2(-shift, -shift);
#pragma unroll
            for (int c0 = 0; c0 < FH; c0 += 32) {
                const uint32_t *v = lv + c0;
#pragma unroll
                for (int c8 = 0; c8 < 4; ++c8) {
                    uint32_t pk[4];
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        const int col = hf * FH + c0 + c8 * 8 + x * 2;
                        const float2 arg = ffma2(make_float2(__uint_as_float(v[c8 * 8 + x * 2]), __uint_as_float(v[c8 * 8 + x * 2 + 1])), l2e, nshift);
                        // every fourth pair on the FMA pipes instead of the special-function unit (measured: none 4.93 ms, an eighth 4.89 ms, a quarter
                        // 4.87 ms, half 4.97 ms on the benchmark step)
                        const float2 pp = (x == 3) ? ex2_poly2(arg) : make_float2(ex2_approx(arg.x), ex2_approx(arg.y));
                        zeta2 = ffma2(pp, *(const float2 *)(abs_ + col), zeta2);
                        pk[x] = pack_bf16(pp.x, pp.y);
                    }
                    const int c8g = ((hf * FH + c0) >> 3) + c8;   // 8-feature chunk index over all MF
                    *(uint4 *)(psi_s + (c8g >> 3) * (128 * 128) + sw_off<128>(t, c8g & 7)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                }
            }
            float zeta = zeta2.x + zeta2.y;
            fence_proxy_async_smem();
            tc_fence_before();
            bar_sync(1 + slot, 256);
            if (issuer) {
                tc_fence_after();
                const uint64_t dpsi = make_smem_desc(smem_u32(psi_s), 0, 1024, kSw128);
                const uint64_t dchi = make_smem_desc(chi_addr, 0, 1024, kSw128), dmb = make_smem_desc(mbt_addr, 0, 1024, kSw128);
#pragma unroll
                for (int ks = 0; ks < MF / 16; ++ks)
                    mma_f16_ss(tmem_sl + TM_P, desc_adv(dpsi, (ks >> 2) * (128 * 128) + (ks & 3) * 32),
                               desc_adv(dchi, (ks >> 2) * (TC_C * 128) + (ks & 3) * 32), idesc_p, ks > 0);
                tc_commit(&bar_mma[slot][1]);
#pragma unroll
                for (int ks = 0; ks < MF / 16; ++ks) {
                    const uint32_t koff = (ks >> 2) * (128 * 128) + (ks & 3) * 32;
                    mma_f16_ss(tmem_sl + TM_L, desc_adv(dmb, koff), desc_adv(dpsi, koff), idesc_2, ks > 0);
                }
            }
            // ---- intra-chunk pair weights (this thread's 8 tokens): mask j <= i, add to the normaliser, hand back as bf16
            mbar_wait(&bar_mma[slot][1], mma_phase, status, 13);
            tc_fence_after();
            {
                uint32_t v[8];
                tmem_ld8(tmem_sl + lane_off + TM_P + hf * 8, v);
                tmem_ld_wait();
                uint32_t pk[4];
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    const int j0 = hf * 8 + 2 * x;
                    const float p0 = (j0 <= il) ? __uint_as_float(v[2 * x]) : 0.f;
                    const float p1 = (j0 + 1 <= il) ? __uint_as_float(v[2 * x + 1]) : 0.f;
                    zeta += p0 + p1;
                    pk[x] = pack_bf16(p0, p1);
                }
                *(uint4 *)(pm_s + sw_off<32>(t, hf)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
            zeta = warp_sum(zeta);
            if (lane == 0) misc[8 + wis] = zeta;
            fence_proxy_async_smem();
            tc_fence_before();
            bar_sync(1 + slot, 256);
            if (issuer) {
                tc_fence_after();
                const uint64_t ad = make_smem_desc(vt_addr, 0, 256, kSw32);
                const uint64_t bd = make_smem_desc(smem_u32(pm_s), 0, 256, kSw32);
                mma_f16_ss(tmem_sl + TM_L, ad, bd, idesc_2, 1);
                tc_commit(&bar_mma[slot][2]);
            }
            if (hf == 1 && t < 2) {
                // the query's stabiliser, normaliser and guard: den = Z' + eps*m*exp(-L)
                const float Lq = fmaxf(fmaxf(misc[2 * t], misc[2 * t + 1]), fmaxf(misc[4 + 2 * t], misc[5 + 2 * t]));
                const float Lf = (Lq > -INFINITY) ? Lq : 0.f;
                const float Z = (misc[8 + 2 * t] + misc[9 + 2 * t]) + (misc[12 + 2 * t] + misc[13 + 2 * t]);
                const float den = fmaxf(Z + ex2_approx(log2_eps_m - Lf * LOG2E), 1e-37f);
                misc[16 + t] = Lf;
                misc[18 + t] = den;
            }
            mbar_wait(&bar_mma[slot][2], mma_phase, status, 14);
            tc_fence_after();
            // ---- epilogue: thread = output channel e = t, steps back [32 hf, 32 hf + 32) of both queries
            const int i0 = n * TC_C + tile * 2;
            if (t < D) {
                // The two queries of the tile share their anchors: anchor i0 - s is column s of query 0 and column
                // s + 1 of query 1, so every u_c[e] is loaded once for both.
                const int s0 = 32 * hf;
                const bool interior = (i0 - 63 >= 0) && (i0 + 1 < T);   // every anchor row exists: no clamping
                const bf16 *ubase = u + seq_off + (long)(i0 + 1 - s0) * D + t;
                float acc0 = 0.f, acc1 = 0.f;
                // (rows outside the sequence and its history have psi' = 0: any finite u will do there)
                auto u_at = [&](int tok) {
                    if (HIST && tok < 0 && tok >= -n_hist) return hist_u[((long)bh * n_hist + n_hist + tok) * D + t];
                    return u[seq_off + (long)min(max(tok, 0), T - 1) * D + t];
                };
                uint32_t v0[32], v1[32];
                tmem_ld32(tmem_sl + lane_off + TM_L + s0, v0);
                tmem_ld32(tmem_sl + lane_off + TM_L + 64 + s0, v1);
                tmem_ld_wait();
                if (interior) {
                    float un = __bfloat162float(ubase[0]);
#pragma unroll
                    for (int x = 0; x < 32; ++x) {
                        const float uj = __bfloat162float(ubase[-(x + 1) * D]);
                        acc1 = fmaf(__uint_as_float(v1[x]), un, acc1);
                        acc0 = fmaf(__uint_as_float(v0[x]), uj, acc0);
                        un = uj;
                    }
                } else {
                    float un = __bfloat162float(u_at(i0 + 1 - s0));
#pragma unroll
                    for (int x = 0; x < 32; ++x) {
                        const float uj = __bfloat162float(u_at(i0 - (s0 + x)));
                        acc1 = fmaf(__uint_as_float(v1[x]), un, acc1);
                        acc0 = fmaf(__uint_as_float(v0[x]), uj, acc0);
                        un = uj;
                    }
                }
                accp[(hf * 2 + 0) * 128 + t] = acc0;
                accp[(hf * 2 + 1) * 128 + t] = acc1;
            }
            tc_fence_before();
            bar_sync(1 + slot, 256);                              // partial sums and misc[16..19] visible; L region read
            if (t < D) {
                const int iq = i0 + hf;                           // half hf finishes query hf
                if (iq < T) {
                    const float den = misc[18 + hf];
                    const float oval = (accp[hf * 128 + t] + accp[(2 + hf) * 128 + t]) / den;
                    if (O32) ((float *)o)[seq_off + (long)iq * D + t] = oval;
                    else o[seq_off + (long)iq * D + t] = __float2bfloat16_rn(oval);
                    if (t == 0) {
                        Lout[(long)bh * T + iq] = misc[16 + hf];
                        lse[(long)bh * T + iq] = misc[16 + hf] + LN2 * log2f(den);
                    }
                }
            }
            mma_phase ^= 1;
        }
        __syncthreads();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base_s, 512);
}

// ------------------------------------------------------------------ host side
template <int D, int MF>
static int fwd_tc_impl(const TcArgs &a, cudaStream_t st)
{
    using G = TcGeom<D, MF>;
    using S = FwdTcSmem<D, MF>;
    const int NC = (a.T + TC_C - 1) / TC_C, BH = a.B * a.H;
    LaunchScope sc = {st, 0};
    const int n_om = a.omega_stride ? a.H : 1;
    LS_LAUNCH(sc, "omega_image_tc", k_omega_image_tc<D, MF><<<n_om, 256, 0, st>>>(a.omega, a.m_real, a.omega_ld, a.omega_stride,
                                                                                 a.om_img));
    {
        using S5 = Prep5Smem<D, MF>;
        const int n_tiles = (NC * TC_C + 127) / 128;
        sc.check(cudaFuncSetAttribute(k_prep_tc5<D, MF>, cudaFuncAttributeMaxDynamicSharedMemorySize, S5::TOTAL + 1024));
        LS_LAUNCH(sc, "prep_tc", k_prep_tc5<D, MF><<<dim3((n_tiles + P5_TILES - 1) / P5_TILES, BH), 256, S5::TOTAL + 1024, st>>>(
            (const bf16 *)a.k, (const bf16 *)a.v, a.omega, a.omega_stride, a.m_real, a.omega_ld, a.H, a.T, NC, a.chi_ml, a.images,
            a.chi32, a.seq_lens, a.status));
    }
    using SS = StateSmem<D, MF>;
    // segments of the state walk: as many as fill the two CTA slots of every SM, at most kStateSegMax, none for short
    // sequences
    int n_seg = (2 * sm_count()) / (BH * (MF / 64));
    if (n_seg > kStateSegMax) n_seg = kStateSegMax;
    if (n_seg > NC / 32) n_seg = NC / 32;
    if (n_seg < 1) n_seg = 1;
    const int seg_len = (NC + n_seg - 1) / n_seg;
    n_seg = (NC + seg_len - 1) / seg_len;
    if (n_seg > 1) {
        sc.check(cudaFuncSetAttribute(k_state_tc<D, MF, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SS::TOTAL + 1024));
        LS_LAUNCH(sc, "state_totals_tc", k_state_tc<D, MF, true><<<dim3(MF / 64, BH, n_seg - 1), 256, SS::TOTAL + 1024, st>>>(
            a.images, a.chi_ml, NC, a.ab, nullptr, nullptr, a.m_real, nullptr, nullptr, a.state_m, a.p_off, a.status, seg_len,
            a.segtot, n_seg));
    }
    sc.check(cudaFuncSetAttribute(k_state_tc<D, MF, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SS::TOTAL + 1024));
    LS_LAUNCH(sc, "state_tc", k_state_tc<D, MF, false><<<dim3(MF / 64, BH, n_seg), 256, SS::TOTAL + 1024, st>>>(
        a.images, a.chi_ml, NC, a.ab, a.S_final, a.z_final, a.m_real, a.S_init, a.z_init, a.state_m, a.p_off, a.status, seg_len,
        a.segtot, n_seg));
    if (a.state_only) return sc.result();
    const int smem = S::TOTAL + 1024;
    const int cpc = a.chunks_per_cta;
    auto launch = [&](auto kern) {
        sc.check(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        LS_LAUNCH(sc, "fwd_tc", kern<<<dim3((NC + cpc - 1) / cpc, BH), TC_NT, smem, st>>>(
            (const bf16 *)a.q, (const bf16 *)a.r, (const bf16 *)a.u, a.om_img, a.omega_stride != 0, a.H, a.T, a.W, NC, cpc,
            a.log2_eps_m, a.images, a.ab, a.o32 ? (bf16 *)a.o32 : (bf16 *)a.o, a.L, a.lse, a.status, a.m_real,
            (const bf16 *)a.hist_r, (const bf16 *)a.hist_u, a.n_hist));
    };
    if (a.o32) {
        if (a.n_hist > 0) return -2;
        launch(k_fwd_tc<D, MF, 2>);
    } else if (a.n_hist > 0) {
        launch(k_fwd_tc<D, MF, 1>);
    } else {
        launch(k_fwd_tc<D, MF, 0>);
    }
    return sc.result();
}

int tc_supported(int d, int m) { return (d == 64 || d == 128) && (m == 32 || m == 64 || m == 128); }

size_t tc_image_bytes(int d, int m)
{
    if (d == 64 && m == 64) return TcGeom<64, 64>::IMG_CHUNK;
    if (d == 64 && m == 128) return TcGeom<64, 128>::IMG_CHUNK;
    if (d == 128 && m == 64) return TcGeom<128, 64>::IMG_CHUNK;
    return TcGeom<128, 128>::IMG_CHUNK;
}

int tc_fwd_run(const TcArgs &a, cudaStream_t st)
{
    if (a.d == 64 && a.m == 64) return fwd_tc_impl<64, 64>(a, st);
    if (a.d == 64 && a.m == 128) return fwd_tc_impl<64, 128>(a, st);
    if (a.d == 128 && a.m == 64) return fwd_tc_impl<128, 64>(a, st);
    if (a.d == 128 && a.m == 128) return fwd_tc_impl<128, 128>(a, st);
    return -2;
}

}  // namespace linsimp
