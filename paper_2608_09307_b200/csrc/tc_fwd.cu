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
// reduction.  The kernel is warp-specialised: row warps (composite queries, exponentials, masks), a product warp
// that issues every tensor-core instruction, channel warps (anchor sums, output) and a load warp hand tiles to one
// another through mbarriers, two tiles in flight on two sets of tensor-memory and shared-memory buffers.
#include "common.cuh"
#include "launch.cuh"
#include "tc_common.cuh"
#include "tc_kernels.h"

#include <cuda_fp16.h>

namespace linsimp {
using namespace tc;

static constexpr int TC_C = kTcChunk;       // tokens per chunk

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
static constexpr int ST_STAGES = 6, ST_STAGES_TWO = 4;       // (with the second image to assemble, fewer stages fit two CTAs per SM)
template <int D, int MF, bool TWO>
struct StateSmem {
    static constexpr int VT = 128 * 32, CB = TC_C * 128;       // V^T image; one 64-feature block of a chi' image
    static constexpr int STAGE = VT + 3 * CB;
    static constexpr int OBUF = 128 * 128;                     // one 64-feature block of a state image, as it lies in global memory
    static constexpr int NST = TWO ? ST_STAGES_TWO : ST_STAGES;
    static constexpr int TOTAL = NST * STAGE + (TWO ? 4 : 2) * OBUF;   // two buffers for the image (and two for its rounding remainder)
};

// The walk over a long sequence is cut into segments (blockIdx.z) so that enough CTAs run: a first launch (TOTALS)
// only accumulates each segment's sum of increments (no state is read back per chunk) into segtot
// [BH][segments][MF/64][128*64 + 64] fp32; the second launch starts every segment from the sums of the segments before it.
static constexpr int kStateSegMax = 8;
static constexpr int kSegTot = 128 * 64 + 64;                  // floats per (unit, segment, feature block)
template <int D, int MF, bool TOTALS, bool TWO>
__global__ void __launch_bounds__(256, 1)
k_state_tc(uint8_t *__restrict__ images, const uint8_t *__restrict__ chi_ml, int NC, float *__restrict__ ab,
           float *__restrict__ S_final, float *__restrict__ z_final, int m_real, const float *__restrict__ S_init,
           const float *__restrict__ z_init, int state_m, int p_off, int *__restrict__ status, int seg_len,
           float *__restrict__ segtot, int n_seg, uint8_t *__restrict__ images_lo)
{
    using G = TcGeom<D, MF>;
    using SS = StateSmem<D, MF, TWO>;
    constexpr int NST = SS::NST;
    extern __shared__ __align__(1024) uint8_t smem_dyn[];
    uint8_t *smem = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
    __shared__ uint64_t full[NST], bar_mma;
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
        for (int x = 0; x < NST; ++x) mbar_init(&full[x], 1);
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
    uint8_t *obuf = smem + NST * SS::STAGE;
    uint8_t *img_bh = images + (long)bh * NC * G::IMG_CHUNK;
    // second bf16 term of the state (what the rounding of the image leaves), same layout, for the backward (nullable)
    uint8_t *lo_bh = (!TOTALS && TWO) ? images_lo + (long)bh * NC * G::IMG_M : nullptr;
    const uint8_t *ml_bh = chi_ml + (long)bh * NC * 2 * G::IMG_CHI;
    auto load = [&](int n) {                                     // (stages and barrier phases count from the segment's first chunk)
        uint8_t *st = smem + ((n - n_begin) % NST) * SS::STAGE;
        uint64_t *bar = &full[(n - n_begin) % NST];
        const uint8_t *img = img_bh + (long)n * G::IMG_CHUNK;
        const uint8_t *ml = ml_bh + (long)n * 2 * G::IMG_CHI;
        mbar_arrive_expect_tx(bar, SS::STAGE);
        bulk_g2s(st, img + G::IMG_M + G::IMG_CHI, SS::VT, bar);
        bulk_g2s(st + SS::VT, img + G::IMG_M + kb * SS::CB, SS::CB, bar);
        bulk_g2s(st + SS::VT + SS::CB, ml + kb * SS::CB, SS::CB, bar);
        bulk_g2s(st + SS::VT + 2 * SS::CB, ml + G::IMG_CHI + kb * SS::CB, SS::CB, bar);
    };
    if (tid == 0)
        for (int n = n_begin; n < n_begin + NST && n < n_end; ++n) load(n);
    const uint32_t idesc = make_idesc_f16(128, 64, 1, 0, 1);     // bf16; A K-major (V^T rows of 16 tokens), B MN-major
    tc_fence_before();
    __syncthreads();                                             // initial state in tensor memory before the first product
    tc_fence_after();
    uint32_t mma_phase = 0;
    for (int n = n_begin; n < n_end; ++n) {
        const int sidx = (n - n_begin) % NST;
        uint8_t *st = smem + sidx * SS::STAGE;
        // the state before chunk n
        if (!TOTALS) {
            tmem_ld32(tm + lane_off + ch * 32, v);
            tmem_ld_wait();
        }
        mbar_wait(&full[sidx], ((n - n_begin) / NST) & 1, status, 30);
        // the image buffer about to be rewritten was handed to a bulk store an iteration ago: its reads must be over
        if (!TOTALS && tid == 0) bulk_wait_read<0>();
        tc_fence_before();
        __syncthreads();                       // every thread holds its part of the state; stage n is in shared memory
        if (tid == 0) {
            // the image of the chunk before is complete in shared memory (written before the barrier): one bulk store
            if (!TOTALS && n > n_begin) {
                bulk_s2g(img_bh + (long)(n - 1) * G::IMG_CHUNK + kb * SS::OBUF, obuf + ((n - 1 - n_begin) & 1) * SS::OBUF, SS::OBUF);
                if (TWO && !TOTALS)
                    bulk_s2g(lo_bh + (long)(n - 1) * G::IMG_M + kb * SS::OBUF, obuf + (2 + ((n - 1 - n_begin) & 1)) * SS::OBUF, SS::OBUF);
            }
            tc_fence_after();
            const uint64_t da = make_smem_desc(smem_u32(st), 0, 256, kSw32);
#pragma unroll
            for (int term = 0; term < 3; ++term)
                mma_f16_ss(tm, da, make_smem_desc(smem_u32(st + SS::VT + term * SS::CB), TC_C * 128, 1024, kSw128), idesc, 1);
            tc_commit(&bar_mma);
            // the stage of chunk n - 1 is free: its products have completed (waited for at the end of the iteration
            // before) and its reads for the normaliser lie before the barrier above
            if (n > n_begin && n - 1 + NST < n_end) load(n - 1 + NST);
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
                if (TWO && !TOTALS) {
                    uint32_t pl[4];
#pragma unroll
                    for (int x = 0; x < 4; ++x)
                        pl[x] = pack_bf16(__uint_as_float(v[i * 8 + 2 * x]) - __uint_as_float(pk[x] << 16),
                                          __uint_as_float(v[i * 8 + 2 * x + 1]) - __uint_as_float(pk[x] & 0xffff0000u));
                    *(uint4 *)(dst + 2 * SS::OBUF + sw_off<128>(e, ch * 4 + i)) = make_uint4(pl[0], pl[1], pl[2], pl[3]);
                }
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
            if (n_end > n_begin) {
                bulk_s2g(img_bh + (long)(n_end - 1) * G::IMG_CHUNK + kb * SS::OBUF, obuf + ((n_end - 1 - n_begin) & 1) * SS::OBUF, SS::OBUF);
                if (TWO && !TOTALS)
                    bulk_s2g(lo_bh + (long)(n_end - 1) * G::IMG_M + kb * SS::OBUF, obuf + (2 + ((n_end - 1 - n_begin) & 1)) * SS::OBUF, SS::OBUF);
            }
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

// ---- shared-memory map of the main kernel
template <int D, int MF>
struct FwdWsSmem {
    using G = TcGeom<D, MF>;
    static constexpr int RING = 6 * TC_C;                         // anchor rows r: ring of 6 groups of 16 tokens
    static constexpr int ROWB = D * 2;                            // bytes per token row
    static constexpr int OFF_OM = 0;
    static constexpr int OFF_IMG = OFF_OM + G::IMG_OM;            // two chunk images
    static constexpr int OFF_PSI = OFF_IMG + 2 * G::IMG_CHUNK;    // per tile buffer: [128][MF] bf16
    static constexpr int PSI_BYTES = 128 * MF * 2;
    static constexpr int OFF_PM = OFF_PSI + 2 * PSI_BYTES;        // per tile buffer: [128][16] bf16 (32-byte rows)
    static constexpr int PM_BYTES = 128 * 32;
    static constexpr int OFF_RWIN = OFF_PM + 2 * PM_BYTES;        // [RING][D] fp16, 16-byte pieces swizzled by row
    static constexpr int OFF_Q = OFF_RWIN + RING * ROWB;          // two chunks of [16][D] fp16
    static constexpr int OFF_AB = OFF_Q + 2 * TC_C * ROWB;        // two chunks of [MF] fp32
    static constexpr int OFF_HN = OFF_AB + 2 * MF * 4;            // per tile buffer: [2 tiles][2 halves][128] fp32 partial |x|^2/2
    static constexpr int OFF_MISC = OFF_HN + 2 * 2 * 2 * 128 * 4; // per tile buffer 32 floats, see below
    static constexpr int TOTAL = OFF_MISC + 2 * 32 * 4;
};

// TMEM column map of the main kernel (512 allocated): per tile buffer the composite queries X (fp16 pairs, the A operand
// of the first product), the 128-column accumulator that holds l and then Dt, the intra-chunk pair weights P; and the
// channel warps' private window of u (bf16 pairs, written twice 40 columns apart so that any 33 consecutive pairs are
// contiguous).
static constexpr uint32_t WS_X = 0, WS_L = 128, WS_P = 384, WS_U = 416;
// Settings of the row warps (each the better of the alternatives that were timed on the main workload).
static constexpr bool WS_X_EARLY = false;      // the next tile's X before the mask (true) or after it (false)
static constexpr int WS_MAX_COLS = 16;         // columns requested per wait in the maximum pass
static constexpr int WS_RS = 2;                // threads per tile row in the row warps (1 or 2)
static constexpr int WS_GW = 4 * WS_RS;        // warps of one row group
static constexpr int WS_CW0 = 2 * WS_GW;       // first channel warp; then the product warp and the load warp
static constexpr int WS_NT = (WS_CW0 + 8) * 32;   // (the last warpgroup: product warp, load warp, two idle warps)

// Bounded wait that also ends when another role of the CTA has already given up (`*abort` set): after one wait of the
// pipeline has run out, every other wait returns at once and the kernel runs to its end with undefined results.
__device__ __forceinline__ void ws_wait(uint64_t *bar, uint32_t parity, int *status, int code, volatile int *abort)
{
    for (uint32_t i = 0; i < kWaitLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return;
        if ((i & 255u) == 255u && *abort) return;
    }
    *abort = 1;
    if (status) atomicExch(status, code);
}
__device__ __forceinline__ void tmem_ld1(uint32_t taddr, uint32_t &r)
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(r) : "r"(taddr) : "memory");
}

// grid (ceil(NC / chunks_per_cta), B*H), WS_NT threads in five roles that hand tiles to one another through mbarriers.
// A tile is 128 composite rows = 2 queries x 64 steps back; tiles alternate between two sets of buffers, so that the
// products of one tile run under the CUDA-core stages of its neighbours:
//   row warps (two groups of eight, one group per buffer; two threads per tile row, half of the columns each):
//       X = q_i * r_c (fp16) into tensor memory, row maximum L_i, psi' = exp(l - L_i) as a bf16 operand tile with the
//       row's part of the normaliser, causal mask of the intra-chunk pair weights; the next tile's X is formed while
//       the pair weights of the current one are being computed;
//   product warp (one thread): l = X . OmegaT;  P = psi' . chi'^T;  Dt = MbT . psi'^T + Vt . Pm^T  (transposed, so that a
//       channel owns a tensor-memory lane);
//   channel warps (thread = output channel e): N_i[e] = sum_c Dt[e,(i,c)] u_c[e] with u from a private window in
//       tensor memory, normaliser and guard, output;
//   load warp: chunk operand images by bulk copy, the chunk's r and q rows (converted to fp16) and boundary normaliser.
// MODE 1 (HIST): the segment continues a sequence (anchors of the n_hist tokens before it come from hist_r, hist_u).
// MODE 2 (O32): `o` points to an fp32 buffer (the output of one feature block, to be combined with the other blocks').
template <int D, int MF, int MODE>
__global__ void __launch_bounds__(WS_NT, 1)
k_fwd_tc(const bf16 *__restrict__ q, const bf16 *__restrict__ r, const bf16 *__restrict__ u,
         const uint8_t *__restrict__ om_img, int om_per_head, int H, int T, int W, int NC, int chunks_per_cta,
         float log2_eps_m, const uint8_t *__restrict__ images, const float *__restrict__ ab_g, bf16 *__restrict__ o,
         float *__restrict__ Lout, float *__restrict__ lse, int *__restrict__ status, int m_real,
         const bf16 *__restrict__ hist_r, const bf16 *__restrict__ hist_u, int n_hist_arg)
{
    constexpr bool HIST = MODE == 1, O32 = MODE == 2;
    const int n_hist = HIST ? n_hist_arg : 0;
    using G = TcGeom<D, MF>;
    using S = FwdWsSmem<D, MF>;
    constexpr float LOG2E = 1.4426950408889634f, LN2 = 0.6931471805599453f;
    constexpr int CH = D / 8;                     // 16-byte pieces per token row
    constexpr int XW = D / 2;                     // packed fp16 words of X per row
    constexpr int NT = TC_C / 2;                  // tiles per chunk
    extern __shared__ __align__(1024) uint8_t smem_dyn[];
    // 1024-byte alignment by an offset into the array (not by pointer casts), so that accesses stay shared-space loads/stores
    uint8_t *smem = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
    // per tile buffer: X written, l ready, psi' written, P ready, Pm written, Dt ready, accumulator read by the channels
    __shared__ uint64_t bar_x[2], bar_l[2], bar_psi[2], bar_p[2], bar_pm[2], bar_dt[2], bar_free[2];
    // per chunk parity: image arrived, image no longer read, rows (r, q, a_b) written, rows no longer read
    __shared__ uint64_t bar_img[2], bar_imgfree[2], bar_rows[2], bar_rowsfree[2], bar_om;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.y;
    const int n_begin = blockIdx.x * chunks_per_cta;
    const int n_end = min(NC, n_begin + chunks_per_cta);
    const long seq_off = (long)bh * T * D;

    if (warp == WS_CW0 + 4) {
        tmem_alloc(&tmem_base_s, 512);
        tmem_relinquish();
    }
    if (tid == 0) {
        for (int b = 0; b < 2; ++b) {
            mbar_init(&bar_x[b], WS_GW);
            mbar_init(&bar_l[b], 1);
            mbar_init(&bar_psi[b], WS_GW);
            mbar_init(&bar_p[b], 1);
            mbar_init(&bar_pm[b], WS_GW);
            mbar_init(&bar_dt[b], 1);
            mbar_init(&bar_free[b], 4);
            mbar_init(&bar_img[b], 1);
            mbar_init(&bar_imgfree[b], 1);
            mbar_init(&bar_rows[b], 1);
            mbar_init(&bar_rowsfree[b], 2 * WS_GW);
        }
        mbar_init(&bar_om, 1);
        abort_s = 0;
        fence_barrier_init();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = tmem_base_s;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    volatile int *abort = &abort_s;

    uint8_t *rwin = smem + S::OFF_RWIN;
    float *misc_all = (float *)(smem + S::OFF_MISC);       // per buffer: [0..15] warp maxima (two sets), [16..23] warp sums, [24..25] L_i
    const uint8_t *img_bh = images + (long)bh * NC * G::IMG_CHUNK;
    // ring row of token `tok` (tok >= -96): the window of a chunk spans five groups, the sixth takes the next chunk's rows
    auto ring_row = [](int tok) { return (tok + S::RING) % S::RING; };

    if (warp < WS_CW0) {
        // ================================================================== row warps
        const int b = warp / WS_GW;                        // tile buffer of this group
        const int w8 = warp % WS_GW;                       // warp inside the group
        const int row = (w8 & 3) * 32 + lane;              // tile row = TMEM lane
        const int hf = w8 >> 2;                            // which half of the row's columns
        const int qi = row >> 6, s = row & 63;             // query of the tile, steps back
        constexpr int FH = MF / WS_RS;                     // feature columns per thread
        constexpr int XH = XW / WS_RS;                     // packed words of X per thread
        float *misc = misc_all + b * 32;
        float *hnp = (float *)(smem + S::OFF_HN) + b * 512;             // [2 tiles][2 halves][128]
        uint8_t *psi_s = smem + S::OFF_PSI + b * S::PSI_BYTES;
        uint8_t *pm_s = smem + S::OFF_PM + b * S::PM_BYTES;
        // X = q_i * r_c (fp16) of tile `tile` of chunk n into tensor memory (this thread's half of the row), its part of
        // |x|^2/2 into shared memory
        auto make_x = [&](int n, int tile, uint32_t kk) {
            const int c = n - n_begin;
            const uint8_t *qs = smem + S::OFF_Q + (c & 1) * (TC_C * S::ROWB);
            const int il = tile * 2 + qi;
            const int rr = ring_row(n * TC_C + il - s);
            const uint8_t *rrow = rwin + rr * S::ROWB;
            const uint8_t *qrow = qs + il * S::ROWB;
            float2 hn2 = make_float2(0.f, 0.f), hn3 = make_float2(0.f, 0.f);
#pragma unroll
            for (int x16 = 0; x16 < XH / 16; ++x16) {
                uint32_t xr[16];
#pragma unroll
                for (int c8 = 0; c8 < 4; ++c8) {
                    const int ch = hf * (XH / 4) + x16 * 4 + c8;
                    const uint4 rv = *(const uint4 *)(rrow + ((ch ^ (rr & 7)) << 4));
                    const uint4 qv = *(const uint4 *)(qrow + (ch << 4));
                    const uint32_t rw[4] = {rv.x, rv.y, rv.z, rv.w}, qw[4] = {qv.x, qv.y, qv.z, qv.w};
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        const __half2 xv = __hmul2(*(const __half2 *)&rw[x], *(const __half2 *)&qw[x]);
                        const float2 xf = __half22float2(xv);
                        if (x & 1) hn3 = ffma2(xf, xf, hn3);
                        else hn2 = ffma2(xf, xf, hn2);
                        xr[c8 * 4 + x] = *(const uint32_t *)&xv;
                    }
                }
                tmem_st16(tm + lane_off + WS_X + b * 64 + hf * XH + x16 * 16, xr);
            }
            hn2 = fadd2(hn2, hn3);
            hnp[((kk & 1) * 2 + hf) * 128 + row] = 0.5f * (hn2.x + hn2.y);
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_x[b]);
        };
        uint32_t k = 0;                                    // tiles this group has worked on
        ws_wait(&bar_rows[0], 0, status, 10, abort);
        if (n_begin < n_end) make_x(n_begin, b, 0);
        for (int n = n_begin; n < n_end; ++n) {
            const int c = n - n_begin;
            const float *abs_ = (const float *)(smem + S::OFF_AB) + (c & 1) * MF;
            for (int tile = b; tile < NT; tile += 2, ++k) {
                const int il = tile * 2 + qi;              // query index inside the chunk
                const int i = n * TC_C + il;               // query token
                const bool valid = (s < W) && (i - s >= -n_hist) && (i < T);
                ws_wait(&bar_l[b], k & 1, status, 12, abort);
                tc_fence_after();
                const float hn = hnp[((k & 1) * 2) * 128 + row] + (WS_RS == 2 ? hnp[((k & 1) * 2 + 1) * 128 + row] : 0.f);
                // ---- maximum of l = l_raw - |x|^2/2 over this thread's columns, then the query's over its 64 rows (four warps)
                float mx = -INFINITY;
                {
                    // (all of this thread's columns are requested before the one wait: a tensor-memory round trip per
                    // piece would dominate the pass)
                    constexpr int PW = FH > WS_MAX_COLS ? WS_MAX_COLS : FH;  // columns per batch of loads
                    float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int c0 = 0; c0 < FH; c0 += PW) {
                        uint32_t lv[PW];
#pragma unroll
                        for (int c1 = 0; c1 < PW; c1 += 16)
                            tmem_ld16(tm + lane_off + WS_L + b * 128 + hf * FH + c0 + c1, (uint32_t(&)[16])lv[c1]);
                        tmem_ld_wait();
#pragma unroll
                        for (int x = 0; x < PW; ++x)
                            if (m_real == MF || hf * FH + c0 + x < m_real)       // zero-padded features take no part in L_i
                                m4[x & 3] = fmaxf(m4[x & 3], __uint_as_float(lv[x]));
                    }
                    mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
                }
                mx = valid ? mx - hn : -INFINITY;
                mx = warp_max(mx);
                if (lane == 0) misc[(k & 1) * 8 + w8] = mx;
                bar_sync(1 + b * 2 + qi, 64 * WS_RS);
                const float *mq = misc + (k & 1) * 8 + 2 * qi;
                float L = fmaxf(mq[0], mq[1]);
                if (WS_RS == 2) L = fmaxf(L, fmaxf(mq[4], mq[5]));
                if (!(L > -INFINITY)) L = 0.f;             // nothing valid (query beyond T)
                // the psi' and Pm tiles of this buffer were last read by the products of the tile two before
                if (k > 0) ws_wait(&bar_dt[b], (k - 1) & 1, status, 13, abort);
                // ---- psi' = exp(l - L) -> bf16 operand tile; zeta = psi' . a_b
                const float shift = valid ? (hn + L) * LOG2E : INFINITY;   // invalid rows: exp2(-inf) = 0
                const float2 l2e = make_float2(LOG2E, LOG2E), nshift = make_float2(-shift, -shift);
                float2 zeta2 = make_float2(0.f, 0.f), zeta3 = make_float2(0.f, 0.f);
                {
                    // pieces of 16 columns; at d = 128 the next piece is requested before the current one is worked on
                    // (at d = 64 that brought nothing)
                    uint32_t lv[2][16];
                    constexpr bool WS_EXP_AHEAD = D == 128;
                    if (WS_EXP_AHEAD) tmem_ld16(tm + lane_off + WS_L + b * 128 + hf * FH, lv[0]);
#pragma unroll
                    for (int pc = 0; pc < FH / 16; ++pc) {
                        const int c0 = pc * 16;
                        if (!WS_EXP_AHEAD) tmem_ld16(tm + lane_off + WS_L + b * 128 + hf * FH + c0, lv[0]);
                        tmem_ld_wait();
                        if (WS_EXP_AHEAD && pc + 1 < FH / 16) tmem_ld16(tm + lane_off + WS_L + b * 128 + hf * FH + c0 + 16, lv[(pc + 1) & 1]);
                        const uint32_t *lc = lv[WS_EXP_AHEAD ? (pc & 1) : 0];
#pragma unroll
                        for (int c8 = 0; c8 < 2; ++c8) {
                            uint32_t pk[4];
#pragma unroll
                            for (int x = 0; x < 4; ++x) {
                                const int col = hf * FH + c0 + c8 * 8 + x * 2;
                                const float2 arg = ffma2(make_float2(__uint_as_float(lc[c8 * 8 + x * 2]), __uint_as_float(lc[c8 * 8 + x * 2 + 1])), l2e, nshift);
                                // d = 128: every fourth pair as a polynomial on the FMA pipes, the rest on the special-function
                                // unit; d = 64: all of them there (the polynomial brought nothing at that width)
                                const float2 pp = (x == 3 && D != 64) ? ex2_poly2(arg) : make_float2(ex2_approx(arg.x), ex2_approx(arg.y));
                                if (x & 1) zeta3 = ffma2(pp, *(const float2 *)(abs_ + col), zeta3);
                                else zeta2 = ffma2(pp, *(const float2 *)(abs_ + col), zeta2);
                                pk[x] = pack_bf16(pp.x, pp.y);
                            }
                            const int c8g = ((hf * FH + c0) >> 3) + c8;    // 8-feature piece over all MF
                            *(uint4 *)(psi_s + (c8g >> 3) * (128 * 128) + sw_off<128>(row, c8g & 7)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                        }
                    }
                }
                zeta2 = fadd2(zeta2, zeta3);
                float zeta = zeta2.x + zeta2.y;
                fence_proxy_async_smem();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(&bar_psi[b]);
                    // the last tile of the chunk for this group: its r, q rows and a_b are not read again
                    if (tile + 2 >= NT) mbar_arrive(&bar_rowsfree[c & 1]);
                }
                // ---- the next tile's X (either here, while the pair weights of this one are being computed, or after the mask)
                if (WS_X_EARLY) {
                    if (tile + 2 < NT) {
                        make_x(n, tile + 2, k + 1);
                    } else if (n + 1 < n_end) {
                        ws_wait(&bar_rows[(c + 1) & 1], ((c + 1) >> 1) & 1, status, 10, abort);
                        make_x(n + 1, b, k + 1);
                    }
                }
                // ---- intra-chunk pair weights (this thread's 8 tokens): mask j <= i, add to the normaliser, hand back as bf16
                ws_wait(&bar_p[b], k & 1, status, 14, abort);
                tc_fence_after();
                {
                    constexpr int PC = TC_C / WS_RS;       // pair-weight columns per thread
                    uint32_t v[PC];
                    if (PC == 16) tmem_ld16(tm + lane_off + WS_P + b * 16, (uint32_t(&)[16])v);
                    else tmem_ld8(tm + lane_off + WS_P + b * 16 + hf * 8, (uint32_t(&)[8])v);
                    tmem_ld_wait();
#pragma unroll
                    for (int pc = 0; pc < PC / 8; ++pc) {
                        uint32_t pk[4];
#pragma unroll
                        for (int x = 0; x < 4; ++x) {
                            const int j0 = hf * PC + pc * 8 + 2 * x;
                            const float p0 = (j0 <= il) ? __uint_as_float(v[pc * 8 + 2 * x]) : 0.f;
                            const float p1 = (j0 + 1 <= il) ? __uint_as_float(v[pc * 8 + 2 * x + 1]) : 0.f;
                            zeta += p0 + p1;
                            pk[x] = pack_bf16(p0, p1);
                        }
                        *(uint4 *)(pm_s + sw_off<32>(row, hf * (PC / 8) + pc)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    }
                }
                zeta = warp_sum(zeta);
                if (lane == 0) {
                    misc[16 + w8] = zeta;
                    if ((w8 & 5) == 0) misc[24 + qi] = L;    // warps 0 and 2 of the group: queries 0 and 1
                }
                fence_proxy_async_smem();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bar_pm[b]);
                if (!WS_X_EARLY) {
                    if (tile + 2 < NT) {
                        make_x(n, tile + 2, k + 1);
                    } else if (n + 1 < n_end) {
                        ws_wait(&bar_rows[(c + 1) & 1], ((c + 1) >> 1) & 1, status, 10, abort);
                        make_x(n + 1, b, k + 1);
                    }
                }
            }
        }
    } else if (warp < WS_CW0 + 4) {
        // ================================================================== channel warps
        const int e = (warp & 3) * 32 + lane;              // output channel = TMEM lane
        const bool live = e < D;
        auto u_at = [&](int tok) -> uint32_t {             // bf16 bits of u[tok][e]; rows outside the sequence: zero
            if (!live) return 0u;
            if (tok >= 0 && tok < T) return (uint32_t)__bfloat16_as_ushort(u[seq_off + (long)tok * D + e]);
            if (HIST && tok < 0 && tok >= -n_hist) return (uint32_t)__bfloat16_as_ushort(hist_u[((long)bh * n_hist + n_hist + tok) * D + e]);
            return 0u;
        };
        uint32_t upf[8];                                   // the next group's 16 values, packed in token pairs
        auto fetch_group = [&](int grp) {
#pragma unroll
            for (int x = 0; x < 8; ++x) upf[x] = u_at(grp * TC_C + 2 * x) | (u_at(grp * TC_C + 2 * x + 1) << 16);
        };
        auto store_group = [&](int grp) {                  // ring position of group grp: 8 columns, mirrored 40 further
            const uint32_t col = 8u * (uint32_t)((grp + 10) % 5);
            tmem_st8(tm + lane_off + WS_U + col, upf);
            tmem_st8(tm + lane_off + WS_U + 40 + col, upf);
        };
        for (int grp = n_begin - 4; grp < n_begin; ++grp) {
            fetch_group(grp);
            store_group(grp);
        }
        fetch_group(n_begin);
        for (int n = n_begin; n < n_end; ++n) {
            const int c = n - n_begin;
            store_group(n);
            tmem_st_wait();
            if (n + 1 < n_end) fetch_group(n + 1);
            for (int tile = 0; tile < NT; ++tile) {
                const int g = c * NT + tile, b = g & 1;
                const uint32_t k = (uint32_t)g >> 1;
                const int i0 = n * TC_C + tile * 2;
                ws_wait(&bar_dt[b], k & 1, status, 15, abort);
                tc_fence_after();
                const float *misc = misc_all + b * 32;
                const float L0 = misc[24], L1 = misc[25];
                // (warps 0, 1, 4, 5 of the row group hold query 0, warps 2, 3, 6, 7 query 1)
                float Z0 = misc[16] + misc[17], Z1 = misc[18] + misc[19];
                if (WS_RS == 2) {
                    Z0 += misc[20] + misc[21];
                    Z1 += misc[22] + misc[23];
                }
                // the guard of the normaliser: den = Z' + eps*m*exp(-L)
                const float den0 = fmaxf(Z0 + ex2_approx(log2_eps_m - L0 * LOG2E), 1e-37f);
                const float den1 = fmaxf(Z1 + ex2_approx(log2_eps_m - L1 * LOG2E), 1e-37f);
                // Pair j (j = 0..32) of the window holds the anchors (i0 - 2j, i0 - 2j + 1) =: (lo, hi).  Query i0 meets lo at
                // step 2j and hi at step 2j - 1, query i0 + 1 meets lo at step 2j + 1 and hi at step 2j.  Column x of
                // `w0` below is step x - 1 of query i0 (loaded one column early so that (hi, lo) pairs line up).
                float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
                const uint32_t ucol = tm + lane_off + WS_U + 8u * (uint32_t)((n - 4 + 10) % 5) + tile;   // pair i0/2 - 32
                const uint32_t dcol = tm + lane_off + WS_L + b * 128;
#pragma unroll
                for (int hq = 0; hq < 4; ++hq) {
                    // steps 16 hq .. 16 hq + 15 of both queries: pairs j = 8 hq .. 8 hq + 7 = window columns 32 - j
                    uint32_t w0[16], w1[16], uu[8];
                    tmem_ld16(dcol + 16 * hq - 1, w0);
                    tmem_ld16(dcol + 64 + 16 * hq, w1);
                    tmem_ld8(ucol + 32 - 8 * hq - 7, uu);             // columns 32 - (8 hq + 7) .. 32 - 8 hq
                    tmem_ld_wait();
#pragma unroll
                    for (int jj = 0; jj < 8; ++jj) {
                        const uint32_t wd = uu[7 - jj];               // pair j = 8 hq + jj
                        const float2 hl = make_float2(__uint_as_float(wd & 0xffff0000u), __uint_as_float(wd << 16));   // (hi, lo)
                        acc1 = ffma2(make_float2(__uint_as_float(w1[2 * jj]), __uint_as_float(w1[2 * jj + 1])), hl, acc1);
                        if (hq == 0 && jj == 0) acc0.y = fmaf(__uint_as_float(w0[1]), hl.y, acc0.y);   // step -1 does not exist
                        else acc0 = ffma2(make_float2(__uint_as_float(w0[2 * jj]), __uint_as_float(w0[2 * jj + 1])), hl, acc0);
                    }
                }
                {
                    // pair j = 32: its hi anchor is step 63 of query i0
                    uint32_t last, ulast;
                    tmem_ld1(dcol + 63, last);
                    tmem_ld1(ucol, ulast);
                    tmem_ld_wait();
                    acc0.x = fmaf(__uint_as_float(last), __uint_as_float(ulast & 0xffff0000u), acc0.x);
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bar_free[b]);
                if (live) {
                    const float o0 = (acc0.x + acc0.y) / den0, o1 = (acc1.x + acc1.y) / den1;
                    if (i0 < T) {
                        if (O32) ((float *)o)[seq_off + (long)i0 * D + e] = o0;
                        else o[seq_off + (long)i0 * D + e] = __float2bfloat16_rn(o0);
                    }
                    if (i0 + 1 < T) {
                        if (O32) ((float *)o)[seq_off + (long)(i0 + 1) * D + e] = o1;
                        else o[seq_off + (long)(i0 + 1) * D + e] = __float2bfloat16_rn(o1);
                    }
                    if (e == 0) {
                        if (i0 < T) {
                            Lout[(long)bh * T + i0] = L0;
                            lse[(long)bh * T + i0] = L0 + LN2 * log2f(den0);
                        }
                        if (i0 + 1 < T) {
                            Lout[(long)bh * T + i0 + 1] = L1;
                            lse[(long)bh * T + i0 + 1] = L1 + LN2 * log2f(den1);
                        }
                    }
                }
            }
        }
    } else if (warp == WS_CW0 + 4) {
        // ================================================================== product warp
        // The whole warp runs the loop convergently (the descriptors stay warp-uniform); one elected lane issues.
        {
            const uint32_t leader = elect_one();
            ws_wait(&bar_om, 0, status, 16, abort);
            const uint32_t idesc_1 = make_idesc_f16(128, MF, 0, 0, 0);        // fp16: X . OmegaT
            const uint32_t idesc_p = make_idesc_f16(128, TC_C, 1, 0, 0);      // bf16: psi . chi'
            const uint32_t idesc_2 = make_idesc_f16(128, 128, 1, 0, 0);       // bf16: MbT . psi, Vt . Pm
            const uint64_t dom = make_smem_desc(smem_u32(smem + S::OFF_OM), 0, 1024, kSw128);
            const int n_tiles = (n_end - n_begin) * NT;
            int gq[2] = {0, 1};                            // next tile of each buffer
            int step[2] = {0, 0};                          // 0: l, 1: P and the state part of Dt, 2: the intra-chunk part of Dt
            int done_in_chunk[2] = {0, 0};                 // per image buffer: tiles whose last product has been issued
            uint32_t spins = 0;
            while ((gq[0] < n_tiles || gq[1] < n_tiles) && !*abort) {
                bool progress = false;
#pragma unroll
                for (int b = 0; b < 2; ++b) {
                    const int g = gq[b];
                    if (g >= n_tiles) continue;
                    const uint32_t k = (uint32_t)g >> 1;
                    const int c = g / NT;
                    const uint32_t tl = tm + WS_L + b * 128;
                    const uint32_t psi_a = smem_u32(smem + S::OFF_PSI + b * S::PSI_BYTES);
                    const uint32_t img_a = smem_u32(smem + S::OFF_IMG + (c & 1) * G::IMG_CHUNK);
                    if (step[b] == 0) {
                        if (!mbar_test_wait(&bar_x[b], k & 1)) continue;
                        if (k > 0 && !mbar_test_wait(&bar_free[b], (k - 1) & 1)) continue;
                        tc_fence_after();
#pragma unroll
                        for (int ks = 0; ks < D / 16; ++ks)
                            mma_f16_ts_if(leader, tl, tm + WS_X + b * 64 + ks * 8, desc_adv(dom, (ks >> 2) * (MF * 128) + (ks & 3) * 32), idesc_1, ks > 0);
                        tc_commit_if(leader, &bar_l[b]);
                        step[b] = 1;
                        progress = true;
                    } else if (step[b] == 1) {
                        if (!mbar_test_wait(&bar_psi[b], k & 1)) continue;
                        if (!mbar_test_wait(&bar_img[c & 1], (c >> 1) & 1)) continue;
                        tc_fence_after();
                        const uint64_t dpsi = make_smem_desc(psi_a, 0, 1024, kSw128);
                        const uint64_t dmb = make_smem_desc(img_a, 0, 1024, kSw128);
                        const uint64_t dchi = make_smem_desc(img_a + G::IMG_M, 0, 1024, kSw128);
#pragma unroll
                        for (int ks = 0; ks < MF / 16; ++ks)
                            mma_f16_ss_if(leader, tm + WS_P + b * 16, desc_adv(dpsi, (ks >> 2) * (128 * 128) + (ks & 3) * 32),
                                          desc_adv(dchi, (ks >> 2) * (TC_C * 128) + (ks & 3) * 32), idesc_p, ks > 0);
                        tc_commit_if(leader, &bar_p[b]);
#pragma unroll
                        for (int ks = 0; ks < MF / 16; ++ks) {
                            const uint32_t koff = (ks >> 2) * (128 * 128) + (ks & 3) * 32;
                            mma_f16_ss_if(leader, tl, desc_adv(dmb, koff), desc_adv(dpsi, koff), idesc_2, ks > 0);
                        }
                        step[b] = 2;
                        progress = true;
                    } else {
                        if (!mbar_test_wait(&bar_pm[b], k & 1)) continue;
                        tc_fence_after();
                        const uint64_t ad = make_smem_desc(img_a + G::IMG_M + G::IMG_CHI, 0, 256, kSw32);
                        const uint64_t bd = make_smem_desc(smem_u32(smem + S::OFF_PM + b * S::PM_BYTES), 0, 256, kSw32);
                        mma_f16_ss_if(leader, tl, ad, bd, idesc_2, 1);
                        tc_commit_if(leader, &bar_dt[b]);
                        // the chunk's image is free once the last product of its eight tiles has completed
                        if (++done_in_chunk[c & 1] == NT) {
                            done_in_chunk[c & 1] = 0;
                            tc_commit_if(leader, &bar_imgfree[c & 1]);
                        }
                        step[b] = 0;
                        gq[b] = g + 2;
                        progress = true;
                    }
                }
                if (progress) spins = 0;
                else if (++spins > kWaitLimit) {
                    *abort = 1;
                    if (status) atomicExch(status, 17);
                }
            }
        }
    } else if (warp == WS_CW0 + 5) {
        // ================================================================== load warp
        if (lane == 0) {
            mbar_arrive_expect_tx(&bar_om, G::IMG_OM);
            bulk_g2s(smem + S::OFF_OM, om_img + (long)(om_per_head ? bh % H : 0) * G::IMG_OM, G::IMG_OM, &bar_om);
            mbar_arrive_expect_tx(&bar_img[0], G::IMG_CHUNK);
            bulk_g2s(smem + S::OFF_IMG, img_bh + (long)n_begin * G::IMG_CHUNK, G::IMG_CHUNK, &bar_img[0]);
        }
        auto r_piece = [&](int tok, int ch) -> uint4 {      // 8 elements of r[tok] as fp16 (exact for bf16 values in the fp16 range)
            uint4 val = make_uint4(0, 0, 0, 0);
            if (tok >= 0 && tok < T) val = *(const uint4 *)(r + seq_off + (long)tok * D + ch * 8);
            else if (HIST && tok < 0 && tok >= -n_hist) val = *(const uint4 *)(hist_r + ((long)bh * n_hist + n_hist + tok) * D + ch * 8);
            return make_uint4(bf2h_(val.x), bf2h_(val.y), bf2h_(val.z), bf2h_(val.w));
        };
        auto put_r = [&](int tok, int ch, uint4 v) {
            const int rr = ring_row(tok);
            *(uint4 *)(rwin + rr * S::ROWB + ((ch ^ (rr & 7)) << 4)) = v;
        };
        // the window before the first chunk: groups n_begin - 4 .. n_begin - 1
        for (int idx = lane; idx < 4 * TC_C * CH; idx += 32) {
            const int tok = (n_begin - 4) * TC_C + idx / CH, ch = idx % CH;
            put_r(tok, ch, r_piece(tok, ch));
        }
        constexpr int PPL = TC_C * CH / 32;                 // 16-byte pieces of a 16-row group per lane
        for (int n = n_begin; n < n_end; ++n) {
            const int c = n - n_begin;
            // chunk n's rows: r group n, q rows, boundary normaliser (loads first, then the wait for the buffers)
            uint4 rp[PPL];
#pragma unroll
            for (int y = 0; y < PPL; ++y) {
                const int idx = lane + 32 * y, tok = n * TC_C + idx / CH, ch = idx % CH;
                rp[y] = r_piece(tok, ch);
            }
            float abv[MF / 32];
#pragma unroll
            for (int y = 0; y < MF / 32; ++y) abv[y] = ab_g[((long)bh * NC + n) * MF + lane + 32 * y];
            // ring slot of group n held group n - 6, q / a_b buffer c & 1 held chunk n - 2: both last read in chunk n - 2
            if (c >= 2) ws_wait(&bar_rowsfree[c & 1], ((c - 2) >> 1) & 1, status, 18, abort);
#pragma unroll
            for (int y = 0; y < PPL; ++y) {
                const int idx = lane + 32 * y, rowi = idx / CH, ch = idx % CH;
                put_r(n * TC_C + rowi, ch, rp[y]);
            }
#pragma unroll
            for (int y = 0; y < PPL; ++y) {
                const int idx = lane + 32 * y, rowi = idx / CH, ch = idx % CH, tok = n * TC_C + rowi;
                uint4 val = make_uint4(0, 0, 0, 0);
                if (tok < T) val = *(const uint4 *)(q + seq_off + (long)tok * D + ch * 8);
                rp[y] = make_uint4(bf2h_(val.x), bf2h_(val.y), bf2h_(val.z), bf2h_(val.w));
            }
#pragma unroll
            for (int y = 0; y < PPL; ++y) {
                const int idx = lane + 32 * y, rowi = idx / CH, ch = idx % CH;
                *(uint4 *)(smem + S::OFF_Q + (c & 1) * (TC_C * S::ROWB) + rowi * S::ROWB + (ch << 4)) = rp[y];
            }
#pragma unroll
            for (int y = 0; y < MF / 32; ++y) ((float *)(smem + S::OFF_AB))[(c & 1) * MF + lane + 32 * y] = abv[y];
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&bar_rows[c & 1]);
                // the next chunk's image, once the products of the chunk before this one have left its buffer
                if (n + 1 < n_end) {
                    if (c >= 1) ws_wait(&bar_imgfree[(c + 1) & 1], ((c - 1) >> 1) & 1, status, 19, abort);
                    mbar_arrive_expect_tx(&bar_img[(c + 1) & 1], G::IMG_CHUNK);
                    bulk_g2s(smem + S::OFF_IMG + ((c + 1) & 1) * G::IMG_CHUNK, img_bh + (long)(n + 1) * G::IMG_CHUNK, G::IMG_CHUNK,
                             &bar_img[(c + 1) & 1]);
                }
            }
            __syncwarp();
        }
    }
    tc_fence_before();
    __syncthreads();
    __syncwarp();
    if (warp == WS_CW0 + 4) tmem_dealloc(tmem_base_s, 512);
}

// ------------------------------------------------------------------ host side
template <int D, int MF>
static int fwd_tc_impl(const TcArgs &a, cudaStream_t st)
{
    using G = TcGeom<D, MF>;
    using S = FwdWsSmem<D, MF>;
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
    // segments of the state walk: as many as fill the two CTA slots of every SM, at most kStateSegMax, none for short
    // sequences
    int n_seg = (2 * sm_count()) / (BH * (MF / 64));
    if (n_seg > kStateSegMax) n_seg = kStateSegMax;
    if (n_seg > NC / 32) n_seg = NC / 32;
    if (n_seg < 1) n_seg = 1;
    const int seg_len = (NC + n_seg - 1) / n_seg;
    n_seg = (NC + seg_len - 1) / seg_len;
    if (n_seg > 1) {
        using SS = StateSmem<D, MF, false>;
        sc.check(cudaFuncSetAttribute(k_state_tc<D, MF, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SS::TOTAL + 1024));
        LS_LAUNCH(sc, "state_totals_tc", k_state_tc<D, MF, true, false><<<dim3(MF / 64, BH, n_seg - 1), 256, SS::TOTAL + 1024, st>>>(
            a.images, a.chi_ml, NC, a.ab, nullptr, nullptr, a.m_real, nullptr, nullptr, a.state_m, a.p_off, a.status, seg_len,
            a.segtot, n_seg, nullptr));
    }
    auto walk = [&](auto kern, int smem_bytes) {
        sc.check(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes));
        LS_LAUNCH(sc, "state_tc", kern<<<dim3(MF / 64, BH, n_seg), 256, smem_bytes, st>>>(
            a.images, a.chi_ml, NC, a.ab, a.S_final, a.z_final, a.m_real, a.S_init, a.z_init, a.state_m, a.p_off, a.status, seg_len,
            a.segtot, n_seg, a.images_lo));
    };
    if (a.images_lo) walk(k_state_tc<D, MF, false, true>, StateSmem<D, MF, true>::TOTAL + 1024);
    else walk(k_state_tc<D, MF, false, false>, StateSmem<D, MF, false>::TOTAL + 1024);
    if (a.state_only) return sc.result();
    const int smem = S::TOTAL + 1024;
    const int cpc = a.chunks_per_cta;
    auto launch = [&](auto kern) {
        sc.check(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        LS_LAUNCH(sc, "fwd_tc", kern<<<dim3((NC + cpc - 1) / cpc, BH), WS_NT, smem, st>>>(
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
