// Tensor-core (tcgen05 / TMEM) backward of the LinSimp hot path for bf16 I/O, m = 64 or 128.
//
// k_bwd_tc walks consecutive 16-token chunks of one (batch, head); a tile is 128 composite
// rows = 2 queries x 64 anchors and all 16 warps work on the same tile (four threads per row
// resp. per output channel, each owning a quarter of the columns).  Per tile, on tcgen05:
//   l    = X . OmegaT                      psi' = exp(l - L_i)               (recomputed features)
//   P    = psi' . chi'^T  (masked j<=i)    Gt   = MbT . psi'^T + Vt . Pm^T   -> du_c += dN_i * g_ic
//   dP   = dg . V^T       (masked j<=i)    dg   = dN_i * u_c
//   dpsiN = dg . Mb^T + dPm . chi'         (= M_i dg_ic, the numerator's part of dpsi)
//   dZ_i = -(dO_i . o_i)/den_i = -(sum_c psi'_ic . dpsiN_ic)/den_i       (the output is recomputed:
//          dN_i . N_i = sum_c dg_ic . g_ic = sum_c psi'_ic . M_i dg_ic, from the operands the other sums use)
//   dl   = (dpsiN + dZ_i a_i) * psi'       a_i = a_b + sum_{j<=i} chi'_j  (fp32, once per chunk)
//   dxT  = Omega . dl^T                    dx = dxT - (1^T dl) x  -> dq_i, dr_c
// and, accumulated over the chunk in TMEM by one product psi'^T [dg | dPm | S] (S = query selector):
//   G^M_n += psi'^T dg,  dchi'_j(intra, numerator part) += psi'^T dPm,  Psi_i = sum_c psi'_ic ;
//   dv_j(intra) += dg^T Pm.  G^a_n = sum_i dZ_i Psi_i and the dZ part of dchi'_j follow in the chunk epilogue.
// Rows of a tile are placed by anchor residue (row = query*64 + (c mod 64)), so the two
// queries of a tile and all later tiles see the same anchor in the same column: the
// anchor gradients du, dr live in two 64-column TMEM windows and an anchor is flushed to
// memory exactly once, when its column is taken over by a newer anchor.
// k_bwd_kv_tc walks the chunks backwards with the running sum of G^M, G^a and finishes dv and dl^k;
// k_bwd_dk_tc turns dl^k into dk.
#include "common.cuh"
#include "launch.cuh"
#include "tc_common.cuh"
#include "tc_kernels.h"

#include <cuda_fp16.h>

#include <type_traits>

namespace linsimp {
using namespace tc;

static constexpr int BC = kTcChunk;         // 16 tokens per chunk
static constexpr int BNT = 512;
static constexpr int BR = 4;                 // threads per tile row / output channel

__device__ __forceinline__ float bf16_round(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }
__device__ __forceinline__ float rcp_approx(float x)
{
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float ex2a(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pk_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *(uint32_t *)&v;
}
__device__ __forceinline__ uint32_t pk_f16(float lo, float hi)
{
    __half2 v = __floats2half2_rn(lo, hi);
    return *(uint32_t *)&v;
}
// two bf16 -> two fp16 (exact inside the fp16 range)
__device__ __forceinline__ uint32_t bf2h(uint32_t w)
{
    __half2 h = __floats2half2_rn(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
    return *(uint32_t *)&h;
}
__device__ __forceinline__ float2 up_bf16(uint32_t w)
{
    __nv_bfloat162 v = *(__nv_bfloat162 *)&w;
    return __bfloat1622float2(v);
}

template <int D, int MF>
struct BwdTcSmem {
    static constexpr int IMG_M = 128 * MF * 2, IMG_CHI = BC * MF * 2, IMG_VT = 128 * 32;
    static constexpr int IMG_CHUNK = IMG_M + IMG_CHI + IMG_VT;
    static constexpr int IMG_OM = MF * 128 * 2;                 // OmegaT fp16 padded to 128 a-columns (2 blocks)
    static constexpr int WROWS = 5 * BC, ROWB = D * 2;          // anchor windows: rings of 5 groups of 16 tokens
    static constexpr int PITCH = ROWB + 16;                     // window row pitch: conflict-free both for one row
                                                                // per thread (16-byte reads) and one channel per thread
    static constexpr int OFF_OM = 0;
    static constexpr int OFF_CHUNK = OFF_OM + IMG_OM;
    static constexpr int OFF_PSI = OFF_CHUNK + IMG_CHUNK;       // [128][MF (padded to 128)] bf16 -> dl fp16 in place
    static constexpr int OFF_XDG = OFF_PSI + 128 * 128 * 2;     // X fp16 [128][D] -> dg bf16 [128][D (padded to 128)]
    static constexpr int OFF_B3 = OFF_XDG + 128 * 128 * 2;      // third 64-column block behind dg: [128][dPm 16 | selector 16 | -]
    static constexpr int OFF_PM = OFF_B3 + 128 * 128;           // masked P, bf16 [128][16]; after the tile's products
    static constexpr int OFF_DQP = OFF_PM;                      //   the same bytes hold dq partials [4 parts][2 queries][128] fp32
    static constexpr int OFF_RWIN = OFF_PM + 4096;
    static constexpr int WIN_BYTES = WROWS * PITCH;
    static constexpr int OFF_UWIN = OFF_RWIN + WIN_BYTES;
    static constexpr int OFF_Q = OFF_UWIN + WIN_BYTES;          // [16][D] fp16
    static constexpr int OFF_DOH = OFF_Q + BC * ROWB;           // [16][D] bf16: dO as given
    static constexpr int OFF_DNH = OFF_DOH + BC * ROWB;         // [17][D] bf16: dN = dO/den rounded, row 16 = zeros
    static constexpr int OFF_AQ = OFF_DNH + (BC + 1) * ROWB;    // [16][MF] fp32: a_i = a_b + sum_{j<=i} chi'_j
    static constexpr int OFF_ROWS = OFF_AQ + BC * MF * 4;       // hn partial [4][128], -sum dl [128]
    static constexpr int OFF_SC = OFF_ROWS + 5 * 128 * 4;       // 1/den[16], L[16], normaliser guard [16], dZ[16]
    static constexpr int TOTAL = OFF_SC + 256 + 128;            // + the warps' partial sums [16][2]
};

// TMEM column map (512 allocated)
static constexpr uint32_t TB_MAIN = 0, TB_DUW = 128, TB_DRW = 192,
                          TB_GM = 256,                  // 160 columns: G^M [128] | dchi' numerator part [16] | Psi [16]
                          TB_DV = 416, TB_P = 432, TB_DP = 448,
                          TB_AUX = 432;                 // 64 columns over P, dP (dead after the masks): first block of dpsiN

// anchor held by residue x when query i is processed
__device__ __forceinline__ int anchor_of(int i, int x) { return i - ((i - x) & 63); }

// MODE 1 (EXT) and 2 (DOT) serve feature ranks above 128, where the layer's numerator and normaliser are sums over
// several 128-feature blocks and a call sees one block.  dZ_i needs sum_c psi'_ic . dpsiN_ic of all blocks: a first
// pass per block in DOT mode computes only that (the tile pipeline up to dpsiN, no gradients) and adds it to
// delta[bh][i]; the second pass per block in EXT mode takes the total from there and writes fp32 gradients that are
// summed over the blocks.
// MODE 3 (HIST) is the backward of a segment that continues a sequence: the anchors of the n_hist tokens before the
// segment come from hist_r, hist_u, and what the segment's queries contribute to the gradients of those anchors
// leaves through the accumulators dhr_acc, dhu_acc [BH][n_hist][D].
template <int D, int MF, int MODE, bool TWO>
__global__ void __launch_bounds__(BNT, 1)
k_bwd_tc(const bf16 *__restrict__ q, const bf16 *__restrict__ r, const bf16 *__restrict__ u,
         const bf16 *__restrict__ dO, const float *__restrict__ Lin, const float *__restrict__ lse,
         const uint8_t *__restrict__ om_img, int om_per_head, int H, int T, int W, int NC, int chunks_per_cta,
         const uint8_t *__restrict__ images, const float *__restrict__ ab_g, bf16 *__restrict__ dq,
         float *__restrict__ dr_acc, float *__restrict__ du_acc, float *__restrict__ gstates,
         float *__restrict__ dv_intra, float *__restrict__ dchi_intra, int *__restrict__ status,
         const float *__restrict__ delta_ext, int grad32, float *__restrict__ delta_out, const int *__restrict__ seq_lens,
         const bf16 *__restrict__ hist_r, const bf16 *__restrict__ hist_u, int n_hist_arg, float *__restrict__ dhr_acc,
         float *__restrict__ dhu_acc, float log2_eps_m, const uint8_t *__restrict__ images_lo)
{
    constexpr bool EXT = MODE == 1, DOT = MODE == 2, HIST = MODE == 3;
    const int n_hist = HIST ? n_hist_arg : 0;
    using S = BwdTcSmem<D, MF>;
    constexpr int CPT = MF / BR;                      // feature columns per thread in the row passes
    constexpr float LOG2E = 1.4426950408889634f;
    constexpr int CH = D / 8;                         // 16-byte chunks per token row
    extern __shared__ __align__(1024) uint8_t smem_dyn[];
    // 1024-byte alignment by an offset into the array (not by pointer casts), so that accesses stay shared-space loads/stores
    uint8_t *smem = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
    __shared__ uint64_t bar_img, bar_om, bar_mma[10], bar_lo, bar_omr, bar_aux;
    __shared__ uint32_t tmem_base_s;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int h = tid >> 7, t = tid & 127;            // h: column quarter (0..3); t: tile row / output channel
    const int bh = blockIdx.y;
    const int n_begin = blockIdx.x * chunks_per_cta;
    const int n_end = min(NC, n_begin + chunks_per_cta);
    const long seq_off = (long)bh * T * D;
    const long E = (long)MF * D + MF;
    // padded batches: dO of tokens at or beyond the sequence's own length is taken as zero
    const int Tl = seq_lens ? min(T, max(0, seq_lens[bh / H])) : T;

    if (warp == 0) {
        tmem_alloc(&tmem_base_s, 512);
        tmem_relinquish();
    }
    if (tid == 0) {
        mbar_init(&bar_img, 1);
        mbar_init(&bar_om, 1);
        for (int x = 0; x < 10; ++x) mbar_init(&bar_mma[x], 1);
        mbar_init(&bar_lo, 1);
        mbar_init(&bar_omr, 1);
        mbar_init(&bar_aux, 1);
        fence_barrier_init();
    }
    // the padding blocks of the psi tile (MF = 64) and of the dg tile (D = 64) must read as zero
    for (int idx = tid; idx < (2 * 128 * 128 * 2 + 128 * 128) / 16; idx += BNT) ((uint4 *)(smem + S::OFF_PSI))[idx] = make_uint4(0, 0, 0, 0);
    for (int idx = tid; idx < S::ROWB / 4; idx += BNT) ((uint32_t *)(smem + S::OFF_DNH + BC * S::ROWB))[idx] = 0;
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = tmem_base_s;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    // zero the du / dr windows
    {
        uint32_t zz[16];
#pragma unroll
        for (int x = 0; x < 16; ++x) zz[x] = 0;
        tmem_st16(tm + lane_off + TB_DUW + h * 16, zz);
        tmem_st16(tm + lane_off + TB_DRW + h * 16, zz);
        tmem_st_wait();
    }
    const uint8_t *img_bh = images + (long)bh * NC * S::IMG_CHUNK;
    // Second bf16 term of the boundary state (what the image's rounding leaves).  dZ_i sees the output the state
    // operand gives, the keys' own values enter exactly, and the two cancel in the key gradients: the image alone
    // leaves its rounding in dk.  No buffer is free for a second image, so it takes turns with Omega, which is read
    // at the two ends of a tile only: in after the first product, out again after the last product that reads it.
    static_assert(S::IMG_M == S::IMG_OM, "the second state term takes the Omega buffer");
    constexpr bool use_lo = TWO;        // (compile-time: the one-term kernel carries none of this)
    const uint8_t *lo_bh = use_lo ? images_lo + (long)bh * NC * S::IMG_M : nullptr;
    const uint8_t *om_src = om_img + (long)(om_per_head ? bh % H : 0) * S::IMG_OM;
    if (tid == 0) {
        mbar_arrive_expect_tx(&bar_om, S::IMG_OM);
        bulk_g2s(smem + S::OFF_OM, om_img + (long)(om_per_head ? bh % H : 0) * S::IMG_OM, S::IMG_OM, &bar_om);
        mbar_arrive_expect_tx(&bar_img, S::IMG_CHUNK);
        bulk_g2s(smem + S::OFF_CHUNK, img_bh + (long)n_begin * S::IMG_CHUNK, S::IMG_CHUNK, &bar_img);
    }
    mbar_wait(&bar_om, 0, status, 20);

    uint8_t *psi_s = smem + S::OFF_PSI, *xdg_s = smem + S::OFF_XDG;
    uint8_t *pm_s = smem + S::OFF_PM, *b3_s = smem + S::OFF_B3;
    uint8_t *rwin = smem + S::OFF_RWIN, *uwin = smem + S::OFF_UWIN, *qs = smem + S::OFF_Q;
    const bf16 *dOh = (const bf16 *)(smem + S::OFF_DOH);
    uint8_t *dNh = smem + S::OFF_DNH;
    // staging of the chunk's G^M block (MF * D * 4 bytes) over tile buffers that hold no zero padding in this instance
    uint8_t *gm_stage = (MF == 128) ? psi_s : (D == 128 ? xdg_s : psi_s);
    float *aq = (float *)(smem + S::OFF_AQ);          // [16][MF]
    float *hnp = (float *)(smem + S::OFF_ROWS);       // [4][128] the column quarters' parts of |x|^2/2, later of zeta
    float *sdlp = hnp + 512;                          // [128] minus the row sums of dl
    float *sdpart = (float *)(smem + S::OFF_PM);      // [4][128] the column quarters' parts of psi'.dpsiN,
                                                      // over the masked pair weights (no product reads them any more)
    float *dqp = (float *)(smem + S::OFF_DQP);        // [4][2][128]
    float *invs = (float *)(smem + S::OFF_SC);        // [16] 1/den_i
    float *Ls = invs + 16;                            // [16]
    float *epsq = Ls + 16;                            // [16] guard of the normaliser, eps m exp(-L_i)
    float *dzs = epsq + 16;                           // [16] dZ_i of the chunk's queries
    float *dred = dzs + 16;                           // [16 warps][2] partial sums of psi' . dpsiN and of zeta

    const uint32_t om_addr = smem_u32(smem + S::OFF_OM);
    const uint32_t mbt_addr = smem_u32(smem + S::OFF_CHUNK);
    const uint32_t chi_addr = mbt_addr + S::IMG_M;
    const uint32_t vt_addr = chi_addr + S::IMG_CHI;
    const uint32_t psi_addr = smem_u32(psi_s), xdg_addr = smem_u32(xdg_s);
    const uint32_t pm_addr = smem_u32(pm_s), b3_addr = smem_u32(b3_s);

    const uint32_t id_lh = make_idesc_f16(128, MF / 2, 0, 0, 0);   // X . OmegaT            (fp16), half the features
    const uint32_t id_p = make_idesc_f16(128, BC, 1, 0, 0);        // psi . chi'^T
    const uint32_t id_gt = make_idesc_f16(128, 128, 1, 0, 0);      // MbT . psi^T, Vt . Pm^T
    const uint32_t id_dp = make_idesc_f16(128, BC, 1, 0, 1);       // dg . V^T              (B MN-major)
    const uint32_t id_gm = make_idesc_f16(128, 160, 1, 1, 1);      // psi^T [dg | dPm | S]  (both MN-major)
    const uint32_t id_n16 = make_idesc_f16(128, BC, 1, 1, 1);      // dg^T Pm
    const uint32_t id_dlo = make_idesc_f16(128, MF, 1, 0, 1);      // dg . Mb_lo^T, all features
    const uint32_t id_dpsih = make_idesc_f16(128, 64, 1, 0, 1);    // dg . Mb^T, dPm . chi' (B MN-major), 64 features
    const uint32_t id_dxh = make_idesc_f16(128, 64, 0, 1, 0);      // Omega . dl^T          (fp16, A MN-major), one query

    uint32_t phase = 0;                // parity of the per-tile MMA barriers
    int last_query = -1;               // last query this CTA has processed (for the final window flush)

    // Rows of the next chunk, requested during the last tile of the chunk before (their latency would otherwise sit
    // between two chunks): threads 0..255 hold 16 bytes of a new anchor row of r and of u, threads 256..511 16 bytes
    // of a query row and of its dO row with the row's L and lse.
    uint4 pf_a = make_uint4(0, 0, 0, 0), pf_b = pf_a;
    float pf_L = 0.f, pf_lse = 0.f;
    auto prefetch_rows = [&](int nn) {
        pf_a = pf_b = make_uint4(0, 0, 0, 0);
        pf_L = pf_lse = 0.f;
        const int idx = tid & (BNT / 2 - 1);
        if (idx >= BC * CH) return;
        const int row = idx / CH, ch = idx - row * CH;
        const int tok = nn * BC + row;
        if (tok >= T) return;
        const long off = seq_off + (long)tok * D + ch * 8;
        if (tid < BNT / 2) {
            pf_a = *(const uint4 *)(r + off);
            pf_b = *(const uint4 *)(u + off);
        } else {
            pf_a = *(const uint4 *)(q + off);
            if (tok < Tl) pf_b = *(const uint4 *)(dO + off);
            pf_L = Lin[(long)bh * T + tok];
            pf_lse = lse[(long)bh * T + tok];
        }
    };

    for (int n = n_begin; n < n_end; ++n) {
        const int it = n - n_begin;
        // ---- chunk prologue: anchor windows, queries, dN.  The windows are rings of five 16-token groups (group g
        //      of the sequence sits in ring slot g mod 5): the chunk needs groups n-4 .. n, of which all but group n
        //      are still there from the chunk before.
        const int b5 = (n + 1) % 5;                          // ring slot of group n - 4
        auto ring_row = [&](int c) {                         // ring row of token c, c in groups n-4 .. n
            int sl = (c >> 4) - (n - 4) + b5;
            sl -= (sl >= 5) ? 5 : 0;
            return sl * BC + (c & 15);
        };
        if (it == 0) {
            const int nitem = 5 * BC * CH;
            for (int idx = tid; idx < nitem; idx += BNT) {
                const int row = idx / CH, ch = idx - row * CH;
                const int tok = (n - 4) * BC + row;
                uint4 rv = make_uint4(0, 0, 0, 0), uv = rv;
                if (tok >= 0 && tok < T) {
                    rv = *(const uint4 *)(r + seq_off + (long)tok * D + ch * 8);
                    uv = *(const uint4 *)(u + seq_off + (long)tok * D + ch * 8);
                } else if (HIST && tok < 0 && tok >= -n_hist) {      // anchors from before the segment
                    rv = *(const uint4 *)(hist_r + ((long)bh * n_hist + n_hist + tok) * D + ch * 8);
                    uv = *(const uint4 *)(hist_u + ((long)bh * n_hist + n_hist + tok) * D + ch * 8);
                }
                const int rr = ring_row(tok);
                // r is kept as fp16 (exact for bf16 values in the fp16 range): X = q * r is then one packed multiply
                *(uint4 *)(rwin + rr * S::PITCH + (ch << 4)) = make_uint4(bf2h(rv.x), bf2h(rv.y), bf2h(rv.z), bf2h(rv.w));
                *(uint4 *)(uwin + rr * S::PITCH + (ch << 4)) = uv;
            }
            prefetch_rows(n);                 // the query half of the CTA takes its rows from the same registers
        } else if (tid < BC * CH) {
            const int row = tid / CH, ch = tid - row * CH;
            const int rr = ring_row(n * BC + row);
            *(uint4 *)(rwin + rr * S::PITCH + (ch << 4)) = make_uint4(bf2h(pf_a.x), bf2h(pf_a.y), bf2h(pf_a.z), bf2h(pf_a.w));
            *(uint4 *)(uwin + rr * S::PITCH + (ch << 4)) = pf_b;
        }
        {
            // the other half of the CTA: queries (fp16), dO as given and dN_i = dO_i / den_i with
            // den_i = exp(lse_i - L_i), 8 channels per thread.  dZ_i needs the output, which is recomputed.
            const int j = tid - BNT / 2;
            if (j >= 0 && j < BC * CH) {
                const int il = j / CH, ch = j - il * CH;
                const int tok = n * BC + il;
                const uint4 qv = pf_a, gv = pf_b;
                const float Lq = pf_L;
                const float inv = (tok < T) ? ex2a((Lq - pf_lse) * LOG2E) : 0.f;
                *(uint4 *)(qs + il * S::ROWB + (ch << 4)) = make_uint4(bf2h(qv.x), bf2h(qv.y), bf2h(qv.z), bf2h(qv.w));
                *(uint4 *)(smem + S::OFF_DOH + il * S::ROWB + (ch << 4)) = gv;
                const uint32_t gw[4] = {gv.x, gv.y, gv.z, gv.w};
                uint32_t nw[4];
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    const float2 gf = up_bf16(gw[x]);
                    nw[x] = pk_bf16(gf.x * inv, gf.y * inv);
                }
                *(uint4 *)(dNh + il * S::ROWB + (ch << 4)) = make_uint4(nw[0], nw[1], nw[2], nw[3]);
                if (ch == 0) {
                    invs[il] = inv;
                    Ls[il] = Lq;
                    // guard of the normaliser in the units of the sum it joins: the block's shifted sums, or (EXT) the
                    // layer's normaliser taken as 1
                    epsq[il] = ex2a(log2_eps_m - (EXT ? pf_lse : Lq) * LOG2E);
                }
            }
        }
        mbar_wait(&bar_img, it & 1, status, 21);
        // the next chunk's image can only be copied once this chunk's products are done (one buffer): have it in L2 by then
        if (tid == 0 && n + 1 < n_end) bulk_prefetch_l2(img_bh + (long)(n + 1) * S::IMG_CHUNK, S::IMG_CHUNK);
        if (tid < MF) {
            // a_i = a_b + sum_{j <= i} chi'_j over the chunk's tokens, from the chi' operand image (bf16, as the
            // tensor cores use it for the pair weights)
            const int p = tid;
            const uint8_t *cb = smem + S::OFF_CHUNK + S::IMG_M + (p >> 6) * (BC * 128) + (p & 7) * 2;
            float acc = ab_g[((long)bh * NC + n) * MF + p];
#pragma unroll
            for (int j = 0; j < BC; ++j) {
                acc += __uint_as_float((uint32_t)(*(const uint16_t *)(cb + sw_off<128>(j, (p & 63) >> 3))) << 16);
                aq[j * MF + p] = acc;
            }
        }
        // the tile buffers the first tile is about to write were handed to the bulk store of the chunk before
        if (!DOT && tid == 0 && it > 0) bulk_wait_read<0>();
        __syncthreads();

        // ---- phase 1 of tile tl: X = q_i * r_c (fp16, K-major tile), a quarter of a row per thread.  Tile 0 runs it
        //      at the top of the loop, the others under the last product of the tile before (the X tile is free then).
        auto phase1 = [&](int tl) {
            const int il1 = tl * 2 + (t >> 6);
            const int c1 = anchor_of(n * BC + il1, t & 63);
            const uint8_t *rrow = rwin + ring_row(c1) * S::PITCH;
            const uint8_t *qrow = qs + il1 * S::ROWB;
            float2 hn2 = make_float2(0.f, 0.f);
#pragma unroll
            for (int c8 = 0; c8 < CH / BR; ++c8) {
                const int ch = h * (CH / BR) + c8;
                const uint4 rv = *(const uint4 *)(rrow + (ch << 4));
                const uint4 qv = *(const uint4 *)(qrow + (ch << 4));
                const uint32_t rw[4] = {rv.x, rv.y, rv.z, rv.w}, qw[4] = {qv.x, qv.y, qv.z, qv.w};
                uint32_t pk[4];
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    const __half2 xv = __hmul2(*(const __half2 *)&rw[x], *(const __half2 *)&qw[x]);
                    const float2 xf = __half22float2(xv);
                    hn2 = ffma2(xf, xf, hn2);
                    pk[x] = *(const uint32_t *)&xv;
                }
                *(uint4 *)(xdg_s + (ch >> 3) * (128 * 128) + sw_off<128>(t, ch & 7)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
            hnp[h * 128 + t] = 0.5f * (hn2.x + hn2.y);
            fence_proxy_async_smem();
        };

        for (int tile = 0; tile < BC / 2; ++tile) {
            const int il = tile * 2 + (t >> 6);
            const int i = n * BC + il;
            const int slot = t & 63;
            const int c = anchor_of(i, slot);
            const int s = i - c;
            const bool valid = (s < W) && (c >= -n_hist) && (i < T);
            const int wrow = ring_row(c);                 // always inside the window (rows outside [0,T) hold zeros)
            if (tile == 0) {
                phase1(0);
                tc_fence_before();
                __syncthreads();
            }
            if (tile == BC / 2 - 1 && n + 1 < n_end) prefetch_rows(n + 1);
            if (tid == 0) {
                tc_fence_after();
                // one half of the features at a time: the exponentials of the first start under the second
                const uint64_t da = make_smem_desc(xdg_addr, 0, 1024, kSw128), db = make_smem_desc(om_addr, 0, 1024, kSw128);
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks)
                        mma_f16_ss(tm + TB_MAIN + hf * (MF / 2), desc_adv(da, (ks >> 2) * (128 * 128) + (ks & 3) * 32),
                                   desc_adv(db, (ks >> 2) * (MF * 128) + (ks & 3) * 32 + hf * (MF / 2) * 128), id_lh, ks > 0);
                    tc_commit(&bar_mma[hf ? 7 : 0]);
                }
            }
            // ---- phase 2: psi' (bf16 tile), dg = dN_i * u_c (bf16, over the X tile)
            {
                // dg = dN_i * u_c as one bf16 multiply per pair (dN rounded to bf16 once per chunk); rows outside
                // the window multiply by the zero row.  Computed while the first product runs, stored after it.
                uint32_t dgk[CH / BR][4];
                {
                    const uint8_t *urow = uwin + wrow * S::PITCH;
                    const uint8_t *dnrow = dNh + (valid ? il : BC) * S::ROWB;
#pragma unroll
                    for (int c8 = 0; c8 < CH / BR; ++c8) {
                        const int ch = h * (CH / BR) + c8;
                        const uint4 uv = *(const uint4 *)(urow + (ch << 4));
                        const uint4 dv4 = *(const uint4 *)(dnrow + (ch << 4));
                        const uint32_t uw[4] = {uv.x, uv.y, uv.z, uv.w}, dw[4] = {dv4.x, dv4.y, dv4.z, dv4.w};
#pragma unroll
                        for (int x = 0; x < 4; ++x) {
                            const __nv_bfloat162 pr = __hmul2(*(const __nv_bfloat162 *)&uw[x], *(const __nv_bfloat162 *)&dw[x]);
                            dgk[c8][x] = *(const uint32_t *)&pr;
                        }
                    }
                }
                mbar_wait(&bar_mma[0], phase, status, 22);
                tc_fence_after();
                // invalid rows get an infinite shift: exp2(-inf) = 0 without a select per element
                const float shift = valid ? (hnp[t] + hnp[128 + t] + hnp[256 + t] + hnp[384 + t] + Ls[il]) * LOG2E : INFINITY;
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    // this thread's CPT/2 columns of feature half hf
                    if (hf == 1) {
                        mbar_wait(&bar_mma[7], phase, status, 29);
                        tc_fence_after();
                        if (tid == 0 && use_lo) {
                            // the first product has read Omega: the buffer takes the state's second term
                            mbar_arrive_expect_tx(&bar_lo, S::IMG_M);
                            bulk_g2s(smem + S::OFF_OM, lo_bh + (long)n * S::IMG_M, S::IMG_M, &bar_lo);
                        }
                    }
                    uint32_t v[CPT / 2];
                    if (CPT == 32) tmem_ld16(tm + lane_off + TB_MAIN + hf * (MF / 2) + h * (CPT / 2), (uint32_t(&)[16])v);
                    else tmem_ld8(tm + lane_off + TB_MAIN + hf * (MF / 2) + h * (CPT / 2), (uint32_t(&)[8])v);
                    tmem_ld_wait();
#pragma unroll
                    for (int c8 = 0; c8 < CPT / 16; ++c8) {
                        uint32_t pk[4];
#pragma unroll
                        for (int x = 0; x < 4; ++x) {
                            const float2 arg = ffma2(make_float2(__uint_as_float(v[c8 * 8 + 2 * x]), __uint_as_float(v[c8 * 8 + 2 * x + 1])),
                                                     make_float2(LOG2E, LOG2E), make_float2(-shift, -shift));
                            // every second pair on the FMA pipes instead of the special-function unit (the forward: every fourth)
                            const float2 pp = (x & 1) ? ex2_poly2(arg) : make_float2(ex2a(arg.x), ex2a(arg.y));
                            pk[x] = pk_bf16(pp.x, pp.y);
                        }
                        const int cg = hf * (MF / 16) + h * (CPT / 16) + c8;   // 8-feature chunk index over all MF
                        *(uint4 *)(psi_s + (cg >> 3) * (128 * 128) + sw_off<128>(t, cg & 7)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    }
                }
#pragma unroll
                for (int c8 = 0; c8 < CH / BR; ++c8) {
                    const int ch = h * (CH / BR) + c8;
                    *(uint4 *)(xdg_s + (ch >> 3) * (128 * 128) + sw_off<128>(t, ch & 7)) =
                        make_uint4(dgk[c8][0], dgk[c8][1], dgk[c8][2], dgk[c8][3]);
                }
            }
            fence_proxy_async_smem();
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {
                tc_fence_after();
                const uint64_t dpsi = make_smem_desc(psi_addr, 0, 1024, kSw128), dchi = make_smem_desc(chi_addr, 0, 1024, kSw128);
                const uint64_t ddg = make_smem_desc(xdg_addr, 0, 1024, kSw128), dvt = make_smem_desc(vt_addr, 0, 256, kSw32);
                const uint64_t dmb = make_smem_desc(mbt_addr, 0, 1024, kSw128);
                // P = psi . chi'^T
#pragma unroll
                for (int ks = 0; ks < MF / 16; ++ks)
                    mma_f16_ss(tm + TB_P, desc_adv(dpsi, (ks >> 2) * (128 * 128) + (ks & 3) * 32),
                               desc_adv(dchi, (ks >> 2) * (BC * 128) + (ks & 3) * 32), id_p, ks > 0);
                // dP = dg . V^T  (V^T image read MN-major: rows = e, 16 tokens contiguous)
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks)
                    mma_f16_ss(tm + TB_DP, desc_adv(ddg, (ks >> 2) * (128 * 128) + (ks & 3) * 32), desc_adv(dvt, ks * 512), id_dp, ks > 0);
                tc_commit(&bar_mma[1]);
                // Gt = MbT . psi^T
                if (!DOT)
#pragma unroll
                for (int ks = 0; ks < MF / 16; ++ks) {
                    const uint32_t ko = (ks >> 2) * (128 * 128) + (ks & 3) * 32;
                    mma_f16_ss(tm + TB_MAIN, desc_adv(dmb, ko), desc_adv(dpsi, ko), id_gt, ks > 0);
                }
            }
            // ---- phase 3: mask the intra-chunk pair weights and their gradients (4 tokens per thread), selector
            mbar_wait(&bar_mma[1], phase, status, 23);
            tc_fence_after();
            {
                uint32_t v[16], w[16];
                tmem_ld16(tm + lane_off + TB_P, v);
                tmem_ld16(tm + lane_off + TB_DP, w);
                tmem_ld_wait();
                uint32_t pp[2] = {0, 0}, dd[2] = {0, 0};
#pragma unroll
                for (int hh = 0; hh < BR; ++hh)
                    if (h == hh) {
#pragma unroll
                        for (int x = 0; x < 2; ++x) {
                            const int j0 = hh * 4 + 2 * x;
                            const bool m0 = (j0 <= il) && valid, m1 = (j0 + 1 <= il) && valid;
                            pp[x] = pk_bf16(m0 ? __uint_as_float(v[hh * 4 + 2 * x]) : 0.f, m1 ? __uint_as_float(v[hh * 4 + 2 * x + 1]) : 0.f);
                            dd[x] = pk_bf16(m0 ? __uint_as_float(w[hh * 4 + 2 * x]) : 0.f, m1 ? __uint_as_float(w[hh * 4 + 2 * x + 1]) : 0.f);
                        }
                    }
                *(uint2 *)(pm_s + sw_off<32>(t, h >> 1) + (h & 1) * 8) = make_uint2(pp[0], pp[1]);
                *(uint2 *)(b3_s + sw_off<128>(t, h >> 1) + (h & 1) * 8) = make_uint2(dd[0], dd[1]);
                if (h >= 2) {
                    // selector: column 16 + il of this row is one (bf16), so that psi'^T S sums the rows of a query
                    const int jj = il - (h - 2) * 8;                  // position inside this 8-column piece
                    const uint32_t one = (jj & 1) ? 0x3F800000u : 0x00003F80u;
                    const int wsel = (jj >= 0 && jj < 8) ? (jj >> 1) : -1;
                    *(uint4 *)(b3_s + sw_off<128>(t, h)) =
                        make_uint4(wsel == 0 ? one : 0u, wsel == 1 ? one : 0u, wsel == 2 ? one : 0u, wsel == 3 ? one : 0u);
                }
            }
            fence_proxy_async_smem();
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {
                tc_fence_after();
                // Gt += Vt . Pm^T
                if (!DOT) mma_f16_ss(tm + TB_MAIN, make_smem_desc(vt_addr, 0, 256, kSw32), make_smem_desc(pm_addr, 0, 256, kSw32), id_gt, 1);
                tc_commit(&bar_mma[2]);
                // first 64-feature block of dpsiN = dg . Mb^T (MbT image read MN-major) + dPm . chi' (chi' image read
                // MN-major), into the columns the pair weights have left: it runs under the du epilogue
                {
                    const uint64_t ddk = make_smem_desc(xdg_addr, 0, 1024, kSw128), dmb = make_smem_desc(mbt_addr, 128 * 128, 1024, kSw128);
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks)
                        mma_f16_ss(tm + TB_AUX, desc_adv(ddk, (ks >> 2) * (128 * 128) + (ks & 3) * 32), desc_adv(dmb, ks * 2048), id_dpsih, ks > 0);
                    mma_f16_ss(tm + TB_AUX, make_smem_desc(b3_addr, 0, 1024, kSw128), make_smem_desc(chi_addr, BC * 128, 1024, kSw128),
                               id_dpsih, 1);
                    tc_commit(&bar_mma[3]);
                }
                // chunk accumulators [G^M | dchi' | Psi] += psi^T [dg | dPm | S]   (K = the tile's 128 rows)
                const uint64_t dpsi = make_smem_desc(psi_addr, 128 * 128, 1024, kSw128);
                const uint64_t ddg = make_smem_desc(xdg_addr, 128 * 128, 1024, kSw128), dpm = make_smem_desc(pm_addr, 0, 256, kSw32);
                if (!DOT)
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    mma_f16_ss(tm + TB_GM, desc_adv(dpsi, ks * 2048), desc_adv(ddg, ks * 2048), id_gm, (tile > 0) || (ks > 0));
                // dv_j(intra) += dg^T Pm
                if (!DOT)
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    mma_f16_ss(tm + TB_DV, desc_adv(ddg, ks * 2048), desc_adv(dpm, ks * 512), id_n16, (tile > 0) || (ks > 0));
            }
            // ---- phase 4: du window update from Gt (thread = channel e, residues [16h, 16h+16))
            const int i0 = n * BC + tile * 2;
            uint32_t wv[16];
            if (t < D && !DOT) tmem_ld16(tm + lane_off + TB_DUW + h * 16, wv);   // the window does not depend on the product
            mbar_wait(&bar_mma[2], phase, status, 24);
            tc_fence_after();
            if (t < D && !DOT) {
#pragma unroll
                for (int qi = 0; qi < 2; ++qi) {
                    const int iq = i0 + qi;
                    uint32_t g[16];
                    tmem_ld16(tm + lane_off + TB_MAIN + qi * 64 + h * 16, g);
                    tmem_ld_wait();
                    const float dn = __bfloat162float(dOh[(tile * 2 + qi) * D + t]) * invs[tile * 2 + qi];
                    const float2 dn2 = make_float2(dn, dn);
                    const int k0 = (iq - 16 * h) & 63;     // residue 16h + k0 is the slot anchor iq takes over (if k0 <= 15)
                    if (k0 <= 15) {
                        // k0 = 2 * tile + qi here (the group that takes the chunk's own tokens in): a switch over the tile
                        // makes the slot a compile-time register index
                        // the anchor that leaves is token iq - 64: inside the segment, among its history rows, or nowhere
                        const int ca = iq - 64;
                        float *dst = du_acc + seq_off + (long)ca * D + t;
                        bool live = ca >= 0 && ca < T;
                        if (HIST && ca < 0 && ca >= -n_hist) {
                            dst = dhu_acc + ((long)bh * n_hist + n_hist + ca) * D + t;
                            live = true;
                        }
#define LS_FLUSH_DU(X) { if (live) atomicAdd(dst, __uint_as_float(wv[X])); wv[X] = 0u; }
                        switch (tile) {
                        case 0: LS_FLUSH_DU(0 + qi) break;
                        case 1: LS_FLUSH_DU(2 + qi) break;
                        case 2: LS_FLUSH_DU(4 + qi) break;
                        case 3: LS_FLUSH_DU(6 + qi) break;
                        case 4: LS_FLUSH_DU(8 + qi) break;
                        case 5: LS_FLUSH_DU(10 + qi) break;
                        case 6: LS_FLUSH_DU(12 + qi) break;
                        default: LS_FLUSH_DU(14 + qi) break;
                        }
#undef LS_FLUSH_DU
                    }
#pragma unroll
                    for (int x = 0; x < 16; x += 2) {
                        const float2 acc = ffma2(dn2, make_float2(__uint_as_float(g[x]), __uint_as_float(g[x + 1])),
                                                 make_float2(__uint_as_float(wv[x]), __uint_as_float(wv[x + 1])));
                        wv[x] = __float_as_uint(acc.x);
                        wv[x + 1] = __float_as_uint(acc.y);
                    }
                }
                tmem_st16(tm + lane_off + TB_DUW + h * 16, wv);
                tmem_st_wait();
            }
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {
                tc_fence_after();
                // the state's second term for all features at once, dg . Mb_lo^T, over Gt (the du epilogue has read it):
                // features 64.. share the accumulator of the block below, features 0..63 are added when dpsiN is read
                const uint64_t ddg = make_smem_desc(xdg_addr, 0, 1024, kSw128);
                if (use_lo) {
                    mbar_wait(&bar_lo, phase, status, 32);
                    tc_fence_after();
                    const uint64_t dml = make_smem_desc(om_addr, 128 * 128, 1024, kSw128);
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks)
                        mma_f16_ss(tm + TB_MAIN, desc_adv(ddg, (ks >> 2) * (128 * 128) + (ks & 3) * 32), desc_adv(dml, ks * 2048), id_dlo, ks > 0);
                    tc_commit(&bar_aux);
                }
                // second 64-feature block of dpsiN
                if (MF == 128) {
                    const uint64_t dmb = make_smem_desc(mbt_addr, 128 * 128, 1024, kSw128);
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks)
                        mma_f16_ss(tm + TB_MAIN + 64, desc_adv(ddg, (ks >> 2) * (128 * 128) + (ks & 3) * 32),
                                   desc_adv(dmb, ks * 2048 + 128 * 128), id_dpsih, use_lo || ks > 0);
                    mma_f16_ss(tm + TB_MAIN + 64, make_smem_desc(b3_addr, 0, 1024, kSw128),
                               make_smem_desc(chi_addr + BC * 128, BC * 128, 1024, kSw128), id_dpsih, 1);
                }
                tc_commit(&bar_mma[5]);
            }
            // ---- phase 5: dZ_i from psi' . dpsiN, then dl = (dpsiN + dZ_i a_i) * psi' (fp16, in place of psi'), row sums
            uint32_t psk[CPT / 2];                              // this thread's psi' values (bf16 pairs)
#pragma unroll
            for (int hf = 0; hf < 2; ++hf)
#pragma unroll
                for (int c8 = 0; c8 < CPT / 16; ++c8) {
                    const int cg = hf * (MF / 16) + h * (CPT / 16) + c8;
                    const uint4 pv = *(const uint4 *)(psi_s + (cg >> 3) * (128 * 128) + sw_off<128>(t, cg & 7));
                    const int o4 = (hf * (CPT / 16) + c8) * 4;
                    psk[o4] = pv.x; psk[o4 + 1] = pv.y; psk[o4 + 2] = pv.z; psk[o4 + 3] = pv.w;
                }
            mbar_wait(&bar_mma[3], phase, status, 25);
            if (use_lo) {
                mbar_wait(&bar_aux, phase, status, 34);
                if (tid == 0) {
                    // the products that read the state's second term are done: Omega returns for dxT and the next tile
                    mbar_arrive_expect_tx(&bar_omr, S::IMG_OM);
                    bulk_g2s(smem + S::OFF_OM, om_src, S::IMG_OM, &bar_omr);
                }
            }
            tc_fence_after();
            {
                uint32_t v[CPT];
                float dot = 0.f;
                const float *aqi = aq + il * MF;
                float2 z2 = make_float2(0.f, 0.f);                    // this thread's part of zeta_ic = psi'_ic . a_i
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    if (hf == 1) {
                        mbar_wait(&bar_mma[5], phase, status, 27);      // second half; every product reading psi' has finished
                        tc_fence_after();
                    }
                    const int f0 = hf * (MF / 2) + h * (CPT / 2);         // first feature of this piece
                    const uint32_t col = (f0 < 64) ? TB_AUX + f0 : TB_MAIN + f0;
                    if (CPT == 32) tmem_ld16(tm + lane_off + col, (uint32_t(&)[16])v[hf * (CPT / 2)]);
                    else tmem_ld8(tm + lane_off + col, (uint32_t(&)[8])v[hf * (CPT / 2)]);
                    if (use_lo && f0 < 64) {
                        uint32_t w[CPT / 2];
                        if (CPT == 32) tmem_ld16(tm + lane_off + TB_MAIN + f0, (uint32_t(&)[16])w);
                        else tmem_ld8(tm + lane_off + TB_MAIN + f0, (uint32_t(&)[8])w);
                        tmem_ld_wait();
#pragma unroll
                        for (int x = 0; x < CPT / 2; ++x)
                            v[hf * (CPT / 2) + x] = __float_as_uint(__uint_as_float(v[hf * (CPT / 2) + x]) + __uint_as_float(w[x]));
                    }
                    tmem_ld_wait();
                    float2 d2 = make_float2(0.f, 0.f);
#pragma unroll
                    for (int c8 = 0; c8 < CPT / 16; ++c8) {
#pragma unroll
                        for (int x = 0; x < 4; ++x) {
                            const int vi = hf * (CPT / 2) + c8 * 8 + 2 * x;
                            const float2 ps = up_bf16(psk[vi >> 1]);
                            d2 = ffma2(ps, make_float2(__uint_as_float(v[vi]), __uint_as_float(v[vi + 1])), d2);
                            z2 = ffma2(ps, *(const float2 *)(aqi + (hf * (MF / 16) + h * (CPT / 16) + c8) * 8 + 2 * x), z2);
                        }
                    }
                    dot += d2.x + d2.y;
                }
                // the row's parts of psi' . dpsiN and of zeta: 1^T dl_ic = psi'.dpsiN + dZ_i zeta_ic needs no second pass
                const float zrow = z2.x + z2.y;
                sdpart[h * 128 + t] = dot;
                hnp[h * 128 + t] = zrow;            // the |x|^2 partials kept there were consumed with the exponentials
                {
                    // both warp sums in one butterfly: the lower half of the warp collects the dots, the upper half zeta
                    const bool lo = lane < 16;
                    float acc = lo ? dot : zrow;
                    acc += __shfl_xor_sync(0xffffffffu, lo ? zrow : dot, 16);
#pragma unroll
                    for (int sh = 8; sh > 0; sh >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, sh);
                    if ((lane & 15) == 0) dred[warp * 2 + (lane >> 4)] = acc;
                }
                __syncthreads();
                // rows of query qi sit in the warps with bit 1 of the warp index equal to qi
                const int qi = t >> 6;
                float dsum = 0.f, zsum = 0.f;
#pragma unroll
                for (int w8 = 0; w8 < 8; ++w8) {
                    const float2 part = *(const float2 *)(dred + 2 * ((w8 >> 1) * 4 + qi * 2 + (w8 & 1)));
                    dsum += part.x;
                    zsum += part.y;
                }
                const long n_rows = (long)gridDim.y * T;              // the buffers hold [BH][T] sums, then [BH][T] normalisers
                if (EXT) dsum = (i < T) ? delta_ext[(long)bh * T + i] : 0.f;
                if (DOT && (t & 63) == 0 && h == 0 && i < T) {
                    atomicAdd(delta_out + (long)bh * T + i, dsum);
                    atomicAdd(delta_out + n_rows + (long)bh * T + i, zsum * invs[il]);
                }
                // dZ_i = -(dN_i . N'_i) / den'_i.  The normaliser is the one these very operands give, den'_i = sum_c
                // zeta_ic + eps m exp(-L_i), not the forward's: the numerator and normaliser parts of the key gradients
                // cancel, and what is left of them is only as exact as the two are consistent with each other.
                // Where the layer is a sum over several calls (EXT), the first passes have added up the calls'
                // normalisers relative to the forward's, sum_b zeta_b / den_fwd, and the forward's 1/den is corrected by it.
                float dz;
                if (EXT) {
                    const float kappa = (i < T) ? delta_ext[n_rows + (long)bh * T + i] + epsq[il] : 1.f;
                    dz = -dsum * invs[il] * rcp_approx(fmaxf(kappa, 1e-37f));
                } else if (DOT) dz = 0.f;
                else dz = -dsum * rcp_approx(fmaxf(zsum + epsq[il], 1e-37f));
                if ((t & 63) == 0 && h == 0) dzs[il] = dz;
                // minus the row sum of dl, in a fixed order (bit-reproducible); read by the dx epilogue after the next barrier
                if (h == 0)
                    sdlp[t] = -((((sdpart[t] + sdpart[128 + t]) + sdpart[256 + t]) + sdpart[384 + t]) +
                                dz * (((hnp[t] + hnp[128 + t]) + hnp[256 + t]) + hnp[384 + t]));
                if (!DOT)
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
#pragma unroll
                    for (int c8 = 0; c8 < CPT / 16; ++c8) {
                        const int cg = hf * (MF / 16) + h * (CPT / 16) + c8;
                        uint4 *cell = (uint4 *)(psi_s + (cg >> 3) * (128 * 128) + sw_off<128>(t, cg & 7));
                        uint32_t pk[4];
#pragma unroll
                        for (int x = 0; x < 4; ++x) {
                            const int col = cg * 8 + 2 * x;
                            const int vi = hf * (CPT / 2) + c8 * 8 + 2 * x;
                            const float2 dd = fmul2(ffma2(make_float2(dz, dz), *(const float2 *)(aqi + col),
                                                          make_float2(__uint_as_float(v[vi]), __uint_as_float(v[vi + 1]))), up_bf16(psk[vi >> 1]));
                            pk[x] = pk_f16(dd.x, dd.y);
                        }
                        *cell = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    }
                }
            }
            fence_proxy_async_smem();
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {
                if (use_lo) mbar_wait(&bar_omr, phase, status, 33);
                tc_fence_after();
                // dxT = Omega . dl^T  (OmegaT image read MN-major: rows = p, 64-wide a blocks), one query
                // (64 tile rows) at a time so that the epilogue of the first starts under the second
                const uint64_t dom = make_smem_desc(om_addr, MF * 128, 1024, kSw128), ddl = make_smem_desc(psi_addr, 0, 1024, kSw128);
#pragma unroll
                for (int qi = 0; qi < 2; ++qi) {
                    if (!DOT)
#pragma unroll
                    for (int ks = 0; ks < MF / 16; ++ks)
                        mma_f16_ss(tm + TB_MAIN + qi * 64, desc_adv(dom, ks * 2048),
                                   desc_adv(ddl, (ks >> 2) * (128 * 128) + (ks & 3) * 32 + qi * 8192), id_dxh, ks > 0);
                    tc_commit(&bar_mma[qi ? 6 : 4]);
                }
            }
            if (tile + 1 < BC / 2) phase1(tile + 1);
            // ---- phase 6: dx = dxT - sdl * x ; dq_i (partial over this thread's residues), dr window
            if (t < D && !DOT) tmem_ld16(tm + lane_off + TB_DRW + h * 16, wv);
            mbar_wait(&bar_mma[4], phase, status, 26);
            tc_fence_after();
            if (t >= D || DOT) mbar_wait(&bar_mma[6], phase, status, 28);
            if (t < D && !DOT) {
#pragma unroll
                for (int qi = 0; qi < 2; ++qi) {
                    const int iq = i0 + qi;
                    if (qi == 1) {
                        mbar_wait(&bar_mma[6], phase, status, 28);
                        tc_fence_after();
                    }
                    uint32_t g[16];
                    tmem_ld16(tm + lane_off + TB_MAIN + qi * 64 + h * 16, g);
                    tmem_ld_wait();
                    const float qa = __half2float(((const __half *)(qs + (tile * 2 + qi) * S::ROWB))[t]);
                    const int k0 = (iq - 16 * h) & 63;
                    // the 16 residues are tokens iq - k0 + x (one ring group) up to x = k0 and the group four before
                    // (the next ring slot) beyond
                    const int ra = ring_row(iq - k0);
                    const uint8_t *pa = rwin + ra * S::PITCH + t * 2;
                    const uint8_t *pb = rwin + (ra >= 4 * BC ? ra - 4 * BC : ra + BC) * S::PITCH + t * 2;
                    const float2 *nsdl2 = (const float2 *)(sdlp + qi * 64 + h * 16);
                    const float2 qa2 = make_float2(qa, qa);
                    float2 dq2 = make_float2(0.f, 0.f);
                    // WRAP: this group of 16 residues holds the slot that anchor iq takes over (k0 <= 15), so
                    // rows come from two places; otherwise it is a plain stream
                    auto pairs = [&](auto wrap_tag) {
                        constexpr bool WRAP = decltype(wrap_tag)::value;
#pragma unroll
                        for (int x = 0; x < 16; x += 2) {
                            const uint8_t *p0 = (!WRAP || x <= k0) ? pa : pb, *p1 = (!WRAP || x + 1 <= k0) ? pa : pb;
                            const float2 rv = make_float2(__half2float(*(const __half *)(p0 + x * S::PITCH)),
                                                          __half2float(*(const __half *)(p1 + (x + 1) * S::PITCH)));
                            const float2 qr = fmul2(qa2, rv);
                            const float2 dxv = ffma2(nsdl2[x >> 1], qr, make_float2(__uint_as_float(g[x]), __uint_as_float(g[x + 1])));
                            dq2 = ffma2(dxv, rv, dq2);
                            const float2 acc = ffma2(dxv, qa2, make_float2(__uint_as_float(wv[x]), __uint_as_float(wv[x + 1])));
                            wv[x] = __float_as_uint(acc.x);
                            wv[x + 1] = __float_as_uint(acc.y);
                        }
                    };
                    if (k0 >= 16) {
                        pairs(std::false_type{});
                    } else {
                        // anchor iq takes residue k0 = 2 * tile + qi over: what the slot holds leaves first (a switch over
                        // the tile makes it a compile-time register index)
                        const int ca = iq - 64;
                        float *dst = dr_acc + seq_off + (long)ca * D + t;
                        bool live = ca >= 0 && ca < T;
                        if (HIST && ca < 0 && ca >= -n_hist) {
                            dst = dhr_acc + ((long)bh * n_hist + n_hist + ca) * D + t;
                            live = true;
                        }
#define LS_FLUSH_DR(X) { if (live) atomicAdd(dst, __uint_as_float(wv[X])); wv[X] = 0u; }
                        switch (tile) {
                        case 0: LS_FLUSH_DR(0 + qi) break;
                        case 1: LS_FLUSH_DR(2 + qi) break;
                        case 2: LS_FLUSH_DR(4 + qi) break;
                        case 3: LS_FLUSH_DR(6 + qi) break;
                        case 4: LS_FLUSH_DR(8 + qi) break;
                        case 5: LS_FLUSH_DR(10 + qi) break;
                        case 6: LS_FLUSH_DR(12 + qi) break;
                        default: LS_FLUSH_DR(14 + qi) break;
                        }
#undef LS_FLUSH_DR
                        pairs(std::true_type{});
                    }
                    const float dqa = dq2.x + dq2.y;
                    dqp[(h * 2 + qi) * 128 + t] = dqa;
                }
                tmem_st16(tm + lane_off + TB_DRW + h * 16, wv);
                tmem_st_wait();
            }
            tc_fence_before();
            __syncthreads();
            if (t < D && h < 2 && !DOT) {
                const int iq = i0 + h;                           // parts h = 0, 1 write queries 0, 1
                if (iq < T) {
                    const float dqv = (dqp[h * 128 + t] + dqp[(2 + h) * 128 + t]) + (dqp[(4 + h) * 128 + t] + dqp[(6 + h) * 128 + t]);
                    if (EXT) {                                   // one feature block of several: fp32, summed over the blocks
                        float *dst = (float *)dq + seq_off + (long)iq * D + t;
                        *dst = (grad32 == 2 ? *dst : 0.f) + dqv;
                    } else {
                        dq[seq_off + (long)iq * D + t] = __float2bfloat16_rn(dqv);
                    }
                }
            }
            last_query = i0 + 1;
            phase ^= 1;
        }
        // ---- chunk epilogue: all MMAs of the chunk have completed (last wait above)
        if (tid == 0 && n + 1 < n_end) {
            mbar_arrive_expect_tx(&bar_img, S::IMG_CHUNK);
            bulk_g2s(smem + S::OFF_CHUNK, img_bh + (long)(n + 1) * S::IMG_CHUNK, S::IMG_CHUNK, &bar_img);
        }
        if (!DOT) {
            float *gout = gstates + ((long)bh * NC + n) * E;
            // G^M_n [p][e]: thread = feature p, a quarter of the channels each.  A row per thread straight to global
            // memory would be 32 separate lines per store instruction: the block is assembled in shared memory (the
            // tile buffers are free between chunks) and leaves as one bulk store after the barrier below.  Inside a row
            // the 16-byte pieces are permuted (piece c at c ^ (p & 7)), which keeps the shared-memory writes free of
            // bank conflicts; the key/value sweep undoes it when it reads (the segment sums are elementwise).
            constexpr int QUART = D / BR;
            if (t >= MF) {
                // lanes beyond the feature rank hold padding only
            } else if (QUART == 32) {
                uint32_t v[32];
                tmem_ld32(tm + lane_off + TB_GM + h * 32, v);
                tmem_ld_wait();
#pragma unroll
                for (int x = 0; x < 32; x += 4)
                    *(float4 *)(gm_stage + t * (D * 4) + (((h * 8 + (x >> 2)) ^ (t & 7)) << 4)) =
                        make_float4(__uint_as_float(v[x]), __uint_as_float(v[x + 1]), __uint_as_float(v[x + 2]), __uint_as_float(v[x + 3]));
            } else {
                uint32_t v[16];
                tmem_ld16(tm + lane_off + TB_GM + h * 16, v);
                tmem_ld_wait();
#pragma unroll
                for (int x = 0; x < 16; x += 4)
                    *(float4 *)(gm_stage + t * (D * 4) + (((h * 4 + (x >> 2)) ^ (t & 7)) << 4)) =
                        make_float4(__uint_as_float(v[x]), __uint_as_float(v[x + 1]), __uint_as_float(v[x + 2]), __uint_as_float(v[x + 3]));
            }
            fence_proxy_async_smem();
            uint32_t v[16];
            if (h == 0 && t < MF) {
                // feature p = t: Psi_i[p] for the chunk's 16 queries, numerator part of dchi'_j[p]
                uint32_t ps[16];
                tmem_ld16(tm + lane_off + TB_GM + 128, v);
                tmem_ld16(tm + lane_off + TB_GM + 144, ps);
                tmem_ld_wait();
                // dchi'_j(intra) = numerator part + sum_{i >= j} dZ_i Psi_i ;  G^a_n = sum_i dZ_i Psi_i
                float *dst = dchi_intra + ((long)bh * NC + n) * BC * MF;
                float suf = 0.f;
#pragma unroll
                for (int j = BC - 1; j >= 0; --j) {
                    suf = fmaf(dzs[j], __uint_as_float(ps[j]), suf);
                    dst[j * MF + t] = __uint_as_float(v[j]) + suf;
                }
                gout[(long)MF * D + t] = suf;
            } else if (h == 1 && t < D) {
                tmem_ld16(tm + lane_off + TB_DV, v);
                tmem_ld_wait();
                float *dst = dv_intra + ((long)bh * NC + n) * BC * D;
#pragma unroll
                for (int j = 0; j < BC; ++j) dst[j * D + t] = __uint_as_float(v[j]);
            }
        }
        tc_fence_before();
        __syncthreads();
        if (!DOT && tid == 0) bulk_s2g(gstates + ((long)bh * NC + n) * E, gm_stage, MF * D * 4);
    }
    if (!DOT && tid == 0) bulk_wait_all<0>();
    // ---- flush what is still in the windows: residue x holds anchor_of(last_query, x)
    if (t < D && last_query >= 0 && !DOT) {
        uint32_t wu[16], wr_[16];
        tmem_ld16(tm + lane_off + TB_DUW + h * 16, wu);
        tmem_ld16(tm + lane_off + TB_DRW + h * 16, wr_);
        tmem_ld_wait();
#pragma unroll
        for (int x = 0; x < 16; ++x) {
            const int ca = anchor_of(last_query, h * 16 + x);
            if (ca >= 0 && ca < T) {
                atomicAdd(du_acc + seq_off + (long)ca * D + t, __uint_as_float(wu[x]));
                atomicAdd(dr_acc + seq_off + (long)ca * D + t, __uint_as_float(wr_[x]));
            } else if (HIST && ca < 0 && ca >= -n_hist) {
                atomicAdd(dhu_acc + ((long)bh * n_hist + n_hist + ca) * D + t, __uint_as_float(wu[x]));
                atomicAdd(dhr_acc + ((long)bh * n_hist + n_hist + ca) * D + t, __uint_as_float(wr_[x]));
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base_s, 512);
}

// OmegaT image padded to 128 a-columns (two 64-wide blocks), fp16.  grid (n_omega)
template <int D, int MF>
__global__ void k_omega_image_pad_tc(const float *__restrict__ omega, int m_real, int omega_ld, long bank_stride,
                                     uint8_t *__restrict__ img)
{
    const float *om = omega + (long)blockIdx.x * bank_stride;
    uint8_t *out = img + (long)blockIdx.x * (MF * 128 * 2);
    for (int idx = threadIdx.x; idx < MF * 16; idx += blockDim.x) {
        const int p = idx >> 4, c8 = idx & 15;
        __align__(16) __half pk[8];
#pragma unroll
        for (int x = 0; x < 8; ++x) pk[x] = __float2half_rn((c8 * 8 + x < D && p < m_real) ? om[(long)(c8 * 8 + x) * omega_ld + p] : 0.f);
        *(uint4 *)(out + (c8 >> 3) * (MF * 128) + sw_off<128>(p, c8 & 7)) = *(const uint4 *)pk;
    }
}

// ------------------------------------------------------------------ key/value sweep
// Per-segment sums of the chunk state gradients: segsum[bh][seg] = sum_{n in seg} G_n.  grid (NSEG, BH).
static constexpr int kTcDkChunks = 8;      // chunks per CTA of the dk kernel (amortises Omega in shared memory)
static constexpr int KV_SEG = kTcKvSeg;    // least number of chunks per segment of the key/value sweep (sizes the workspace)

__global__ void __launch_bounds__(256) k_seg_sum_tc(const float *__restrict__ g, int NC, long E, float *__restrict__ segsum,
                                                    int seg_len)
{
    const int seg = blockIdx.x, bh = blockIdx.y, NSEG = gridDim.x;
    const int n0 = seg * seg_len, n1 = min(NC, n0 + seg_len);
    const long E4 = E / 4;
    for (long f = blockIdx.z * 256 + threadIdx.x; f < E4; f += 256 * gridDim.z) {     // grid.z splits the state's elements
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        const float4 *src = (const float4 *)(g + ((long)bh * NC + n0) * E) + f;
#pragma unroll 8
        for (int n = n0; n < n1; ++n) {
            const float4 x = src[(long)(n - n0) * E4];
            acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
        }
        ((float4 *)(segsum + ((long)bh * NSEG + seg) * E))[f] = acc;
    }
}

// warp-level m16n8k8 TF32 MMA, fp32 accumulate (the M = 16 GEMMs of one chunk fit it exactly)
__device__ __forceinline__ void mma_tf32(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2])
{
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
__device__ __forceinline__ uint32_t to_tf32(float x)
{
    uint32_t y;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(y) : "f"(x));
    return y;
}

// C[16][n0..n0+16) += A[16][K] . B, A row-major in smem (lda), B element (k, n) at Bs[k*sk + n*sn].
// SPLIT_A / SPLIT_B add the tf32 residual of the operand (two-term split, ~fp32 accuracy of that operand).
template <int K, bool SPLIT_A, bool SPLIT_B>
__device__ __forceinline__ void warp_gemm16(float (&c)[2][4], const float *As, int lda, const float *Bs, int sk, int sn, int n0)
{
    const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
#pragma unroll 4
    for (int k0 = 0; k0 < K; k0 += 8) {
        float af[4] = {As[g * lda + k0 + t], As[(g + 8) * lda + k0 + t], As[g * lda + k0 + t + 4], As[(g + 8) * lda + k0 + t + 4]};
        uint32_t ah[4], al[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            ah[x] = to_tf32(af[x]);
            al[x] = SPLIT_A ? to_tf32(af[x] - __uint_as_float(ah[x])) : 0u;
        }
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
            const int n = n0 + nt * 8 + g;
            float bf[2] = {Bs[(k0 + t) * sk + n * sn], Bs[(k0 + t + 4) * sk + n * sn]};
            uint32_t bhh[2], bl[2];
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                bhh[x] = to_tf32(bf[x]);
                bl[x] = SPLIT_B ? to_tf32(bf[x] - __uint_as_float(bhh[x])) : 0u;
            }
            mma_tf32(c[nt], ah, bhh);
            if (SPLIT_B) mma_tf32(c[nt], ah, bl);
            if (SPLIT_A) mma_tf32(c[nt], al, bhh);
        }
    }
}

// grid (NSEG, BH), 256 threads = 8 warps, two CTAs per SM.  A CTA walks the chunks of its segment backwards with
// the running D = sum_{n' > n} G^M_n' [p][e] and e = sum G^a in shared memory (fp32):
//   dl^k_j = (D v_j + e + intra) * chi'_j ,   dv_j = D^T chi'_j + intra
// chi'_j (fp32) comes from the pre-pass; dl^k_j replaces it in place and k_bwd_dk_tc turns it into dk.  The two
// [16 x 128] products per chunk run on warp-level TF32 tensor-core MMAs; D in the cancelling sum D v + e is
// split in two TF32 terms.
template <int D, int MF>
__global__ void __launch_bounds__(256, 2)
k_bwd_kv_tc(const bf16 *__restrict__ v, int T, int NC, const float *__restrict__ gstates, const float *__restrict__ segsum,
            const float *__restrict__ dv_intra, const float *__restrict__ dchi_intra, float *__restrict__ chi_dl,
            bf16 *__restrict__ dv, int grad32, int seg_len, const float *__restrict__ dS_fin, const float *__restrict__ dz_fin,
            int state_m, int m_real)
{
    constexpr int LDD = D + 4, LDK = D + 4, LDC = MF + 4;
    extern __shared__ float sm[];
    float *Ds = sm;                        // D [MF][LDD]
    float *es = Ds + MF * LDD;             // [MF]
    float *vs = es + MF;                   // [16][LDK]
    float *chi = vs + BC * LDK;            // [16][LDC]
    const int seg = blockIdx.x, bh = blockIdx.y, NSEG = gridDim.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const long seq_off = (long)bh * T * D;
    const long E = (long)MF * D + MF;
    // suffix over the later segments
    for (int idx = threadIdx.x; idx < MF * D; idx += 256) {
        float acc = 0.f;
        for (int s2 = seg + 1; s2 < NSEG; ++s2) acc += segsum[((long)bh * NSEG + s2) * E + idx];
        const int p = idx / D, e0 = idx - p * D;
        const int e = (((e0 >> 2) ^ (p & 7)) << 2) | (e0 & 3);         // the tile kernel permutes the 16-byte pieces of a row
        // (a continued segment: the gradient that later segments send into the state after this one)
        if (dS_fin && p < m_real) acc += dS_fin[((long)bh * state_m + p) * D + e];
        Ds[p * LDD + e] = acc;
    }
    for (int p = threadIdx.x; p < MF; p += 256) {
        float acc = 0.f;
        for (int s2 = seg + 1; s2 < NSEG; ++s2) acc += segsum[((long)bh * NSEG + s2) * E + (long)MF * D + p];
        if (dz_fin && p < m_real) acc += dz_fin[(long)bh * state_m + p];
        es[p] = acc;
    }
    const int n_hi = min(NC, (seg + 1) * seg_len) - 1;
    // each staging thread holds 8 consecutive channels of one token's v and 8 consecutive features of its chi'
    constexpr int VT = BC * D / 8, CT = BC * MF / 8;                   // staging threads (<= 256 each)
    const int v_j = threadIdx.x / (D / 8), v_c = threadIdx.x % (D / 8);
    uint4 vq = make_uint4(0, 0, 0, 0);
    float4 cq0 = make_float4(0.f, 0.f, 0.f, 0.f), cq1 = cq0;
    auto fetch = [&](int nn) {
        vq = make_uint4(0, 0, 0, 0);
        cq0 = cq1 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (nn < 0) return;
        const int tok = nn * BC + v_j;
        if (threadIdx.x < VT && tok < T) vq = *(const uint4 *)(v + seq_off + (long)tok * D + v_c * 8);
        if (threadIdx.x < CT) {
            const float4 *src = (const float4 *)(chi_dl + ((long)bh * NC + nn) * BC * MF) + threadIdx.x * 2;
            cq0 = src[0];
            cq1 = src[1];
        }
    };
    fetch(n_hi);
    // the intra-chunk parts this thread's product fragments are added to, requested before the products
    const int n0 = warp * 16;                           // this warp's 16 features / channels
    float2 di[2][2], iv[2][2];
    auto fetch_intra = [&](int nn) {
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const int j = g + hh * 8, c0 = n0 + nt * 8 + 2 * t;
                di[nt][hh] = iv[nt][hh] = make_float2(0.f, 0.f);
                if (n0 < MF) di[nt][hh] = *(const float2 *)(dchi_intra + ((long)bh * NC + nn) * BC * MF + j * MF + c0);
                if (n0 < D) iv[nt][hh] = *(const float2 *)(dv_intra + ((long)bh * NC + nn) * BC * D + j * D + c0);
            }
    };
    constexpr int GQ = MF * D / 4 / 256;               // float4 pieces of G^M_n per thread
    for (int n = n_hi; n >= seg * seg_len; --n) {
        __syncthreads();                               // D, e of this chunk complete; tiles free
        if (threadIdx.x < VT) {
            const uint32_t vw[4] = {vq.x, vq.y, vq.z, vq.w};
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                vs[v_j * LDK + v_c * 8 + 2 * x] = __uint_as_float(vw[x] << 16);
                vs[v_j * LDK + v_c * 8 + 2 * x + 1] = __uint_as_float(vw[x] & 0xffff0000u);
            }
        }
        if (threadIdx.x < CT) {
            const int cj = threadIdx.x / (MF / 8), cc = threadIdx.x % (MF / 8);
            *(float4 *)(chi + cj * LDC + cc * 8) = cq0;
            *(float4 *)(chi + cj * LDC + cc * 8 + 4) = cq1;
        }
        // requests whose latency the products below cover: this chunk's state gradient, the next chunk's tokens
        const float *gs = gstates + ((long)bh * NC + n) * E;
        float4 gq[GQ];
#pragma unroll
        for (int x = 0; x < GQ; ++x) gq[x] = ((const float4 *)gs)[threadIdx.x + 256 * x];
        const float ga_n = (threadIdx.x < MF) ? gs[(long)MF * D + threadIdx.x] : 0.f;
        fetch(n - 1 >= seg * seg_len ? n - 1 : -1);
        fetch_intra(n);
        __syncthreads();
        if (n0 < MF) {
            float c[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
            warp_gemm16<D, false, true>(c, vs, LDK, Ds, 1, LDD, n0);          // D v : B(k = e, n = p) = D[p][e]
            float *dlo = chi_dl + ((long)bh * NC + n) * BC * MF;              // dl^k over chi' (this thread's own elements)
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const int j = g + hh * 8, p = n0 + nt * 8 + 2 * t;
                    const float2 cx = *(const float2 *)(chi + j * LDC + p);
                    // the intra-chunk part belongs to pair weights formed from the bf16 image of chi'
                    *(float2 *)(dlo + j * MF + p) = make_float2(fmaf(c[nt][hh * 2] + es[p], cx.x, di[nt][hh].x * bf16_round(cx.x)),
                                                                fmaf(c[nt][hh * 2 + 1] + es[p + 1], cx.y, di[nt][hh].y * bf16_round(cx.y)));
                }
        }
        if (n0 < D) {
            float c[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
            warp_gemm16<MF, false, false>(c, chi, LDC, Ds, LDD, 1, n0);       // D^T chi' : B(k = p, n = e) = D[p][e]
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const int j = g + hh * 8, e = n0 + nt * 8 + 2 * t;
                    const int tok = n * BC + j;
                    if (tok < T) {
                        const float2 val = make_float2(c[nt][hh * 2] + iv[nt][hh].x, c[nt][hh * 2 + 1] + iv[nt][hh].y);
                        if (grad32) {
                            float2 *dst = (float2 *)((float *)dv + seq_off + (long)tok * D + e);
                            const float2 old = grad32 == 2 ? *dst : make_float2(0.f, 0.f);
                            *dst = make_float2(old.x + val.x, old.y + val.y);
                        } else {
                            *(__nv_bfloat162 *)(dv + seq_off + (long)tok * D + e) = __floats2bfloat162_rn(val.x, val.y);
                        }
                    }
                }
        }
        __syncthreads();                                 // every read of D done
        // D += G^M_n, e += G^a_n (the chunk's own gradient enters only for earlier chunks)
#pragma unroll
        for (int x = 0; x < GQ; ++x) {
            const int idx = threadIdx.x + 256 * x;
            const int p = (idx * 4) / D, e0 = (idx * 4) - p * D;
            float *dst = Ds + p * LDD + (((e0 >> 2) ^ (p & 7)) << 2);
            dst[0] += gq[x].x; dst[1] += gq[x].y; dst[2] += gq[x].z; dst[3] += gq[x].w;
        }
        if (threadIdx.x < MF) es[threadIdx.x] += ga_n;
    }
}

// The same sweep on tcgen05 for d = m = 128 and bf16 dv (the warp-level kernel above keeps the other shapes and the
// fp32-accumulating case).  The running D [p][e] is held in registers (64 values per thread, in the layout the tile
// kernel stores G^M_n in); after every update it is written as three bf16 terms (24 mantissa bits: D v + e cancels)
// into one swizzled operand image that serves both products of the next chunk:
//   dchi^T[p][j] = sum_e D[p][e] v_j[e]      A = the image K-major,  B = the chunk's v rows       (3 terms)
//   dv^T[e][j]   = sum_p D[p][e] chi'_j[p]   A = the image MN-major, B = chi' in two bf16 terms   (hi.hi, hi.mid, mid.hi)
// with N = 16 tokens and the two [128 x 16] accumulators in tensor memory.  The chunk's G^M_n is added to the registers
// while the products run.  grid (NSEG, BH), 256 threads, two CTAs per SM.
struct Kv5Smem {
    static constexpr int DIMG = 128 * 128 * 2;                 // one bf16 term of D: [p][e], per 64-wide e block [128][128 B]
    static constexpr int VB = BC * 128 * 2;                    // v rows [j][e], per 64-wide e block [16][128 B]
    static constexpr int XB = BC * 128 * 2;                    // one bf16 term of chi' [j][p]
    static constexpr int OFF_D = 0, OFF_V = 3 * DIMG, OFF_X = OFF_V + VB, TOTAL = OFF_X + 2 * XB;
};

__global__ void __launch_bounds__(256, 2)
k_bwd_kv_tc5(const bf16 *__restrict__ v, int T, int NC, const float *__restrict__ gstates, const float *__restrict__ segsum,
             const float *__restrict__ dv_intra, const float *__restrict__ dchi_intra, float *__restrict__ chi_dl,
             bf16 *__restrict__ dv, int seg_len, int *__restrict__ status, const float *__restrict__ dS_fin,
             const float *__restrict__ dz_fin)
{
    constexpr int D = 128, MF = 128, NX = MF * D / 4 / 256;    // 16 float4 of D per thread
    using S = Kv5Smem;
    extern __shared__ __align__(1024) uint8_t smem_dyn[];
    uint8_t *smem = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
    __shared__ uint64_t bar_mma;
    __shared__ uint32_t tmem_base_s;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int seg = blockIdx.x, bh = blockIdx.y, NSEG = gridDim.x;
    const long seq_off = (long)bh * T * D;
    const long E = (long)MF * D + MF;
    if (warp == 0) {
        tmem_alloc(&tmem_base_s, 32);
        tmem_relinquish();
    }
    if (tid == 0) {
        mbar_init(&bar_mma, 1);
        fence_barrier_init();
    }
    // this thread's part of D: float4 number tid + 256 x of the [p][e] block, i.e. row p = warp + 8 x, stored piece
    // `lane`, which holds channels 4 (lane ^ (p & 7)) .. + 3 (the tile kernel permutes the 16-byte pieces of a row)
    float4 Dr[NX];
#pragma unroll
    for (int x = 0; x < NX; ++x) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s2 = seg + 1; s2 < NSEG; ++s2) {
            const float4 w = ((const float4 *)(segsum + ((long)bh * NSEG + s2) * E))[tid + 256 * x];
            acc.x += w.x; acc.y += w.y; acc.z += w.z; acc.w += w.w;
        }
        if (dS_fin) {
            // a continued segment: the gradient that later segments send into the state after this one ([p][e], plain order)
            const int p = warp + 8 * x, e = (lane ^ (p & 7)) * 4;
            const float4 w = *(const float4 *)(dS_fin + ((long)bh * MF + p) * D + e);
            acc.x += w.x; acc.y += w.y; acc.z += w.z; acc.w += w.w;
        }
        Dr[x] = acc;
    }
    const int row = (warp & 3) * 32 + lane, half = warp >> 2;   // accumulator row (p resp. e) and token half of the epilogues
    float es = 0.f;                                             // e[p] for p = row
    for (int s2 = seg + 1; s2 < NSEG; ++s2) es += segsum[((long)bh * NSEG + s2) * E + (long)MF * D + row];
    if (dz_fin) es += dz_fin[(long)bh * MF + row];
    auto store_images = [&]() {
#pragma unroll
        for (int x = 0; x < NX; ++x) {
            const int p = warp + 8 * x, e = (lane ^ (p & 7)) * 4;
            const float wv[4] = {Dr[x].x, Dr[x].y, Dr[x].z, Dr[x].w};
            uint32_t t0[2], t1[2], t2[2];
#pragma unroll
            for (int y = 0; y < 2; ++y) {
                const __nv_bfloat162 h2 = __floats2bfloat162_rn(wv[2 * y], wv[2 * y + 1]);
                const float2 hf = __bfloat1622float2(h2);
                const float r0 = wv[2 * y] - hf.x, r1 = wv[2 * y + 1] - hf.y;
                const __nv_bfloat162 m2 = __floats2bfloat162_rn(r0, r1);
                const float2 mf = __bfloat1622float2(m2);
                const __nv_bfloat162 l2 = __floats2bfloat162_rn(r0 - mf.x, r1 - mf.y);
                t0[y] = *(const uint32_t *)&h2;
                t1[y] = *(const uint32_t *)&m2;
                t2[y] = *(const uint32_t *)&l2;
            }
            const uint32_t off = (e >> 6) * (128 * 128) + sw_off<128>(p, (e & 63) >> 3) + (e & 4) * 2;
            *(uint2 *)(smem + S::OFF_D + off) = make_uint2(t0[0], t0[1]);
            *(uint2 *)(smem + S::OFF_D + S::DIMG + off) = make_uint2(t1[0], t1[1]);
            *(uint2 *)(smem + S::OFF_D + 2 * S::DIMG + off) = make_uint2(t2[0], t2[1]);
        }
    };
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = tmem_base_s;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t id1 = make_idesc_f16(128, BC, 1, 0, 0);       // D (K-major) . v^T
    const uint32_t id2 = make_idesc_f16(128, BC, 1, 1, 0);       // D^T (the image read MN-major) . chi'^T
    const int n_hi = min(NC, (seg + 1) * seg_len) - 1, n_lo = seg * seg_len;
    // the chunk's v rows (one 16-byte piece per thread) and chi' rows (two float4 per thread), fetched a chunk ahead
    uint4 vq;
    float4 cq0, cq1;
    auto fetch = [&](int nn) {
        vq = make_uint4(0, 0, 0, 0);
        cq0 = cq1 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (nn < n_lo) return;
        const int tok = nn * BC + (tid >> 4);
        if (tok < T) vq = *(const uint4 *)(v + seq_off + (long)tok * D + (tid & 15) * 8);
        const float4 *src = (const float4 *)(chi_dl + ((long)bh * NC + nn) * BC * MF) + tid * 2;
        cq0 = src[0];
        cq1 = src[1];
    };
    fetch(n_hi);
    store_images();
    uint32_t phase = 0;
    for (int n = n_hi; n >= n_lo; --n) {
        // B operands of chunk n
        {
            const int j = tid >> 4, c = tid & 15;                           // v: row j, 16-byte piece c (8 channels)
            *(uint4 *)(smem + S::OFF_V + (c >> 3) * (BC * 128) + sw_off<128>(j, c & 7)) = vq;
            const int jx = tid >> 4, p0 = (tid & 15) * 8;                   // chi': row jx, features p0 .. p0 + 7
            const float wv[8] = {cq0.x, cq0.y, cq0.z, cq0.w, cq1.x, cq1.y, cq1.z, cq1.w};
            uint32_t hh[4], mm[4];
#pragma unroll
            for (int y = 0; y < 4; ++y) {
                const __nv_bfloat162 h2 = __floats2bfloat162_rn(wv[2 * y], wv[2 * y + 1]);
                const float2 hf = __bfloat1622float2(h2);
                const __nv_bfloat162 m2 = __floats2bfloat162_rn(wv[2 * y] - hf.x, wv[2 * y + 1] - hf.y);
                hh[y] = *(const uint32_t *)&h2;
                mm[y] = *(const uint32_t *)&m2;
            }
            const uint32_t off = (p0 >> 6) * (BC * 128) + sw_off<128>(jx, (p0 & 63) >> 3);
            *(uint4 *)(smem + S::OFF_X + off) = make_uint4(hh[0], hh[1], hh[2], hh[3]);
            *(uint4 *)(smem + S::OFF_X + S::XB + off) = make_uint4(mm[0], mm[1], mm[2], mm[3]);
        }
        // this thread's chi' (fp32) and intra-chunk parts for the epilogues: row = feature resp. channel, 8 tokens
        float xc[8], di[8], iv[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const long tokc = ((long)bh * NC + n) * BC + half * 8 + j;
            xc[j] = chi_dl[tokc * MF + row];
            di[j] = dchi_intra[tokc * MF + row];
            iv[j] = dv_intra[tokc * D + row];
        }
        fetch(n - 1);
        // what the chunk before will read with plain loads while its products run: have it in L2 by then
        if (tid == 0 && n > n_lo) {
            bulk_prefetch_l2(gstates + ((long)bh * NC + n - 1) * E, (uint32_t)(E * 4));
            bulk_prefetch_l2(dchi_intra + ((long)bh * NC + n - 1) * BC * MF, BC * MF * 4);
            bulk_prefetch_l2(dv_intra + ((long)bh * NC + n - 1) * BC * D, BC * D * 4);
        }
        fence_proxy_async_smem();
        tc_fence_before();
        __syncthreads();
        if (tid == 0) {
            tc_fence_after();
            const uint64_t dv_ = make_smem_desc(smem_u32(smem + S::OFF_V), 0, 1024, kSw128);
#pragma unroll
            for (int term = 0; term < 3; ++term) {
                const uint64_t da = make_smem_desc(smem_u32(smem + S::OFF_D + term * S::DIMG), 0, 1024, kSw128);
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks)
                    mma_f16_ss(tm, desc_adv(da, (ks >> 2) * (128 * 128) + (ks & 3) * 32),
                               desc_adv(dv_, (ks >> 2) * (BC * 128) + (ks & 3) * 32), id1, (term > 0) || (ks > 0));
            }
#pragma unroll
            for (int term = 0; term < 3; ++term) {
                // hi.hi, hi.mid, mid.hi
                const uint64_t da = make_smem_desc(smem_u32(smem + S::OFF_D + (term == 2 ? S::DIMG : 0)), 128 * 128, 1024, kSw128);
                const uint64_t dx = make_smem_desc(smem_u32(smem + S::OFF_X + (term == 1 ? S::XB : 0)), 0, 1024, kSw128);
#pragma unroll
                for (int ks = 0; ks < MF / 16; ++ks)
                    mma_f16_ss(tm + BC, desc_adv(da, ks * 2048), desc_adv(dx, (ks >> 2) * (BC * 128) + (ks & 3) * 32), id2,
                               (term > 0) || (ks > 0));
            }
            tc_commit(&bar_mma);
        }
        // while the products run: D += G^M_n (takes effect for the chunks before n), e likewise after its use below
        const float *gs = gstates + ((long)bh * NC + n) * E;
#pragma unroll
        for (int x0 = 0; x0 < NX; x0 += 4) {
            float4 gq[4];
#pragma unroll
            for (int y = 0; y < 4; ++y) gq[y] = __ldcs(((const float4 *)gs) + tid + 256 * (x0 + y));
#pragma unroll
            for (int y = 0; y < 4; ++y) {
                Dr[x0 + y].x += gq[y].x; Dr[x0 + y].y += gq[y].y; Dr[x0 + y].z += gq[y].z; Dr[x0 + y].w += gq[y].w;
            }
        }
        const float ga = gs[(long)MF * D + row];
        mbar_wait(&bar_mma, phase, status, 35);
        phase ^= 1;
        tc_fence_after();
        {
            uint32_t a1[8], a2[8];
            tmem_ld8(tm + lane_off + half * 8, a1);
            tmem_ld8(tm + lane_off + BC + half * 8, a2);
            tmem_ld_wait();
            float *dlo = chi_dl + (((long)bh * NC + n) * BC + half * 8) * MF + row;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                // the intra-chunk part belongs to pair weights formed from the bf16 image of chi'
                dlo[(long)j * MF] = fmaf(__uint_as_float(a1[j]) + es, xc[j], di[j] * bf16_round(xc[j]));
                const int tok = n * BC + half * 8 + j;
                if (tok < T) dv[seq_off + (long)tok * D + row] = __float2bfloat16_rn(__uint_as_float(a2[j]) + iv[j]);
            }
        }
        es += ga;
        // the products have read the image: write the updated D for the chunk before
        if (n > n_lo) store_images();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base_s, 32);
}

// dk_j = Omega dl^k_j - (1^T dl^k_j) k_j for every token (no dependence between chunks).  grid (ceil(NC / kTcDkChunks), BH),
// 256 threads = 8 warps; Omega staged in shared memory once per kTcDkChunks chunks; the [16 x 128] x [128 x 128]
// product per chunk on warp-level TF32 MMAs.
template <int D, int MF>
__global__ void __launch_bounds__(256)
k_bwd_dk_tc(const bf16 *__restrict__ k, const float *__restrict__ omega, long omega_stride, int m_real, int omega_ld, int H, int T, int NC,
            const float *__restrict__ dl_g, bf16 *__restrict__ dk, int grad32)
{
    constexpr int LDO = MF + 4, LDK = D + 4, LDC = MF + 4, DKC = kTcDkChunks;
    extern __shared__ float sm[];
    float *Os = sm;                        // Omega [D][LDO]
    float *ks = Os + D * LDO;              // [16][LDK]
    float *dl = ks + BC * LDK;             // [16][LDC]
    float *sdl = dl + BC * LDC;            // [16]
    const int bh = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const long seq_off = (long)bh * T * D;
    const float *om = omega + (long)(bh % H) * omega_stride;
    for (int idx = threadIdx.x; idx < D * MF; idx += 256) {
        const int a = idx / MF, p = idx - a * MF;
        Os[a * LDO + p] = (p < m_real) ? om[(long)a * omega_ld + p] : 0.f;   // features beyond m_real are zero padding
    }
    // the chunk's k rows and dl^k rows, fetched one chunk ahead of their use
    const int n_last = min(NC, (int)(blockIdx.x + 1) * DKC);
    uint4 kq;
    float4 dq0, dq1;
    auto fetch = [&](int n) {
        kq = make_uint4(0, 0, 0, 0);
        dq0 = dq1 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (n >= n_last) return;
        if (threadIdx.x < BC * D / 8) {
            const int j = threadIdx.x / (D / 8), c8 = threadIdx.x % (D / 8);
            const int tok = n * BC + j;
            if (tok < T) kq = *(const uint4 *)(k + seq_off + (long)tok * D + c8 * 8);
        }
        if (threadIdx.x < BC * MF / 8) {
            const float4 *src = (const float4 *)(dl_g + ((long)bh * NC + n) * BC * MF) + threadIdx.x * 2;
            dq0 = src[0];
            dq1 = src[1];
        }
    };
    fetch(blockIdx.x * DKC);
    for (int n = blockIdx.x * DKC; n < n_last; ++n) {
        __syncthreads();                   // Omega staged; previous chunk's tiles free
        if (threadIdx.x < BC * D / 8) {
            const int j = threadIdx.x / (D / 8), c8 = threadIdx.x % (D / 8);
            const uint32_t kw[4] = {kq.x, kq.y, kq.z, kq.w};
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                ks[j * LDK + c8 * 8 + 2 * x] = __uint_as_float(kw[x] << 16);
                ks[j * LDK + c8 * 8 + 2 * x + 1] = __uint_as_float(kw[x] & 0xffff0000u);
            }
        }
        if (threadIdx.x < BC * MF / 8) {
            const int j = threadIdx.x / (MF / 8), cc = threadIdx.x % (MF / 8);
            *(float4 *)(dl + j * LDC + cc * 8) = dq0;
            *(float4 *)(dl + j * LDC + cc * 8 + 4) = dq1;
        }
        fetch(n + 1);
        __syncthreads();
        {
            const int j = threadIdx.x >> 4, part = threadIdx.x & 15;
            float s2 = 0.f;
#pragma unroll
            for (int x = 0; x < MF / 16; ++x) s2 += dl[j * LDC + part * (MF / 16) + x];
#pragma unroll
            for (int off = 8; off > 0; off >>= 1) s2 += __shfl_xor_sync(0xffffffffu, s2, off);
            if (part == 0) sdl[j] = s2;
        }
        __syncthreads();
        const int n0 = warp * 16;
        if (n0 < D) {
            float c[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
            warp_gemm16<MF, false, false>(c, dl, LDC, Os, 1, LDO, n0);        // Omega dl : B(k = p, n = a) = Omega[a][p]
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const int j = g + hh * 8, a = n0 + nt * 8 + 2 * t;
                    const int tok = n * BC + j;
                    if (tok < T) {
                        const float2 val = make_float2(c[nt][hh * 2] - sdl[j] * ks[j * LDK + a],
                                                       c[nt][hh * 2 + 1] - sdl[j] * ks[j * LDK + a + 1]);
                        if (grad32) {
                            float2 *dst = (float2 *)((float *)dk + seq_off + (long)tok * D + a);
                            const float2 old = grad32 == 2 ? *dst : make_float2(0.f, 0.f);
                            *dst = make_float2(old.x + val.x, old.y + val.y);
                        } else {
                            *(__nv_bfloat162 *)(dk + seq_off + (long)tok * D + a) = __floats2bfloat162_rn(val.x, val.y);
                        }
                    }
                }
        }
    }
}

// The same product on tcgen05 (used when dk is written as bf16; the fp32-accumulating variant of the feature blocks stays
// on the kernel above).  grid (ceil(tiles / DK5_TILES), BH), 256 threads; a tile is 128 tokens:
//   acc[tok][a] = sum_p dl^k[tok][p] Omega[a][p],   dk = acc - (1^T dl^k[tok]) k[tok]
// dl^k and Omega are split in two bf16 terms each (hi + mid, 16 mantissa bits; the product keeps hi.hi, hi.mid, mid.hi),
// the accumulator sits in tensor memory, the bf16 result is assembled in shared memory and leaves as one bulk store.
static constexpr int DK5_TILES = 8;
template <int D, int MF>
struct Dk5Smem {
    static constexpr int BIMG = D * MF * 2;                    // Omega image [a][p], per 64-wide p block [D][128 B]
    static constexpr int AIMG = 128 * MF * 2;                  // dl^k image [tok][p], per 64-wide p block [128][128 B]
    static constexpr int KS = 128 * D * 2;                     // k rows, 16-byte pieces permuted (piece c at c ^ (row & 7))
    static constexpr int OFF_B = 0, OFF_A = 2 * BIMG, OFF_K = OFF_A + 2 * AIMG, OFF_O = OFF_K + KS, OFF_S = OFF_O + KS;
    static constexpr int TOTAL = OFF_S + 128 * 4;
};

template <int D, int MF>
__global__ void __launch_bounds__(256, 1)
k_bwd_dk_tc5(const bf16 *__restrict__ k, const float *__restrict__ omega, long omega_stride, int m_real, int omega_ld, int H, int T,
             int NC, const float *__restrict__ dl_g, bf16 *__restrict__ dk, int *__restrict__ status)
{
    using S = Dk5Smem<D, MF>;
    extern __shared__ __align__(1024) uint8_t smem_dyn[];
    uint8_t *smem = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
    __shared__ uint64_t bar_mma;
    __shared__ uint32_t tmem_base_s;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.y;
    const long seq_off = (long)bh * T * D;
    const float *om = omega + (long)(bh % H) * omega_stride;
    if (warp == 0) {
        tmem_alloc(&tmem_base_s, 128);
        tmem_relinquish();
    }
    if (tid == 0) {
        mbar_init(&bar_mma, 1);
        fence_barrier_init();
    }
    // rows of fp32 values -> two bf16 terms in a K-major operand image (rows of 64 columns = 128 bytes, 128-byte swizzle)
    auto split_store = [&](uint8_t *hi_img, uint8_t *mid_img, int rows_per_blk, int row, int col, float4 w) {
        const float wv[4] = {w.x, w.y, w.z, w.w};
        uint32_t hh[2], mm[2];
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(wv[2 * x], wv[2 * x + 1]);
            const float2 hf = __bfloat1622float2(h2);
            const __nv_bfloat162 m2 = __floats2bfloat162_rn(wv[2 * x] - hf.x, wv[2 * x + 1] - hf.y);
            hh[x] = *(const uint32_t *)&h2;
            mm[x] = *(const uint32_t *)&m2;
        }
        const uint32_t off = (col >> 6) * (rows_per_blk * 128) + sw_off<128>(row, (col & 63) >> 3) + (col & 4) * 2;
        *(uint2 *)(hi_img + off) = make_uint2(hh[0], hh[1]);
        *(uint2 *)(mid_img + off) = make_uint2(mm[0], mm[1]);
    };
    // Omega [a][p] once per CTA (columns beyond m_real are zero padding)
    for (int idx = tid; idx < D * MF / 4; idx += 256) {
        const int a = idx / (MF / 4), p = (idx % (MF / 4)) * 4;
        const float4 w = (p < m_real) ? *(const float4 *)(om + (long)a * omega_ld + p) : make_float4(0.f, 0.f, 0.f, 0.f);
        split_store(smem + S::OFF_B, smem + S::OFF_B + S::BIMG, D, a, p, w);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = tmem_base_s;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t idesc = make_idesc_f16(128, D, 1, 0, 0);
    float *sdl = (float *)(smem + S::OFF_S);
    const int n_tiles = (T + 127) / 128;
    uint32_t phase = 0;
    bool store_pending = false;
    for (int tile = blockIdx.x * DK5_TILES; tile < min(n_tiles, (int)(blockIdx.x + 1) * DK5_TILES); ++tile) {
        const int tok0 = tile * 128;
        // dl^k rows (fp32, one row per warp and pass: coalesced) -> operand images, row sums.  The loads of eight passes
        // are issued before any is used (a pass per load latency would dominate the tile).
        constexpr int RPP = 256 / (MF / 4);                      // rows per pass
        constexpr int NB = 8;                                    // passes per batch
        const int prow = tid / (MF / 4), q4 = tid % (MF / 4);
        // k rows first: their latency hides behind the conversions
        constexpr int KPT = 128 * (D / 8) / 256;                 // 16-byte pieces of k per thread
        uint4 kreg[KPT];
#pragma unroll
        for (int y = 0; y < KPT; ++y) {
            const int idx = tid + 256 * y;
            const int row = idx / (D / 8), c = idx % (D / 8);
            const int tok = tok0 + row;
            kreg[y] = make_uint4(0, 0, 0, 0);
            if (tok < T) kreg[y] = *(const uint4 *)(k + seq_off + (long)tok * D + c * 8);
        }
        for (int r0 = 0; r0 < 128; r0 += RPP * NB) {
            float4 w[NB];
#pragma unroll
            for (int y = 0; y < NB; ++y) {
                const int tok = tok0 + r0 + y * RPP + prow;
                w[y] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (tok < NC * BC) w[y] = __ldcs((const float4 *)(dl_g + ((long)bh * NC * BC + tok) * MF + q4 * 4));
            }
#pragma unroll
            for (int y = 0; y < NB; ++y) {
                const int row = r0 + y * RPP + prow;
                split_store(smem + S::OFF_A, smem + S::OFF_A + S::AIMG, 128, row, q4 * 4, w[y]);
                float rs = (w[y].x + w[y].y) + (w[y].z + w[y].w);
#pragma unroll
                for (int o_ = (MF / 4) / 2; o_ > 0; o_ >>= 1) rs += __shfl_xor_sync(0xffffffffu, rs, o_);
                if (q4 == 0) sdl[row] = rs;
            }
        }
#pragma unroll
        for (int y = 0; y < KPT; ++y) {
            const int idx = tid + 256 * y;
            const int row = idx / (D / 8), c = idx % (D / 8);
            *(uint4 *)(smem + S::OFF_K + row * (D * 2) + ((c ^ (row & 7)) << 4)) = kreg[y];
        }
        // the output buffer was handed to a bulk store a tile ago
        if (tid == 0 && store_pending) bulk_wait_read<0>();
        fence_proxy_async_smem();
        tc_fence_before();
        __syncthreads();
        if (tid == 0) {
            tc_fence_after();
            const uint64_t da_h = make_smem_desc(smem_u32(smem + S::OFF_A), 0, 1024, kSw128);
            const uint64_t da_m = make_smem_desc(smem_u32(smem + S::OFF_A + S::AIMG), 0, 1024, kSw128);
            const uint64_t db_h = make_smem_desc(smem_u32(smem + S::OFF_B), 0, 1024, kSw128);
            const uint64_t db_m = make_smem_desc(smem_u32(smem + S::OFF_B + S::BIMG), 0, 1024, kSw128);
#pragma unroll
            for (int term = 0; term < 3; ++term) {
                const uint64_t da = term == 2 ? da_m : da_h, db = term == 1 ? db_m : db_h;
#pragma unroll
                for (int ks = 0; ks < MF / 16; ++ks)
                    mma_f16_ss(tm, desc_adv(da, (ks >> 2) * (128 * 128) + (ks & 3) * 32), desc_adv(db, (ks >> 2) * (D * 128) + (ks & 3) * 32),
                               idesc, (term > 0) || (ks > 0));
            }
            tc_commit(&bar_mma);
        }
        mbar_wait(&bar_mma, phase, status, 34);
        phase ^= 1;
        tc_fence_after();
        // epilogue: thread = token row, half of the channels
        {
            const int row = (warp & 3) * 32 + lane, half = warp >> 2;
            const float sd = sdl[row];
            const uint8_t *krow = smem + S::OFF_K + row * (D * 2);
            uint8_t *orow = smem + S::OFF_O + row * (D * 2);
#pragma unroll
            for (int c0 = 0; c0 < D / 2; c0 += 32) {
                uint32_t v[32];
                tmem_ld32(tm + lane_off + half * (D / 2) + c0, v);
                tmem_ld_wait();
#pragma unroll
                for (int c8 = 0; c8 < 4; ++c8) {
                    const int c = (half * (D / 2) + c0) / 8 + c8;            // 16-byte piece of the row
                    const uint4 kq = *(const uint4 *)(krow + ((c ^ (row & 7)) << 4));
                    const uint32_t kw[4] = {kq.x, kq.y, kq.z, kq.w};
                    uint32_t pk[4];
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        const float2 kf = up_bf16(kw[x]);
                        pk[x] = pk_bf16(__uint_as_float(v[c8 * 8 + 2 * x]) - sd * kf.x, __uint_as_float(v[c8 * 8 + 2 * x + 1]) - sd * kf.y);
                    }
                    *(uint4 *)(orow + (c << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                }
            }
        }
        fence_proxy_async_smem();
        tc_fence_before();
        __syncthreads();
        if (tid == 0) {
            const int rows = min(128, T - tok0);
            bulk_s2g(dk + seq_off + (long)tok0 * D, smem + S::OFF_O, rows * D * 2);
            store_pending = true;
        }
    }
    if (tid == 0 && store_pending) bulk_wait_all<0>();
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base_s, 128);
}

// Gradient with respect to the state a continued segment started from: every chunk's state gradient plus what flows into
// the state after the segment.  dS_init [BH][state_m][D] (plain [p][e] order), dz_init [BH][state_m].  grid (BH).
__global__ void __launch_bounds__(256) k_state_grad_total(const float *__restrict__ segsum, int NSEG, int MF, int D, int m_real,
                                                          int state_m, const float *__restrict__ dS_fin,
                                                          const float *__restrict__ dz_fin, float *__restrict__ dS_init,
                                                          float *__restrict__ dz_init)
{
    const int bh = blockIdx.x;
    const long E = (long)MF * D + MF;
    for (int idx = threadIdx.x; idx < m_real * D; idx += 256) {
        const int p = idx / D, e = idx - p * D;
        const int e0 = (((e >> 2) ^ (p & 7)) << 2) | (e & 3);          // where the tile kernel's permuted rows keep channel e
        float acc = dS_fin ? dS_fin[((long)bh * state_m + p) * D + e] : 0.f;
        for (int s2 = 0; s2 < NSEG; ++s2) acc += segsum[((long)bh * NSEG + s2) * E + (long)p * D + e0];
        dS_init[((long)bh * state_m + p) * D + e] = acc;
    }
    for (int p = threadIdx.x; p < m_real; p += 256) {
        float acc = dz_fin ? dz_fin[(long)bh * state_m + p] : 0.f;
        for (int s2 = 0; s2 < NSEG; ++s2) acc += segsum[((long)bh * NSEG + s2) * E + (long)MF * D + p];
        dz_init[(long)bh * state_m + p] = acc;
    }
}

// n is a multiple of 8 (d is 64 or 128) and both buffers are 16-byte aligned
__global__ void k_f32_to_bf16(const float *__restrict__ src, bf16 *__restrict__ dst, long n)
{
    for (long i = ((long)blockIdx.x * blockDim.x + threadIdx.x) * 8; i < n; i += (long)gridDim.x * blockDim.x * 8) {
        const float4 a = __ldcs((const float4 *)(src + i)), b = __ldcs((const float4 *)(src + i + 4));
        *(uint4 *)(dst + i) = make_uint4(pk_bf16(a.x, a.y), pk_bf16(a.z, a.w), pk_bf16(b.x, b.y), pk_bf16(b.z, b.w));
    }
}

template <int D, int MF>
static int bwd_tc_impl(const TcArgs &a, cudaStream_t st)
{
    using S = BwdTcSmem<D, MF>;
    const int NC = (a.T + BC - 1) / BC, BH = a.B * a.H;
    const long E = (long)MF * D + MF;
    const long ntok = (long)BH * a.T * D;
    LaunchScope sc = {st, 0};
    const int n_om = a.omega_stride ? a.H : 1;
    // state pipeline of the forward (boundary images), then the padded Omega image
    TcArgs pre = a;
    pre.state_only = 1;
    pre.S_final = nullptr;
    pre.z_final = nullptr;
    if (!a.reuse_state) {
        const int c0 = tc_fwd_run(pre, st);
        if (c0 < 0) return c0;
        sc.count += c0;
    }
    LS_LAUNCH(sc, "omega_image_tc", k_omega_image_pad_tc<D, MF><<<n_om, 256, 0, st>>>(a.omega, a.m_real, a.omega_ld,
                                                                                     a.omega_stride, a.om_img));
    if (!a.keep_acc) {
        sc.check(cudaMemsetAsync(a.dr_acc, 0, sizeof(float) * ntok, st));
        sc.check(cudaMemsetAsync(a.du_acc, 0, sizeof(float) * ntok, st));
    }
    const long nhist = (long)BH * a.n_hist * D;
    if (a.n_hist > 0) {
        sc.check(cudaMemsetAsync(a.dhr_acc, 0, sizeof(float) * nhist, st));
        sc.check(cudaMemsetAsync(a.dhu_acc, 0, sizeof(float) * nhist, st));
    }
    const int smem = S::TOTAL + 1024;
    const int cpc = a.chunks_per_cta;
    auto launch = [&](auto kern) {
        sc.check(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        LS_LAUNCH(sc, "bwd_tc", kern<<<dim3((NC + cpc - 1) / cpc, BH), BNT, smem, st>>>(
            (const bf16 *)a.q, (const bf16 *)a.r, (const bf16 *)a.u, (const bf16 *)a.dO, a.L, a.lse,
            a.om_img, a.omega_stride != 0, a.H, a.T, a.W, NC, cpc, a.images, a.ab, (bf16 *)a.dq, a.dr_acc, a.du_acc,
            a.gstates, a.dv_intra, a.dchi_intra, a.status, a.delta_ext, a.grad32, a.delta_out, a.seq_lens,
            (const bf16 *)a.hist_r, (const bf16 *)a.hist_u, a.n_hist, a.dhr_acc, a.dhu_acc, a.log2_eps_m, a.images_lo));
    };
    const bool two = a.images_lo != nullptr;
    if (a.delta_out) {
        if (two) launch(k_bwd_tc<D, MF, 2, true>);
        else launch(k_bwd_tc<D, MF, 2, false>);
        return sc.result();                   // first pass of a feature block: only its part of the layer's dO . o
    }
    if (a.delta_ext) {
        if (two) launch(k_bwd_tc<D, MF, 1, true>);
        else launch(k_bwd_tc<D, MF, 1, false>);
    } else if (a.n_hist > 0) {
        if (two) launch(k_bwd_tc<D, MF, 3, true>);
        else launch(k_bwd_tc<D, MF, 3, false>);
    } else {
        if (two) launch(k_bwd_tc<D, MF, 0, true>);
        else launch(k_bwd_tc<D, MF, 0, false>);
    }
    // Segments of the key/value sweep: one wave of CTAs (two per SM) where the sequence is long enough, never shorter
    // than KV_SEG chunks (the workspace holds one partial sum per KV_SEG chunks).
    const int slots = 2 * sm_count();
    const int want = slots / BH > 0 ? slots / BH : 1;
    int seg_len = (NC + want - 1) / want;
    if (seg_len < KV_SEG) seg_len = KV_SEG;
    const int NSEG = (NC + seg_len - 1) / seg_len;
    LS_LAUNCH(sc, "seg_sum_tc", k_seg_sum_tc<<<dim3(NSEG, BH, 4), 256, 0, st>>>(a.gstates, NC, E, a.segsum, seg_len));
    const int kv_smem = sizeof(float) * (MF * (D + 4) + MF + BC * (D + 4) + BC * (MF + 4));
    sc.check(cudaFuncSetAttribute(k_bwd_kv_tc<D, MF>, cudaFuncAttributeMaxDynamicSharedMemorySize, kv_smem));
    if (D == 128 && MF == 128 && !a.grad32) {
        sc.check(cudaFuncSetAttribute(k_bwd_kv_tc5, cudaFuncAttributeMaxDynamicSharedMemorySize, Kv5Smem::TOTAL + 1024));
        LS_LAUNCH(sc, "bwd_kv_tc", k_bwd_kv_tc5<<<dim3(NSEG, BH), 256, Kv5Smem::TOTAL + 1024, st>>>(
            (const bf16 *)a.v, a.T, NC, a.gstates, a.segsum, a.dv_intra, a.dchi_intra, a.chi32, (bf16 *)a.dv, seg_len, a.status,
            a.dS_final, a.dz_final));
    } else {
        LS_LAUNCH(sc, "bwd_kv_tc", k_bwd_kv_tc<D, MF><<<dim3(NSEG, BH), 256, kv_smem, st>>>(
            (const bf16 *)a.v, a.T, NC, a.gstates, a.segsum, a.dv_intra, a.dchi_intra, a.chi32, (bf16 *)a.dv, a.grad32, seg_len,
            a.dS_final, a.dz_final, a.state_m, a.m_real));
    }
    if (a.dS_init)
        LS_LAUNCH(sc, "state_grad_total", k_state_grad_total<<<BH, 256, 0, st>>>(a.segsum, NSEG, MF, D, a.m_real, a.state_m, a.dS_final,
                                                                             a.dz_final, a.dS_init, a.dz_init));
    const int dk_smem = sizeof(float) * (D * (MF + 4) + BC * (D + 4) + BC * (MF + 4) + BC);
    sc.check(cudaFuncSetAttribute(k_bwd_dk_tc<D, MF>, cudaFuncAttributeMaxDynamicSharedMemorySize, dk_smem));
    if (a.grad32) {
        LS_LAUNCH(sc, "bwd_dk_tc", k_bwd_dk_tc<D, MF><<<dim3((NC + kTcDkChunks - 1) / kTcDkChunks, BH), 256, dk_smem, st>>>(
            (const bf16 *)a.k, a.omega, a.omega_stride, a.m_real, a.omega_ld, a.H, a.T, NC, a.chi32, (bf16 *)a.dk, a.grad32));
    } else {
        using S5 = Dk5Smem<D, MF>;
        const int n_tiles = (a.T + 127) / 128;
        sc.check(cudaFuncSetAttribute(k_bwd_dk_tc5<D, MF>, cudaFuncAttributeMaxDynamicSharedMemorySize, S5::TOTAL + 1024));
        LS_LAUNCH(sc, "bwd_dk_tc", k_bwd_dk_tc5<D, MF><<<dim3((n_tiles + DK5_TILES - 1) / DK5_TILES, BH), 256, S5::TOTAL + 1024, st>>>(
            (const bf16 *)a.k, a.omega, a.omega_stride, a.m_real, a.omega_ld, a.H, a.T, NC, a.chi32, (bf16 *)a.dk, a.status));
    }
    if (!a.hold_acc) {
        LS_LAUNCH(sc, "convert_out", k_f32_to_bf16<<<2368, 256, 0, st>>>(a.dr_acc, (bf16 *)a.dr, ntok));
        LS_LAUNCH(sc, "convert_out", k_f32_to_bf16<<<2368, 256, 0, st>>>(a.du_acc, (bf16 *)a.du, ntok));
    }
    if (a.n_hist > 0) {
        LS_LAUNCH(sc, "convert_out", k_f32_to_bf16<<<64, 256, 0, st>>>(a.dhr_acc, (bf16 *)a.d_hist_r, nhist));
        LS_LAUNCH(sc, "convert_out", k_f32_to_bf16<<<64, 256, 0, st>>>(a.dhu_acc, (bf16 *)a.d_hist_u, nhist));
    }
    return sc.result();
}

int tc_bwd_supported(int d, int m) { return (d == 64 || d == 128) && (m == 32 || m == 64 || m == 128); }

int tc_bwd_run(const TcArgs &a, cudaStream_t st)
{
    if (a.d == 64 && a.m == 64) return bwd_tc_impl<64, 64>(a, st);
    if (a.d == 64 && a.m == 128) return bwd_tc_impl<64, 128>(a, st);
    if (a.d == 128 && a.m == 64) return bwd_tc_impl<128, 64>(a, st);
    if (a.d == 128 && a.m == 128) return bwd_tc_impl<128, 128>(a, st);
    return -2;
}

}  // namespace linsimp
