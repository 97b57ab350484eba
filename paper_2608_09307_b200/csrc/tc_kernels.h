// Host-side interface of the tensor-core (tcgen05) kernels (internal to the library).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace linsimp {

static const int kTcChunk = 16;      // tokens per chunk of the tensor-core path
static const int kTcKvSeg = 64;      // chunks per segment of the key/value sweep of the backward

struct TcArgs {
    int B, H, T, d, m, W;            // m: feature rank the kernels run with (64 or 128)
    int m_real;                      // caller's feature rank (<= m): Omega is [d][m_real]; features beyond it are zero
    int omega_ld;                    // row stride of Omega in elements (>= m_real: the kernels may work on a column block)
    int state_m, p_off;              // S_final / z_final / S_init / z_init hold state_m features per unit, this call's at p_off
    long omega_stride;               // 0 (shared) or the distance between the heads' banks
    float log2_eps_m;                // log2(eps * m); -inf when eps == 0
    int chunks_per_cta;
    int state_only;                  // run only the pre-pass (prefix state)
    int reuse_state;                 // backward: the boundary images in the workspace are valid, skip the pre-pass
    const void *q, *k, *v, *r, *u;
    const float *omega;
    void *o;                         // forward: out; backward: in
    float *o32;                      // forward: when set, the output goes here in fp32 instead of o
    const float *delta_ext;          // backward: when set, [BH][T] the layer's sum_c psi'_ic . dpsiN_ic to use instead of the block's own,
                                     // followed by [BH][T] the layer's normaliser relative to the forward's
    float *delta_out;                // backward: when set, only those two sums of this block are computed and added there (no gradients)
    int keep_acc, hold_acc;          // backward: do not zero the dr / du accumulators first; do not convert them out at the end
    int grad32;                      // backward: dq, dk, dv point to fp32 buffers; 1 = write them, 2 = add to them
    float *L, *lse;
    float *S_final, *z_final;
    // continuation of a sequence (all nullable / 0): state before the first token, r and u of the n_hist tokens before it
    const float *S_init, *z_init;
    const void *hist_r, *hist_u;
    int n_hist;
    const int *seq_lens;             // [B] device, nullable: tokens at or beyond seq_lens[b] are padding (keys masked, dO taken as 0)
    const void *dO;
    void *dq, *dk, *dv, *dr, *du;
    // workspace pieces
    float *segtot;                   // [BH][8][m/64][128*64 + 64] fp32 per-segment sums of the state walk
    uint8_t *chi_ml;                 // [BH][NC][2][16*m*2] the second and third bf16 term of chi' (chi' operand image layout)
    uint8_t *images;                 // [BH][NC][tc_image_bytes] operand images
    float *ab;                       // [BH][NC][m] exclusive boundary normalisers
    uint8_t *images_lo;              // [BH][NC][128 x m] bf16 (nullable): what the bf16 rounding of each boundary state image leaves,
                                     // in the image's layout; written by the pre-pass for the backward's second state term
    float *chi32;                    // [BH][NC*16][m] fp32 key features chi' (nullable): written by the pre-pass for the
                                     // backward's key/value sweep, which turns it into dl^k in place
    uint8_t *om_img;                 // [n_omega][m*d*2] OmegaT fp16 image
    int *status;                     // device word: first bounded wait that gave up (0 = none)
    // backward only
    float *gstates;                  // [BH][NC][m*d + m] chunk state gradients ([p][e] order)
    float *segsum;                   // [BH][ceil(NC/kTcKvSeg)][m*d + m] per-segment sums of gstates
    float *dv_intra;                 // [BH][NC][16][d]  intra-chunk part of dv
    float *dchi_intra;               // [BH][NC][16][m]  intra-chunk part of d chi'
    float *dr_acc, *du_acc;          // [BH][T][d] fp32 accumulators of the anchor gradients
    // backward of a continued segment (all nullable / 0 otherwise; S_init, z_init, hist_r, hist_u, n_hist as in the forward)
    const float *dS_final, *dz_final;   // gradient flowing into the state after the segment ([BH][state_m][d], [BH][state_m])
    float *dS_init, *dz_init;           // out: gradient with respect to the state the segment started from
    void *d_hist_r, *d_hist_u;          // out: [BH][n_hist][d] gradient with respect to the history anchors
    float *dhr_acc, *dhu_acc;           // [BH][n_hist][d] fp32 accumulators behind them
};

int tc_supported(int d, int m);
size_t tc_image_bytes(int d, int m);
int tc_fwd_run(const TcArgs &a, cudaStream_t st);
int tc_bwd_supported(int d, int m);
int tc_bwd_run(const TcArgs &a, cudaStream_t st);

// Feature ranks above 128 as several 128-feature column blocks of Omega (the numerator and the normaliser are sums
// over the features, so the blocks' results combine exactly).  Workspace pieces beyond the one-block layout:
struct TcBlockWs {
    float *o32[4], *Lb[4], *lseb[4];   // per block: fp32 output, row shift, log-normaliser
    float *delta;                      // backward: [BH][T] dO_i . o_i den_i of the whole layer, then [BH][T] its normaliser relative to the forward's
    float *g32[5];                     // backward: dq, dk, dv (and, for the two views, dr, du) summed in fp32
};
int tc_blocks_supported(int d, int m);
size_t tc_blocks_extra_bytes(int B, int H, int T, int d, int m, int op);
void tc_blocks_carve(char *base, int B, int H, int T, int d, int m, int op, TcBlockWs *w);
int tc_blocks_fwd_run(const TcArgs &a, int m_total, const TcBlockWs &w, float eps_m, cudaStream_t st);
int tc_blocks_state_run(const TcArgs &a, int m_total, cudaStream_t st);
int tc_blocks_bwd_run(const TcArgs &a, int m_total, const TcBlockWs &w, float eps_m, cudaStream_t st);

// Both orientations of the trilinear score averaged (Eq. two-views): the estimator as it stands plus the one with the
// two key streams and their values exchanged, combined through their log-normalisers.
size_t tc_views_extra_bytes(int B, int H, int T, int d, int op);
void tc_views_carve(char *base, int B, int H, int T, int d, int op, TcBlockWs *w);
int tc_views_fwd_run(const TcArgs &a, const TcBlockWs &w, float eps_m, cudaStream_t st);
int tc_views_bwd_run(const TcArgs &a, const TcBlockWs &w, cudaStream_t st);

}  // namespace linsimp
