// Feature ranks above 128 on the 128-feature tensor-core kernels: Omega is taken as column blocks of 128 features.
// Eqs. Ni, Zi are sums over the features, so with N_b, Z_b the parts of block b (each computed with its own row
// shift L_b),
//   o = (sum_b N_b) / (sum_b Z_b + eps),   e^{lse_b} = m (Z_b + eps)   =>   o = sum_b o_b w_b / (sum_b w_b - (B-1) m eps)
// with w_b = e^{lse_b}; the blocks' outputs are combined in fp32.  In the backward dN_i and dZ_i are the same for all
// blocks; dZ_i = -(dO_i . o_i)/den_i needs the whole layer's output: the backward tile kernel runs twice per block,
// first in a mode that only adds the block's sum_c psi'_ic . dpsiN_ic (its part of dO_i . o_i den_i, from the very
// operands the gradients are built from, which keeps the cancellation between the numerator and normaliser parts
// exact) to a buffer, then in full with dZ_i taken from that buffer; every gradient is the sum of the blocks'
// gradients (fp32, rounded once).
#include "common.cuh"
#include "launch.cuh"
#include "tc_kernels.h"

namespace linsimp {

static constexpr int kBlk = 128;

// o = sum_b o_b w_b / den, den = sum_b w_b - (nb-1) eps*m, all relative to the largest lse_b.  One thread per output
// element; thread e == 0 of a row also writes the row's L and lse.
__global__ void k_blocks_combine(int nb, const float *__restrict__ o0, const float *__restrict__ o1,
                                 const float *__restrict__ o2, const float *__restrict__ o3,
                                 const float *__restrict__ L0, const float *__restrict__ L1, const float *__restrict__ L2,
                                 const float *__restrict__ L3, const float *__restrict__ s0, const float *__restrict__ s1,
                                 const float *__restrict__ s2, const float *__restrict__ s3, float log_eps_m, float guards_off, long rows, int d,
                                 bf16 *__restrict__ o, float *__restrict__ o_tot, float *__restrict__ Lout,
                                 float *__restrict__ lse)
{
    const float *ob[4] = {o0, o1, o2, o3}, *Lb[4] = {L0, L1, L2, L3}, *sb[4] = {s0, s1, s2, s3};
    for (long idx = (long)blockIdx.x * blockDim.x + threadIdx.x; idx < rows * d; idx += (long)gridDim.x * blockDim.x) {
        const long row = idx / d;
        float M = -INFINITY, Lm = -INFINITY;
        for (int b = 0; b < nb; ++b) {
            M = fmaxf(M, sb[b][row]);
            Lm = fmaxf(Lm, Lb[b][row]);
        }
        float num = 0.f, den = 0.f;
        if (M > -INFINITY) {
            for (int b = 0; b < nb; ++b) {
                const float w = expf(sb[b][row] - M);
                den += w;
                num = fmaf(ob[b][idx], w, num);
            }
            den -= guards_off * expf(log_eps_m - M);           // every w_b carries the guard once
        }
        const float val = den > 0.f ? num / den : 0.f;
        if (o) o[idx] = __float2bfloat16_rn(val);
        if (o_tot) o_tot[idx] = val;
        if (idx == row * d) {
            if (Lout) Lout[row] = Lm > -INFINITY ? Lm : 0.f;
            if (lse) lse[row] = (den > 0.f) ? M + logf(den) : M;
        }
    }
}

__global__ void k_blocks_round(const float *__restrict__ src, bf16 *__restrict__ dst, long n)
{
    for (long i = (long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long)gridDim.x * blockDim.x)
        dst[i] = __float2bfloat16_rn(src[i]);
}

int tc_blocks_supported(int d, int m) { return (d == 64 || d == 128) && m > kBlk && m % kBlk == 0 && m / kBlk <= 4; }

static size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }

size_t tc_blocks_extra_bytes(int B, int H, int T, int d, int m, int op)
{
    const size_t rows = (size_t)B * H * T, nb = m / kBlk;
    size_t n = nb * (up256(rows * d * 4) + 2 * up256(rows * 4));
    if (op == 1) n = up256(rows * 8) + 3 * up256(rows * d * 4);
    return n;
}

void tc_blocks_carve(char *base, int B, int H, int T, int d, int m, int op, TcBlockWs *w)
{
    const size_t rows = (size_t)B * H * T, nb = m / kBlk;
    size_t off = 0;
    for (size_t b = 0; b < 4; ++b) {
        w->o32[b] = w->Lb[b] = w->lseb[b] = nullptr;
        if (b >= nb || op == 1) continue;
        w->o32[b] = (float *)(base + off); off += up256(rows * d * 4);
        w->Lb[b] = (float *)(base + off); off += up256(rows * 4);
        w->lseb[b] = (float *)(base + off); off += up256(rows * 4);
    }
    w->delta = nullptr;
    for (int x = 0; x < 5; ++x) w->g32[x] = nullptr;
    if (op == 1) {
        w->delta = (float *)(base + off); off += up256(rows * 8);
        for (int x = 0; x < 3; ++x) {
            w->g32[x] = (float *)(base + off); off += up256(rows * d * 4);
        }
    }
}

static TcArgs block_args(const TcArgs &a, int m_total, int b)
{
    TcArgs x = a;
    x.m = kBlk;
    x.m_real = kBlk;
    x.omega = a.omega + (long)b * kBlk;
    x.omega_ld = m_total;
    x.state_m = m_total;
    x.p_off = b * kBlk;
    return x;
}

// guards_off: how many copies of the guard eps*m the combined normaliser gives up (feature blocks of one estimator
// keep one of their nb copies; the views of the two-orientation average keep theirs)
static int combine(LaunchScope &sc, const TcArgs &a, int nb, const TcBlockWs &w, float log_eps_m, bf16 *o, float *o_tot,
                   float *L, float *lse, float guards_off)
{
    const long rows = (long)a.B * a.H * a.T;
    LS_LAUNCH(sc, "blocks_combine", k_blocks_combine<<<1184, 256, 0, sc.stream>>>(
        nb, w.o32[0], w.o32[1], w.o32[2], w.o32[3], w.Lb[0], w.Lb[1], w.Lb[2], w.Lb[3], w.lseb[0], w.lseb[1], w.lseb[2],
        w.lseb[3], log_eps_m, guards_off, rows, a.d, o, o_tot, L, lse));
    return 0;
}

// forward of every block (fp32 outputs, own L and lse), then the combination
static int blocks_forward(LaunchScope &sc, const TcArgs &a, int m_total, const TcBlockWs &w, float log_eps_m, bf16 *o,
                          float *o_tot, float *L, float *lse)
{
    const int nb = m_total / kBlk;
    for (int b = 0; b < nb; ++b) {
        TcArgs x = block_args(a, m_total, b);
        x.o32 = w.o32[b];
        x.L = w.Lb[b];
        x.lse = w.lseb[b];
        x.chi32 = nullptr;
        x.images_lo = nullptr;
        const int c = tc_fwd_run(x, sc.stream);
        if (c < 0) return c;
        sc.count += c;
    }
    return combine(sc, a, nb, w, log_eps_m, o, o_tot, L, lse, (float)(nb - 1));
}

int tc_blocks_fwd_run(const TcArgs &a, int m_total, const TcBlockWs &w, float log_eps_m, cudaStream_t st)
{
    LaunchScope sc = {st, 0};
    const int rc = blocks_forward(sc, a, m_total, w, log_eps_m, (bf16 *)a.o, nullptr, a.L, a.lse);
    return rc < 0 ? rc : sc.result();
}

int tc_blocks_state_run(const TcArgs &a, int m_total, cudaStream_t st)
{
    int total = 0;
    for (int b = 0; b < m_total / kBlk; ++b) {
        TcArgs x = block_args(a, m_total, b);
        x.state_only = 1;
        const int c = tc_fwd_run(x, st);
        if (c < 0) return c;
        total += c;
    }
    return total;
}

int tc_blocks_bwd_run(const TcArgs &a, int m_total, const TcBlockWs &w, float log_eps_m, cudaStream_t st)
{
    LaunchScope sc = {st, 0};
    const int nb = m_total / kBlk;
    const long rows = (long)a.B * a.H * a.T, ntok = rows * a.d;
    // first pass per block: the block's part of sum_c psi'_ic . dpsiN_ic (= dO_i . o_i den_i of the layer), from the
    // backward's own tile pipeline, added up over the blocks
    (void)log_eps_m;
    sc.check(cudaMemsetAsync(w.delta, 0, sizeof(float) * 2 * rows, st));
    // The workspace holds the boundary images of one block at a time.  Order of the passes: the first pass starts with
    // the last block (whose images the forward left behind, if the caller says so) and ends with block nb - 2; the
    // second pass starts there, on the images still in place.  Two of the 2 nb pre-passes are saved that way.
    for (int i = 0; i < nb; ++i) {
        const int b = (i == 0) ? nb - 1 : i - 1;
        TcArgs x = block_args(a, m_total, b);
        x.reuse_state = (i == 0) && a.reuse_state && !a.images_lo;   // (the forward's block passes leave no second state term behind)
        x.delta_out = w.delta;
        const int c = tc_bwd_run(x, st);
        if (c < 0) return c;
        sc.count += c;
    }
    for (int i = 0; i < nb; ++i) {
        const int b = (i == 0) ? nb - 2 : (i - 1 < nb - 2 ? i - 1 : i);     // nb - 2 first, then the others
        TcArgs x = block_args(a, m_total, b);
        x.reuse_state = (i == 0);
        x.delta_ext = w.delta;
        x.keep_acc = i > 0;                 // dr, du: all blocks sum into the same fp32 accumulators
        x.hold_acc = i + 1 < nb;
        x.grad32 = i == 0 ? 1 : 2;          // dq, dk, dv: summed over the blocks in fp32 (the blocks' parts cancel in places)
        x.dq = w.g32[0];
        x.dk = w.g32[1];
        x.dv = w.g32[2];
        const int c = tc_bwd_run(x, st);
        if (c < 0) return c;
        sc.count += c;
    }
    LS_LAUNCH(sc, "blocks_round", k_blocks_round<<<1184, 256, 0, st>>>(w.g32[0], (bf16 *)a.dq, ntok));
    LS_LAUNCH(sc, "blocks_round", k_blocks_round<<<1184, 256, 0, st>>>(w.g32[1], (bf16 *)a.dk, ntok));
    LS_LAUNCH(sc, "blocks_round", k_blocks_round<<<1184, 256, 0, st>>>(w.g32[2], (bf16 *)a.dv, ntok));
    return sc.result();
}

// ------------------------------------------------------------------ both orientations of the trilinear score, averaged
// View 1 is the estimator as it stands; view 2 exchanges the two key streams and their values (k <-> r, v <-> u).  The
// kernel estimates are averaged: o = (N1 + N2) / (Z1 + Z2 + 2 eps), which in terms of the views' outputs and
// log-normalisers is the same weighted mean the feature blocks use (every view keeps its guard).  In the backward both
// views share dN_i and dZ_i of the combined estimator: the tile kernel runs per view in its sum-only mode first
// (sum_c psi'_ic . dpsiN_ic of both views = dO_i . o_i den_i), then in full; view 2's gradients return exchanged.
size_t tc_views_extra_bytes(int B, int H, int T, int d, int op)
{
    const size_t rows = (size_t)B * H * T;
    if (op == 1) return up256(rows * 8) + 5 * up256(rows * d * 4);
    return 2 * (up256(rows * d * 4) + 2 * up256(rows * 4));
}

void tc_views_carve(char *base, int B, int H, int T, int d, int op, TcBlockWs *w)
{
    const size_t rows = (size_t)B * H * T;
    size_t off = 0;
    for (int b = 0; b < 4; ++b) w->o32[b] = w->Lb[b] = w->lseb[b] = nullptr;
    w->delta = nullptr;
    for (int x = 0; x < 5; ++x) w->g32[x] = nullptr;
    if (op == 1) {
        w->delta = (float *)(base + off); off += up256(rows * 8);
        for (int x = 0; x < 5; ++x) {
            w->g32[x] = (float *)(base + off); off += up256(rows * d * 4);
        }
        return;
    }
    for (int b = 0; b < 2; ++b) {
        w->o32[b] = (float *)(base + off); off += up256(rows * d * 4);
        w->Lb[b] = (float *)(base + off); off += up256(rows * 4);
        w->lseb[b] = (float *)(base + off); off += up256(rows * 4);
    }
}

static TcArgs view_args(const TcArgs &a, int view)
{
    TcArgs x = a;
    if (view == 1) {
        x.k = a.r; x.r = a.k;
        x.v = a.u; x.u = a.v;
    }
    x.reuse_state = 0;
    x.S_final = view == 0 ? a.S_final : nullptr;        // the state of the (k, v) stream is the one the caller knows
    x.z_final = view == 0 ? a.z_final : nullptr;
    return x;
}

int tc_views_fwd_run(const TcArgs &a, const TcBlockWs &w, float log_eps_m, cudaStream_t st)
{
    LaunchScope sc = {st, 0};
    for (int view = 0; view < 2; ++view) {
        TcArgs x = view_args(a, view);
        x.o32 = w.o32[view];
        x.L = w.Lb[view];
        x.lse = w.lseb[view];
        x.chi32 = nullptr;
        x.images_lo = nullptr;
        const int c = tc_fwd_run(x, st);
        if (c < 0) return c;
        sc.count += c;
    }
    combine(sc, a, 2, w, log_eps_m, (bf16 *)a.o, nullptr, a.L, a.lse, 0.f);
    return sc.result();
}

int tc_views_bwd_run(const TcArgs &a, const TcBlockWs &w, cudaStream_t st)
{
    LaunchScope sc = {st, 0};
    const long rows = (long)a.B * a.H * a.T, ntok = rows * a.d;
    sc.check(cudaMemsetAsync(w.delta, 0, sizeof(float) * 2 * rows, st));
    for (int view = 0; view < 2; ++view) {
        TcArgs x = view_args(a, view);
        x.delta_out = w.delta;
        const int c = tc_bwd_run(x, st);
        if (c < 0) return c;
        sc.count += c;
    }
    // fp32 sums: g32[0..4] = dq, dk, dv, dr, du.  View 1 writes dq, dk, dv and accumulates dr, du; view 2 adds its dq,
    // adds what it calls dk, dv (the gradients of its key stream: r, u) onto dr, du, and accumulates what it calls dr, du
    // onto dk, dv.
    for (int view = 0; view < 2; ++view) {
        TcArgs x = view_args(a, view);
        x.delta_ext = w.delta;
        x.log2_eps_m = a.log2_eps_m + 1.f;       // the combined normaliser carries the guard of both views
        x.grad32 = view == 0 ? 1 : 2;
        x.keep_acc = view == 1;
        x.hold_acc = 1;
        x.dq = w.g32[0];
        x.dk = w.g32[view == 0 ? 1 : 3];
        x.dv = w.g32[view == 0 ? 2 : 4];
        x.dr_acc = w.g32[view == 0 ? 3 : 1];
        x.du_acc = w.g32[view == 0 ? 4 : 2];
        const int c = tc_bwd_run(x, st);
        if (c < 0) return c;
        sc.count += c;
    }
    void *out[5] = {a.dq, a.dk, a.dv, a.dr, a.du};
    for (int x = 0; x < 5; ++x)
        LS_LAUNCH(sc, "blocks_round", k_blocks_round<<<1184, 256, 0, st>>>(w.g32[x], (bf16 *)out[x], ntok));
    return sc.result();
}

}  // namespace linsimp
