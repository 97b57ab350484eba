// C ABI of the LinSimp library: argument checks, workspace carving, kernel selection.
#include <math.h>
#include <string.h>

#include <initializer_list>
#include <string>
#include <vector>

#include "../../include/linsimp.h"
#include "common.cuh"
#include "launch.cuh"
#include "norm_gate.h"
#include "packed.h"
#include "simt_kernels.h"
#include "tc_kernels.h"

using namespace linsimp;

namespace linsimp {

thread_local bool g_profile_on = false;

namespace {
struct ProfRecord {
    const char *name;
    cudaEvent_t start, stop;
};
thread_local std::vector<ProfRecord> g_records;
thread_local std::vector<cudaEvent_t> g_event_pool;
thread_local bool g_profile_error = false;

cudaEvent_t take_event()
{
    cudaEvent_t e = nullptr;
    if (!g_event_pool.empty()) {
        e = g_event_pool.back();
        g_event_pool.pop_back();
    } else if (cudaEventCreate(&e) != cudaSuccess) {
        g_profile_error = true;
        e = nullptr;
    }
    return e;
}
}  // namespace

// events recorded into a stream capture cannot be read back: launches under capture are not profiled
static bool capturing(cudaStream_t st)
{
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    return cudaStreamIsCapturing(st, &cs) == cudaSuccess && cs != cudaStreamCaptureStatusNone;
}

void profile_before(const char *name, cudaStream_t st)
{
    if (capturing(st)) return;
    ProfRecord r = {name, take_event(), take_event()};
    if (r.start) cudaEventRecord(r.start, st);
    g_records.push_back(r);
}

void profile_after(cudaStream_t st)
{
    if (capturing(st)) return;
    if (!g_records.empty() && g_records.back().stop) cudaEventRecord(g_records.back().stop, st);
}

}  // namespace linsimp

namespace {

thread_local int g_launches[7] = {0, 0, 0, 0, 0, 0, 0};

bool params_ok(const linsimp_params *p, int op, bool dv_taken = false)
{
    if (!p) return false;
    if (p->dv < 0) return false;
    if (p->dv != 0 && p->dv != p->d) {
        // a value width of its own: forward and backward only, rows of whole 16-byte pieces, no variant on top of it
        if (!dv_taken) return false;
        if (((size_t)p->dv * (p->io_dtype == LINSIMP_F32 ? 4 : 2)) % 16) return false;
        if (p->flags & LINSIMP_FLAG_TWO_VIEWS) return false;
    }
    if (p->B < 1 || p->H < 1 || p->d < 1 || p->m < 1 || p->W < 1) return false;
    if (op != LINSIMP_OP_DECODE && p->T < 1) return false;
    if (op != LINSIMP_OP_DECODE && (long long)p->B * p->H > 65535) return false;   // grid.y limit of the chunked kernels
    if (p->io_dtype != LINSIMP_F32 && p->io_dtype != LINSIMP_BF16) return false;
    if (p->algo != LINSIMP_ALGO_DEFAULT && p->algo != LINSIMP_ALGO_FP32) return false;
    if (!(p->eps >= 0.f)) return false;
    if (p->flags & ~(LINSIMP_FLAG_REUSE_FWD_STATE | LINSIMP_FLAG_OMEGA_IMAGE | LINSIMP_FLAG_TWO_VIEWS | LINSIMP_FLAG_STATE_TWO_TERMS))
        return false;
    if ((p->flags & LINSIMP_FLAG_TWO_VIEWS) && !(op == LINSIMP_OP_FWD || op == LINSIMP_OP_BWD)) return false;
    return true;
}

bool aligned16(const void *p) { return ((uintptr_t)p & 15u) == 0; }

// the normalisation / gate calls use B, H, T, d and io_dtype only
bool norm_shape_ok(const linsimp_params *p)
{
    if (!p || p->B < 1 || p->H < 1 || p->T < 1 || p->d < 1) return false;
    if ((long long)p->B * p->H > 65535) return false;
    return p->io_dtype == LINSIMP_F32 || p->io_dtype == LINSIMP_BF16;
}

NormGateArgs norm_args(const linsimp_params *p)
{
    NormGateArgs a;
    memset(&a, 0, sizeof(a));
    a.B = p->B; a.H = p->H; a.T = p->T; a.d = p->d;
    a.norm_floor = LINSIMP_NORM_FLOOR;
    return a;
}

// `rows`: the [B,H,T,d] streams (16-byte aligned); `heads`: the [H] fp32 arrays (4-byte aligned)
int norm_check(const linsimp_params *p, std::initializer_list<const void *> rows, std::initializer_list<const void *> heads)
{
    if (!norm_shape_ok(p)) return LINSIMP_EINVAL;
    for (const void *x : rows)
        if (!x) return LINSIMP_EINVAL;
    for (const void *x : heads)
        if (!x) return LINSIMP_EINVAL;
    if (!norm_gate_supported(p->d)) return LINSIMP_EUNSUPPORTED;
    for (const void *x : rows)
        if (!aligned16(x)) return LINSIMP_EALIGN;
    for (const void *x : heads)
        if ((uintptr_t)x & 3u) return LINSIMP_EALIGN;
    return LINSIMP_OK;
}

int norm_workspace_check(const linsimp_params *p, const void *workspace, size_t bytes)
{
    if (!workspace || bytes < norm_gate_partial_bytes(p->B, p->H, p->T)) return LINSIMP_EWORKSPACE;
    if ((uintptr_t)workspace & 255u) return LINSIMP_EALIGN;
    return LINSIMP_OK;
}

int decode_banks(const linsimp_params *p) { return p->omega_per_head ? p->H : 1; }

// A shape is served either by the CUDA-core kernels (any io_dtype and algo) or, for feature ranks above 128, by the
// tensor-core feature blocks, which exist for bf16 I/O with the default algo only.
bool shape_supported(const linsimp_params *p)
{
    if (p->W > 64) return false;
    if (simt_supported(p->d, p->m)) return true;
    return p->io_dtype == LINSIMP_BF16 && p->algo == LINSIMP_ALGO_DEFAULT && tc_blocks_supported(p->d, p->m);
}

// feature ranks above 128 (bf16 I/O, default algo): several 128-feature column blocks on the tensor-core kernels
bool use_tc_blocks(const linsimp_params *p, int op)
{
    if (p->io_dtype != LINSIMP_BF16 || p->algo != LINSIMP_ALGO_DEFAULT) return false;
    if (!(op == LINSIMP_OP_FWD || op == LINSIMP_OP_BWD || op == LINSIMP_OP_STATE)) return false;
    return tc_blocks_supported(p->d, p->m) != 0;
}

// bf16 I/O with the default algo runs on the tensor-core kernels where an instance exists (forward, backward and
// prefix state for d in {64,128}, m in {32,64,128}); everything else runs on the fp32 CUDA-core kernels.
bool use_tc(const linsimp_params *p, int op)
{
    if (p->io_dtype != LINSIMP_BF16 || p->algo != LINSIMP_ALGO_DEFAULT) return false;
    if (op == LINSIMP_OP_BWD) return tc_bwd_supported(p->d, p->m) != 0;
    if (!(op == LINSIMP_OP_FWD || op == LINSIMP_OP_STATE)) return false;
    return tc_supported(p->d, p->m) != 0;
}

struct TcLayout {
    size_t status, chi_ml, segtot, images, ab, om_img, chi32, images_lo, gstates, segsum, dv_intra, dchi_intra, dr_acc, du_acc, dhr_acc,
        dhu_acc, total;
};

// feature rank the tensor-core kernels run with: ranks below 64 are zero-padded to 64
int tc_mf(int m) { return m < 64 ? 64 : m; }

TcLayout tc_layout(const linsimp_params *p, int op)
{
    TcLayout L;
    memset(&L, 0, sizeof(L));
    const int mf = tc_mf(p->m);
    const size_t BH = (size_t)p->B * p->H;
    const size_t NC = ((size_t)p->T + kTcChunk - 1) / kTcChunk;
    const size_t E = (size_t)mf * p->d + mf;
    size_t off = 0;
    L.status = off;
    off = 256;
    L.chi_ml = off;
    off = align_up(off + BH * NC * 2 * (size_t)kTcChunk * mf * 2, 1024);
    L.segtot = off;
    off = align_up(off + BH * 8 * (size_t)(mf / 64) * (128 * 64 + 64) * sizeof(float), 1024);
    L.images = off;
    off = align_up(off + BH * NC * tc_image_bytes(p->d, mf), 1024);
    L.ab = off;
    off = align_up(off + BH * NC * mf * sizeof(float), 1024);
    L.om_img = off;
    off = align_up(off + (size_t)(p->omega_per_head ? p->H : 1) * mf * 128 * 2, 1024);
    if (op == LINSIMP_OP_BWD) {
        L.chi32 = off;                       // first, so that a forward given a backward-sized workspace can fill it
        off = align_up(off + BH * NC * kTcChunk * mf * sizeof(float), 1024);
        L.images_lo = off;                   // second, for the same reason
        if (p->flags & LINSIMP_FLAG_STATE_TWO_TERMS) off = align_up(off + BH * NC * (size_t)128 * mf * 2, 1024);
        L.gstates = off;
        off = align_up(off + BH * NC * E * sizeof(float), 1024);
        L.segsum = off;
        off = align_up(off + BH * ((NC + kTcKvSeg - 1) / kTcKvSeg) * E * sizeof(float), 1024);
        L.dv_intra = off;
        off = align_up(off + BH * NC * kTcChunk * p->d * sizeof(float), 1024);
        L.dchi_intra = off;
        off = align_up(off + BH * NC * kTcChunk * mf * sizeof(float), 1024);
        L.dr_acc = off;
        off = align_up(off + BH * p->T * p->d * sizeof(float), 1024);
        L.du_acc = off;
        off = align_up(off + BH * p->T * p->d * sizeof(float), 1024);
        // a continued segment: gradients of up to W - 1 <= 63 history anchors per unit
        L.dhr_acc = off;
        off = align_up(off + BH * 64 * p->d * sizeof(float), 1024);
        L.dhu_acc = off;
        off = align_up(off + BH * 64 * p->d * sizeof(float), 1024);
    }
    L.total = off;
    return L;
}

struct SimtLayout {
    size_t states, gstates, omegaT, dz, dr_acc, du_acc, total;
};

SimtLayout simt_layout(const linsimp_params *p, int op)
{
    SimtLayout L;
    memset(&L, 0, sizeof(L));
    if (op == LINSIMP_OP_DECODE) return L;
    const size_t BH = (size_t)p->B * p->H;
    const size_t NC = ((size_t)p->T + kSimtChunk - 1) / kSimtChunk;
    const size_t E = (size_t)p->m * p->d + p->m;
    size_t off = 0;
    L.states = off;
    off = align_up(off + BH * NC * E * sizeof(float), 256);
    if (op == LINSIMP_OP_BWD) {
        L.gstates = off;
        off = align_up(off + BH * NC * E * sizeof(float), 256);
        L.omegaT = off;
        off = align_up(off + (size_t)(p->omega_per_head ? p->H : 1) * p->m * p->d * sizeof(float), 256);
        L.dz = off;
        off = align_up(off + 2 * BH * p->T * sizeof(float), 256);
        if (p->io_dtype != LINSIMP_F32) {
            L.dr_acc = off;
            off = align_up(off + BH * p->T * p->d * sizeof(float), 256);
            L.du_acc = off;
            off = align_up(off + BH * p->T * p->d * sizeof(float), 256);
        }
    }
    L.total = off;
    return L;
}


float log_eps_m(const linsimp_params *p)
{
    if (p->eps <= 0.f) return -INFINITY;
    return (float)(log((double)p->eps) + log((double)p->m));
}

int finish(int op, int launched)
{
    if (launched == -2) return LINSIMP_EUNSUPPORTED;
    if (launched == -1) return LINSIMP_ECUDA;
    if (cudaPeekAtLastError() != cudaSuccess) return LINSIMP_ECUDA;
    g_launches[op] = launched;
    return LINSIMP_OK;
}

struct TcHistory {
    const float *S_init = nullptr, *z_init = nullptr;
    const void *hist_r = nullptr, *hist_u = nullptr;
    int n_hist = 0;
    const int *seq_lens = nullptr;        // padded batch: the sequences' own lengths
};

int run_tc(const linsimp_params *p, const void *q, const void *k, const void *v, const void *r, const void *u,
           const float *omega, void *o, float *rowmax_L, float *lse, float *S_final, float *z_final, void *workspace,
           size_t workspace_bytes, linsimp_stream stream, int state_only, const TcHistory &hist = TcHistory())
{
    const TcLayout L = tc_layout(p, state_only ? LINSIMP_OP_STATE : LINSIMP_OP_FWD);
    if (!workspace || workspace_bytes < L.total) return LINSIMP_EWORKSPACE;
    if ((uintptr_t)workspace & 255u) return LINSIMP_EALIGN;
    char *ws = (char *)workspace;
    TcArgs a;
    memset(&a, 0, sizeof(a));
    a.B = p->B; a.H = p->H; a.T = p->T; a.d = p->d; a.m = tc_mf(p->m); a.m_real = p->m; a.omega_ld = p->m; a.state_m = p->m; a.p_off = 0; a.W = p->W;
    a.omega_stride = p->omega_per_head ? (long)p->d * p->m : 0;
    a.log2_eps_m = p->eps > 0.f ? (float)(log2((double)p->eps) + log2((double)p->m)) : -INFINITY;
    a.chunks_per_cta = 16;
    a.state_only = state_only;
    a.q = q; a.k = k; a.v = v; a.r = r; a.u = u; a.omega = omega;
    a.o = o; a.L = rowmax_L; a.lse = lse; a.S_final = S_final; a.z_final = z_final;
    a.S_init = hist.S_init; a.z_init = hist.z_init; a.hist_r = hist.hist_r; a.hist_u = hist.hist_u; a.n_hist = hist.n_hist;
    a.seq_lens = hist.seq_lens;
    a.status = (int *)(ws + L.status);
    a.chi_ml = (uint8_t *)(ws + L.chi_ml);
    a.segtot = (float *)(ws + L.segtot);
    a.images = (uint8_t *)(ws + L.images);
    a.ab = (float *)(ws + L.ab);
    a.om_img = (uint8_t *)(ws + L.om_img);
    if (!state_only && use_tc(p, LINSIMP_OP_BWD)) {
        // a workspace of the backward's size: leave the fp32 key features where LINSIMP_FLAG_REUSE_FWD_STATE expects them
        const TcLayout LB = tc_layout(p, LINSIMP_OP_BWD);
        if (workspace_bytes >= LB.total) {
            a.chi32 = (float *)(ws + LB.chi32);
            if (p->flags & LINSIMP_FLAG_STATE_TWO_TERMS) a.images_lo = (uint8_t *)(ws + LB.images_lo);
        }
    }
    if (cudaMemsetAsync(a.status, 0, 256, (cudaStream_t)stream) != cudaSuccess) return LINSIMP_ECUDA;
    const int op = state_only ? LINSIMP_OP_STATE : LINSIMP_OP_FWD;
    return finish(op, tc_fwd_run(a, (cudaStream_t)stream));
}

// what a continued segment adds to the backward's arguments
struct TcBwdHistory {
    const float *S_init = nullptr, *z_init = nullptr;
    const void *hist_r = nullptr, *hist_u = nullptr;
    int n_hist = 0;
    const float *dS_final = nullptr, *dz_final = nullptr;
    float *dS_init = nullptr, *dz_init = nullptr;
    void *d_hist_r = nullptr, *d_hist_u = nullptr;
};

int run_tc_bwd(const linsimp_params *p, const void *q, const void *k, const void *v, const void *r, const void *u,
               const float *omega, const void *o, const float *rowmax_L, const float *lse, const void *dO, void *dq, void *dk,
               void *dv, void *dr, void *du, void *workspace, size_t workspace_bytes, linsimp_stream stream,
               const int *seq_lens, const TcBwdHistory &hist = TcBwdHistory())
{
    const TcLayout TL = tc_layout(p, LINSIMP_OP_BWD);
    if (!workspace || workspace_bytes < TL.total) return LINSIMP_EWORKSPACE;
    if ((uintptr_t)workspace & 255u) return LINSIMP_EALIGN;
    char *tws = (char *)workspace;
    TcArgs a;
    memset(&a, 0, sizeof(a));
    a.B = p->B; a.H = p->H; a.T = p->T; a.d = p->d; a.m = tc_mf(p->m); a.m_real = p->m; a.omega_ld = p->m; a.state_m = p->m; a.p_off = 0; a.W = p->W;
    a.omega_stride = p->omega_per_head ? (long)p->d * p->m : 0;
    a.chunks_per_cta = 16;
    a.log2_eps_m = p->eps > 0.f ? (float)(log2((double)p->eps) + log2((double)p->m)) : -INFINITY;
    // the forward of the same parameters ran on the same kernels, so its boundary images can be taken over
    a.reuse_state = (p->flags & LINSIMP_FLAG_REUSE_FWD_STATE) && use_tc(p, LINSIMP_OP_FWD);
    a.q = q; a.k = k; a.v = v; a.r = r; a.u = u; a.omega = omega;
    a.o = (void *)o; a.L = (float *)rowmax_L; a.lse = (float *)lse; a.dO = dO;
    a.dq = dq; a.dk = dk; a.dv = dv; a.dr = dr; a.du = du;
    a.seq_lens = seq_lens;
    a.status = (int *)(tws + TL.status);
    a.chi_ml = (uint8_t *)(tws + TL.chi_ml);
        a.segtot = (float *)(tws + TL.segtot);
    a.images = (uint8_t *)(tws + TL.images);
    a.ab = (float *)(tws + TL.ab);
    a.om_img = (uint8_t *)(tws + TL.om_img);
    a.chi32 = (float *)(tws + TL.chi32);
    if (p->flags & LINSIMP_FLAG_STATE_TWO_TERMS) a.images_lo = (uint8_t *)(tws + TL.images_lo);
    a.gstates = (float *)(tws + TL.gstates);
    a.segsum = (float *)(tws + TL.segsum);
    a.dv_intra = (float *)(tws + TL.dv_intra);
    a.dchi_intra = (float *)(tws + TL.dchi_intra);
    a.dr_acc = (float *)(tws + TL.dr_acc);
    a.du_acc = (float *)(tws + TL.du_acc);
    a.dhr_acc = (float *)(tws + TL.dhr_acc);
    a.dhu_acc = (float *)(tws + TL.dhu_acc);
    a.S_init = hist.S_init; a.z_init = hist.z_init; a.hist_r = hist.hist_r; a.hist_u = hist.hist_u; a.n_hist = hist.n_hist;
    a.dS_final = hist.dS_final; a.dz_final = hist.dz_final; a.dS_init = hist.dS_init; a.dz_init = hist.dz_init;
    a.d_hist_r = hist.d_hist_r; a.d_hist_u = hist.d_hist_u;
    if (cudaMemsetAsync(a.status, 0, 256, (cudaStream_t)stream) != cudaSuccess) return LINSIMP_ECUDA;
    return finish(LINSIMP_OP_BWD, tc_bwd_run(a, (cudaStream_t)stream));
}

// the two-orientation average runs on the single-block tensor-core kernels
bool views_supported(const linsimp_params *p)
{
    return p->io_dtype == LINSIMP_BF16 && p->algo == LINSIMP_ALGO_DEFAULT && tc_supported(p->d, p->m) && tc_bwd_supported(p->d, p->m);
}

int run_tc_views(int op, const linsimp_params *p, const void *q, const void *k, const void *v, const void *r, const void *u,
                 const float *omega, void *o, float *rowmax_L, float *lse, float *S_final, float *z_final, const void *dO,
                 void *dq, void *dk, void *dv, void *dr, void *du, void *workspace, size_t workspace_bytes, linsimp_stream stream)
{
    const TcLayout L = tc_layout(p, op);
    const size_t base = align_up(L.total, 256);
    if (!workspace || workspace_bytes < base + tc_views_extra_bytes(p->B, p->H, p->T, p->d, op)) return LINSIMP_EWORKSPACE;
    if ((uintptr_t)workspace & 255u) return LINSIMP_EALIGN;
    char *ws = (char *)workspace;
    TcArgs a;
    memset(&a, 0, sizeof(a));
    a.B = p->B; a.H = p->H; a.T = p->T; a.d = p->d; a.m = tc_mf(p->m); a.m_real = p->m; a.omega_ld = p->m; a.state_m = p->m; a.p_off = 0; a.W = p->W;
    a.omega_stride = p->omega_per_head ? (long)p->d * p->m : 0;
    a.log2_eps_m = p->eps > 0.f ? (float)(log2((double)p->eps) + log2((double)p->m)) : -INFINITY;
    a.chunks_per_cta = 16;
    a.q = q; a.k = k; a.v = v; a.r = r; a.u = u; a.omega = omega;
    a.o = o; a.L = rowmax_L; a.lse = lse; a.S_final = S_final; a.z_final = z_final; a.dO = dO;
    a.dq = dq; a.dk = dk; a.dv = dv; a.dr = dr; a.du = du;
    a.status = (int *)(ws + L.status);
    a.chi_ml = (uint8_t *)(ws + L.chi_ml);
    a.segtot = (float *)(ws + L.segtot);
    a.images = (uint8_t *)(ws + L.images);
    a.ab = (float *)(ws + L.ab);
    a.om_img = (uint8_t *)(ws + L.om_img);
    if (op == LINSIMP_OP_BWD) {
        a.chi32 = (float *)(ws + L.chi32);
        if (p->flags & LINSIMP_FLAG_STATE_TWO_TERMS) a.images_lo = (uint8_t *)(ws + L.images_lo);
        a.gstates = (float *)(ws + L.gstates);
        a.segsum = (float *)(ws + L.segsum);
        a.dv_intra = (float *)(ws + L.dv_intra);
        a.dchi_intra = (float *)(ws + L.dchi_intra);
        a.dr_acc = (float *)(ws + L.dr_acc);
        a.du_acc = (float *)(ws + L.du_acc);
    }
    if (cudaMemsetAsync(a.status, 0, 256, (cudaStream_t)stream) != cudaSuccess) return LINSIMP_ECUDA;
    TcBlockWs bw;
    tc_views_carve(ws + base, p->B, p->H, p->T, p->d, op, &bw);
    if (op == LINSIMP_OP_FWD) return finish(op, tc_views_fwd_run(a, bw, log_eps_m(p), (cudaStream_t)stream));
    return finish(op, tc_views_bwd_run(a, bw, (cudaStream_t)stream));
}

// Feature rank above 128: fills the kernel arguments for one 128-feature block layout and runs all blocks.
int run_tc_blocks(int op, const linsimp_params *p, const void *q, const void *k, const void *v, const void *r, const void *u,
                  const float *omega, void *o, float *rowmax_L, float *lse, float *S_final, float *z_final, const void *dO,
                  void *dq, void *dk, void *dv, void *dr, void *du, void *workspace, size_t workspace_bytes,
                  linsimp_stream stream)
{
    linsimp_params pb = *p;
    pb.m = 128;
    const TcLayout L = tc_layout(&pb, op);
    const size_t base = align_up(L.total, 256);
    if (!workspace || workspace_bytes < base + tc_blocks_extra_bytes(p->B, p->H, p->T, p->d, p->m, op)) return LINSIMP_EWORKSPACE;
    if ((uintptr_t)workspace & 255u) return LINSIMP_EALIGN;
    char *ws = (char *)workspace;
    TcArgs a;
    memset(&a, 0, sizeof(a));
    a.B = p->B; a.H = p->H; a.T = p->T; a.d = p->d; a.m = 128; a.m_real = 128; a.W = p->W;
    a.omega_ld = p->m; a.state_m = p->m; a.p_off = 0;
    a.omega_stride = p->omega_per_head ? (long)p->d * p->m : 0;
    a.log2_eps_m = p->eps > 0.f ? (float)(log2((double)p->eps) + log2((double)p->m)) : -INFINITY;
    a.chunks_per_cta = 16;
    a.q = q; a.k = k; a.v = v; a.r = r; a.u = u; a.omega = omega;
    a.o = o; a.L = rowmax_L; a.lse = lse; a.S_final = S_final; a.z_final = z_final; a.dO = dO;
    a.dq = dq; a.dk = dk; a.dv = dv; a.dr = dr; a.du = du;
    a.status = (int *)(ws + L.status);
    a.chi_ml = (uint8_t *)(ws + L.chi_ml);
    a.segtot = (float *)(ws + L.segtot);
    a.images = (uint8_t *)(ws + L.images);
    a.ab = (float *)(ws + L.ab);
    a.om_img = (uint8_t *)(ws + L.om_img);
    if (op == LINSIMP_OP_BWD) {
        // (the forward of the same parameters leaves the last block's boundary images in place)
        a.reuse_state = (p->flags & LINSIMP_FLAG_REUSE_FWD_STATE) != 0;
        a.chi32 = (float *)(ws + L.chi32);
        if (p->flags & LINSIMP_FLAG_STATE_TWO_TERMS) a.images_lo = (uint8_t *)(ws + L.images_lo);
        a.gstates = (float *)(ws + L.gstates);
        a.segsum = (float *)(ws + L.segsum);
        a.dv_intra = (float *)(ws + L.dv_intra);
        a.dchi_intra = (float *)(ws + L.dchi_intra);
        a.dr_acc = (float *)(ws + L.dr_acc);
        a.du_acc = (float *)(ws + L.du_acc);
    }
    if (cudaMemsetAsync(a.status, 0, 256, (cudaStream_t)stream) != cudaSuccess) return LINSIMP_ECUDA;
    TcBlockWs bw;
    tc_blocks_carve(ws + base, p->B, p->H, p->T, p->d, p->m, op, &bw);
    const float lem = log_eps_m(p);
    if (op == LINSIMP_OP_STATE) return finish(op, tc_blocks_state_run(a, p->m, (cudaStream_t)stream));
    if (op == LINSIMP_OP_FWD) return finish(op, tc_blocks_fwd_run(a, p->m, bw, lem, (cudaStream_t)stream));
    return finish(op, tc_blocks_bwd_run(a, p->m, bw, lem, (cudaStream_t)stream));
}

// Packed batches: the inner (padded-batch) workspace first, then the sequences' lengths and the padded copies of the
// token streams (and of the per-row scalars).
struct PackedLayout {
    size_t inner_bytes, lens, rows[11], scal[2], total;
};

PackedLayout packed_layout(const linsimp_params *p, int op)
{
    PackedLayout L;
    memset(&L, 0, sizeof(L));
    const int inner_op = op == LINSIMP_OP_FWD_PACKED ? LINSIMP_OP_FWD : LINSIMP_OP_BWD;
    L.inner_bytes = tc_layout(p, inner_op).total;
    size_t off = align_up(L.inner_bytes, 256);
    L.lens = off;
    off = align_up(off + (size_t)p->B * sizeof(int32_t), 256);
    const size_t nrow = align_up((size_t)p->B * p->H * p->T * p->d * 2, 256);
    const int n_rows = op == LINSIMP_OP_FWD_PACKED ? 6 : 11;
    for (int x = 0; x < n_rows; ++x) {
        L.rows[x] = off;
        off += nrow;
    }
    for (int x = 0; x < 2; ++x) {
        L.scal[x] = off;
        off += align_up((size_t)p->B * p->H * p->T * sizeof(float), 256);
    }
    L.total = off;
    return L;
}

bool packed_supported(const linsimp_params *p)
{
    return p->io_dtype == LINSIMP_BF16 && shape_supported(p) && use_tc(p, LINSIMP_OP_FWD) && use_tc(p, LINSIMP_OP_BWD) &&
           !(p->flags & LINSIMP_FLAG_REUSE_FWD_STATE);
}

bool own_value_width(const linsimp_params *p) { return p->dv != 0 && p->dv != p->d; }

}  // namespace

namespace linsimp {
int winsimp_run(const linsimp_params *p, int w1, const void *q, const void *k, const void *v, const void *r, const void *u, void *o,
                float *lse, cudaStream_t st);
size_t value_width_workspace_bytes(const linsimp_params *p, int op);
int value_width_fwd(const linsimp_params *p, const void *q, const void *k, const void *v, const void *r, const void *u,
                    const float *omega, void *o, float *rowmax_L, float *lse, float *S_final, float *z_final, void *workspace,
                    size_t workspace_bytes, linsimp_stream stream, int *launched);
int value_width_bwd(const linsimp_params *p, const void *q, const void *k, const void *v, const void *r, const void *u,
                    const float *omega, const void *o, const float *rowmax_L, const float *lse, const void *dO, void *dq, void *dk,
                    void *dv, void *dr, void *du, void *workspace, size_t workspace_bytes, linsimp_stream stream, int *launched);
}  // namespace linsimp

extern "C" {

size_t linsimp_workspace_bytes(const linsimp_params *p, int op)
{
    if (p && own_value_width(p))
        return ((op == LINSIMP_OP_FWD || op == LINSIMP_OP_BWD) && params_ok(p, op, true)) ? value_width_workspace_bytes(p, op) : 0;
    if (op == LINSIMP_OP_FWD_PACKED || op == LINSIMP_OP_BWD_PACKED)
        return (params_ok(p, LINSIMP_OP_FWD) && packed_supported(p)) ? packed_layout(p, op).total : 0;
    if (op == LINSIMP_OP_NORM)
        return (norm_shape_ok(p) && norm_gate_supported(p->d)) ? norm_gate_partial_bytes(p->B, p->H, p->T) : 0;
    if (op < 0 || op > 3 || !params_ok(p, op) || !shape_supported(p)) return 0;
    if (p->flags & LINSIMP_FLAG_TWO_VIEWS)
        return views_supported(p) ? align_up(tc_layout(p, op).total, 256) + tc_views_extra_bytes(p->B, p->H, p->T, p->d, op) : 0;
    if (op == LINSIMP_OP_DECODE)
        return (p->io_dtype == LINSIMP_BF16 && p->algo == LINSIMP_ALGO_DEFAULT &&
                decode_mma_supported(p->d, p->m, p->W, decode_banks(p)))
                   ? align_up(decode_mma_image_bytes(p->d, p->m, decode_banks(p)), 256)
                   : 0;
    if (use_tc_blocks(p, op)) {
        linsimp_params pb = *p;
        pb.m = 128;
        return align_up(tc_layout(&pb, op).total, 256) + tc_blocks_extra_bytes(p->B, p->H, p->T, p->d, p->m, op);
    }
    if (use_tc(p, op)) return tc_layout(p, op).total;
    return simt_layout(p, op).total;
}

int linsimp_fwd(const linsimp_params *p, const void *q, const void *k, const void *v, const void *r, const void *u,
                const float *omega, void *o, float *rowmax_L, float *lse, float *S_final, float *z_final,
                void *workspace, size_t workspace_bytes, linsimp_stream stream)
{
    if (!params_ok(p, LINSIMP_OP_FWD, true)) return LINSIMP_EINVAL;
    if (!q || !k || !v || !r || !u || !omega || !o || !rowmax_L || !lse) return LINSIMP_EINVAL;
    if ((S_final == nullptr) != (z_final == nullptr)) return LINSIMP_EINVAL;
    if (!shape_supported(p)) return LINSIMP_EUNSUPPORTED;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(r) || !aligned16(u) || !aligned16(o) ||
        !aligned16(omega))
        return LINSIMP_EALIGN;
    if (own_value_width(p)) {
        int extra = 0;
        const int rc = value_width_fwd(p, q, k, v, r, u, omega, o, rowmax_L, lse, S_final, z_final, workspace, workspace_bytes, stream, &extra);
        if (rc == LINSIMP_OK) g_launches[LINSIMP_OP_FWD] = g_launches[LINSIMP_OP_FWD] * ((p->dv + p->d - 1) / p->d) + extra;
        return rc;
    }
    if (p->flags & LINSIMP_FLAG_TWO_VIEWS) {
        if (!views_supported(p)) return LINSIMP_EUNSUPPORTED;
        return run_tc_views(LINSIMP_OP_FWD, p, q, k, v, r, u, omega, o, rowmax_L, lse, S_final, z_final, nullptr, nullptr, nullptr,
                            nullptr, nullptr, nullptr, workspace, workspace_bytes, stream);
    }
    if (use_tc_blocks(p, LINSIMP_OP_FWD))
        return run_tc_blocks(LINSIMP_OP_FWD, p, q, k, v, r, u, omega, o, rowmax_L, lse, S_final, z_final, nullptr, nullptr,
                             nullptr, nullptr, nullptr, nullptr, workspace, workspace_bytes, stream);
    if (use_tc(p, LINSIMP_OP_FWD))
        return run_tc(p, q, k, v, r, u, omega, o, rowmax_L, lse, S_final, z_final, workspace, workspace_bytes, stream, 0);
    const SimtLayout L = simt_layout(p, LINSIMP_OP_FWD);
    if (!workspace || workspace_bytes < L.total) return LINSIMP_EWORKSPACE;
    if ((uintptr_t)workspace & 255u) return LINSIMP_EALIGN;
    char *ws = (char *)workspace;
    SimtArgs a;
    memset(&a, 0, sizeof(a));
    a.B = p->B; a.H = p->H; a.T = p->T; a.d = p->d; a.m = p->m; a.W = p->W; a.C = kSimtChunk;
    a.omega_stride = p->omega_per_head ? (long)p->d * p->m : 0;
    a.log_eps_m = log_eps_m(p);
    a.q = q; a.k = k; a.v = v; a.r = r; a.u = u; a.omega = omega;
    a.o = o; a.L = rowmax_L; a.lse = lse; a.S_final = S_final; a.z_final = z_final;
    a.states = (float *)(ws + L.states);
    return finish(LINSIMP_OP_FWD, simt_run(LINSIMP_OP_FWD, p->io_dtype, a, (cudaStream_t)stream));
}

int linsimp_fwd_continue(const linsimp_params *p, const void *q, const void *k, const void *v, const void *r,
                         const void *u, const float *omega, const float *S_init, const float *z_init,
                         const void *hist_r, const void *hist_u, int32_t n_hist, void *o, float *rowmax_L, float *lse,
                         float *S_final, float *z_final, void *workspace, size_t workspace_bytes, linsimp_stream stream)
{
    if (!params_ok(p, LINSIMP_OP_FWD)) return LINSIMP_EINVAL;
    if (!q || !k || !v || !r || !u || !omega || !o || !rowmax_L || !lse) return LINSIMP_EINVAL;
    if ((S_final == nullptr) != (z_final == nullptr) || (S_init == nullptr) != (z_init == nullptr)) return LINSIMP_EINVAL;
    if (n_hist < 0 || n_hist > p->W - 1 || (n_hist > 0 && (!hist_r || !hist_u))) return LINSIMP_EINVAL;
    if (!shape_supported(p) || !use_tc(p, LINSIMP_OP_FWD)) return LINSIMP_EUNSUPPORTED;
    const void *ptrs[] = {q, k, v, r, u, o, omega, S_init, z_init, hist_r, hist_u};
    for (const void *x : ptrs)
        if (x && !aligned16(x)) return LINSIMP_EALIGN;
    TcHistory h;
    h.S_init = S_init; h.z_init = z_init; h.hist_r = hist_r; h.hist_u = hist_u; h.n_hist = n_hist;
    return run_tc(p, q, k, v, r, u, omega, o, rowmax_L, lse, S_final, z_final, workspace, workspace_bytes, stream, 0, h);
}

int linsimp_bwd_continue(const linsimp_params *p, const void *q, const void *k, const void *v, const void *r, const void *u,
                         const float *omega, const float *S_init, const float *z_init, const void *hist_r,
                         const void *hist_u, int32_t n_hist, const float *rowmax_L, const float *lse, const void *dO,
                         const float *dS_final, const float *dz_final, void *dq, void *dk, void *dv, void *dr, void *du,
                         void *d_hist_r, void *d_hist_u, float *dS_init, float *dz_init, void *workspace,
                         size_t workspace_bytes, linsimp_stream stream)
{
    if (!params_ok(p, LINSIMP_OP_BWD)) return LINSIMP_EINVAL;
    if (!q || !k || !v || !r || !u || !omega || !rowmax_L || !lse || !dO || !dq || !dk || !dv || !dr || !du) return LINSIMP_EINVAL;
    if ((S_init == nullptr) != (z_init == nullptr) || (dS_final == nullptr) != (dz_final == nullptr) ||
        (dS_init == nullptr) != (dz_init == nullptr))
        return LINSIMP_EINVAL;
    if (n_hist < 0 || n_hist > p->W - 1 || (n_hist > 0 && (!hist_r || !hist_u || !d_hist_r || !d_hist_u))) return LINSIMP_EINVAL;
    if (p->flags & LINSIMP_FLAG_REUSE_FWD_STATE) return LINSIMP_EINVAL;      // the segment's pre-pass always runs
    if (!shape_supported(p) || !use_tc(p, LINSIMP_OP_BWD)) return LINSIMP_EUNSUPPORTED;
    const void *ptrs[] = {q, k, v, r, u, omega, dO, dq, dk, dv, dr, du, S_init, z_init, hist_r, hist_u, dS_final, dz_final,
                          d_hist_r, d_hist_u, dS_init, dz_init};
    for (const void *x : ptrs)
        if (x && !aligned16(x)) return LINSIMP_EALIGN;
    TcBwdHistory h;
    h.S_init = S_init; h.z_init = z_init; h.hist_r = hist_r; h.hist_u = hist_u; h.n_hist = n_hist;
    h.dS_final = dS_final; h.dz_final = dz_final; h.dS_init = dS_init; h.dz_init = dz_init;
    h.d_hist_r = d_hist_r; h.d_hist_u = d_hist_u;
    return run_tc_bwd(p, q, k, v, r, u, omega, nullptr, rowmax_L, lse, dO, dq, dk, dv, dr, du, workspace, workspace_bytes, stream,
                      nullptr, h);
}

int linsimp_ring_fill(const linsimp_params *p, const void *r, const void *u, int64_t t_first, void *ring_r, void *ring_u,
                      linsimp_stream stream)
{
    if (!params_ok(p, LINSIMP_OP_FWD) || !r || !u || !ring_r || !ring_u || t_first < 0) return LINSIMP_EINVAL;
    if (p->W > 64) return LINSIMP_EUNSUPPORTED;
    if (!aligned16(r) || !aligned16(u) || !aligned16(ring_r) || !aligned16(ring_u)) return LINSIMP_EALIGN;
    return finish(LINSIMP_OP_STATE, ring_fill_run(p->B * p->H, p->T, p->d, p->W, p->io_dtype == LINSIMP_F32 ? 4 : 2, r, u,
                                                  (long long)t_first, ring_r, ring_u, nullptr, p->H, (cudaStream_t)stream));
}

int linsimp_fwd_padded(const linsimp_params *p, const void *q, const void *k, const void *v, const void *r, const void *u,
                       const float *omega, const int32_t *seq_lens, void *o, float *rowmax_L, float *lse, float *S_final,
                       float *z_final, void *workspace, size_t workspace_bytes, linsimp_stream stream)
{
    if (!params_ok(p, LINSIMP_OP_FWD)) return LINSIMP_EINVAL;
    if (!q || !k || !v || !r || !u || !omega || !o || !rowmax_L || !lse || !seq_lens) return LINSIMP_EINVAL;
    if ((S_final == nullptr) != (z_final == nullptr)) return LINSIMP_EINVAL;
    if (!shape_supported(p) || !use_tc(p, LINSIMP_OP_FWD)) return LINSIMP_EUNSUPPORTED;
    const void *ptrs[] = {q, k, v, r, u, o, omega};
    for (const void *x : ptrs)
        if (!aligned16(x)) return LINSIMP_EALIGN;
    if ((uintptr_t)seq_lens & 3u) return LINSIMP_EALIGN;
    TcHistory h;
    h.seq_lens = seq_lens;
    return run_tc(p, q, k, v, r, u, omega, o, rowmax_L, lse, S_final, z_final, workspace, workspace_bytes, stream, 0, h);
}

int linsimp_bwd_padded(const linsimp_params *p, const void *q, const void *k, const void *v, const void *r, const void *u,
                       const float *omega, const int32_t *seq_lens, const void *o, const float *rowmax_L, const float *lse,
                       const void *dO, void *dq, void *dk, void *dv, void *dr, void *du, void *workspace,
                       size_t workspace_bytes, linsimp_stream stream)
{
    if (!params_ok(p, LINSIMP_OP_BWD)) return LINSIMP_EINVAL;
    if (!q || !k || !v || !r || !u || !omega || !o || !rowmax_L || !lse || !dO || !dq || !dk || !dv || !dr || !du || !seq_lens)
        return LINSIMP_EINVAL;
    if (!shape_supported(p) || !use_tc(p, LINSIMP_OP_BWD)) return LINSIMP_EUNSUPPORTED;
    const void *ptrs[] = {q, k, v, r, u, omega, o, dO, dq, dk, dv, dr, du};
    for (const void *x : ptrs)
        if (!aligned16(x)) return LINSIMP_EALIGN;
    if ((uintptr_t)seq_lens & 3u) return LINSIMP_EALIGN;
    return run_tc_bwd(p, q, k, v, r, u, omega, o, rowmax_L, lse, dO, dq, dk, dv, dr, du, workspace, workspace_bytes, stream,
                      seq_lens);
}

int linsimp_winsimp_fwd(const linsimp_params *p, int32_t w1, const void *q, const void *k, const void *v, const void *r,
                        const void *u, void *o, float *lse, linsimp_stream stream)
{
    if (!p || p->B < 1 || p->H < 1 || p->T < 1 || p->W < 1 || w1 < 1 || (long long)p->B * p->H > 65535) return LINSIMP_EINVAL;
    if (!q || !k || !v || !r || !u || !o) return LINSIMP_EINVAL;
    if ((p->dv != 0 && p->dv != p->d) || p->flags) return LINSIMP_EINVAL;
    if (p->io_dtype != LINSIMP_BF16 || !(p->d == 64 || p->d == 128) || p->W > 32) return LINSIMP_EUNSUPPORTED;
    const void *ptrs[] = {q, k, v, r, u, o};
    for (const void *x : ptrs)
        if (!aligned16(x)) return LINSIMP_EALIGN;
    if ((uintptr_t)lse & 3u) return LINSIMP_EALIGN;
    return finish(LINSIMP_OP_FWD, winsimp_run(p, w1, q, k, v, r, u, o, lse, (cudaStream_t)stream));
}

int linsimp_fwd_packed(const linsimp_params *p, const void *q, const void *k, const void *v, const void *r, const void *u,
                       const float *omega, const int32_t *cu_seqlens, int64_t total_tokens, void *o, float *rowmax_L, float *lse,
                       float *S_final, float *z_final, void *workspace, size_t workspace_bytes, linsimp_stream stream)
{
    if (!params_ok(p, LINSIMP_OP_FWD)) return LINSIMP_EINVAL;
    if (!q || !k || !v || !r || !u || !omega || !o || !rowmax_L || !lse || !cu_seqlens || total_tokens < 0) return LINSIMP_EINVAL;
    if ((S_final == nullptr) != (z_final == nullptr)) return LINSIMP_EINVAL;
    if (p->flags & LINSIMP_FLAG_REUSE_FWD_STATE) return LINSIMP_EINVAL;
    if (!packed_supported(p)) return LINSIMP_EUNSUPPORTED;
    const void *ptrs[] = {q, k, v, r, u, o, omega};
    for (const void *x : ptrs)
        if (!aligned16(x)) return LINSIMP_EALIGN;
    if ((uintptr_t)cu_seqlens & 3u) return LINSIMP_EALIGN;
    const PackedLayout L = packed_layout(p, LINSIMP_OP_FWD_PACKED);
    if (!workspace || workspace_bytes < L.total) return LINSIMP_EWORKSPACE;
    if ((uintptr_t)workspace & 255u) return LINSIMP_EALIGN;
    char *ws = (char *)workspace;
    cudaStream_t st = (cudaStream_t)stream;
    int32_t *lens = (int32_t *)(ws + L.lens);
    int launched = 0;
    auto add = [&](int c) { if (c < 0) launched = -1; else if (launched >= 0) launched += c; };
    add(packed_lens_run(cu_seqlens, p->B, p->T, lens, st));
    const void *in[5] = {q, k, v, r, u};
    for (int x = 0; x < 5; ++x) add(packed_unpack_run(in[x], cu_seqlens, p->B, p->H, p->T, total_tokens, p->d, 2, ws + L.rows[x], st));
    if (launched < 0) return LINSIMP_ECUDA;
    const int rc = linsimp_fwd_padded(p, ws + L.rows[0], ws + L.rows[1], ws + L.rows[2], ws + L.rows[3], ws + L.rows[4], omega, lens,
                                      ws + L.rows[5], (float *)(ws + L.scal[0]), (float *)(ws + L.scal[1]), S_final, z_final, ws,
                                      L.inner_bytes, stream);
    if (rc != LINSIMP_OK) return rc;
    launched += g_launches[LINSIMP_OP_FWD];
    add(packed_pack_run(ws + L.rows[5], cu_seqlens, p->B, p->H, p->T, total_tokens, p->d, 2, o, st));
    add(packed_pack_run(ws + L.scal[0], cu_seqlens, p->B, p->H, p->T, total_tokens, 1, 4, rowmax_L, st));
    add(packed_pack_run(ws + L.scal[1], cu_seqlens, p->B, p->H, p->T, total_tokens, 1, 4, lse, st));
    return finish(LINSIMP_OP_FWD_PACKED, launched);
}

int linsimp_bwd_packed(const linsimp_params *p, const void *q, const void *k, const void *v, const void *r, const void *u,
                       const float *omega, const int32_t *cu_seqlens, int64_t total_tokens, const float *rowmax_L, const float *lse,
                       const void *dO, void *dq, void *dk, void *dv, void *dr, void *du, void *workspace, size_t workspace_bytes,
                       linsimp_stream stream)
{
    if (!params_ok(p, LINSIMP_OP_BWD)) return LINSIMP_EINVAL;
    if (!q || !k || !v || !r || !u || !omega || !rowmax_L || !lse || !dO || !dq || !dk || !dv || !dr || !du || !cu_seqlens ||
        total_tokens < 0)
        return LINSIMP_EINVAL;
    if (p->flags & LINSIMP_FLAG_REUSE_FWD_STATE) return LINSIMP_EINVAL;
    if (!packed_supported(p)) return LINSIMP_EUNSUPPORTED;
    const void *ptrs[] = {q, k, v, r, u, omega, dO, dq, dk, dv, dr, du};
    for (const void *x : ptrs)
        if (!aligned16(x)) return LINSIMP_EALIGN;
    if (((uintptr_t)cu_seqlens & 3u) || ((uintptr_t)rowmax_L & 3u) || ((uintptr_t)lse & 3u)) return LINSIMP_EALIGN;
    const PackedLayout L = packed_layout(p, LINSIMP_OP_BWD_PACKED);
    if (!workspace || workspace_bytes < L.total) return LINSIMP_EWORKSPACE;
    if ((uintptr_t)workspace & 255u) return LINSIMP_EALIGN;
    char *ws = (char *)workspace;
    cudaStream_t st = (cudaStream_t)stream;
    int32_t *lens = (int32_t *)(ws + L.lens);
    int launched = 0;
    auto add = [&](int c) { if (c < 0) launched = -1; else if (launched >= 0) launched += c; };
    add(packed_lens_run(cu_seqlens, p->B, p->T, lens, st));
    const void *in[6] = {q, k, v, r, u, dO};
    for (int x = 0; x < 6; ++x) add(packed_unpack_run(in[x], cu_seqlens, p->B, p->H, p->T, total_tokens, p->d, 2, ws + L.rows[x], st));
    add(packed_unpack_run(rowmax_L, cu_seqlens, p->B, p->H, p->T, total_tokens, 1, 4, ws + L.scal[0], st));
    add(packed_unpack_run(lse, cu_seqlens, p->B, p->H, p->T, total_tokens, 1, 4, ws + L.scal[1], st));
    if (launched < 0) return LINSIMP_ECUDA;
    // (the output argument of the padded backward is not read: any valid pointer will do)
    const int rc = linsimp_bwd_padded(p, ws + L.rows[0], ws + L.rows[1], ws + L.rows[2], ws + L.rows[3], ws + L.rows[4], omega, lens,
                                      ws + L.rows[5], (const float *)(ws + L.scal[0]), (const float *)(ws + L.scal[1]), ws + L.rows[5],
                                      ws + L.rows[6], ws + L.rows[7], ws + L.rows[8], ws + L.rows[9], ws + L.rows[10], ws,
                                      L.inner_bytes, stream);
    if (rc != LINSIMP_OK) return rc;
    launched += g_launches[LINSIMP_OP_BWD];
    void *out[5] = {dq, dk, dv, dr, du};
    for (int x = 0; x < 5; ++x) add(packed_pack_run(ws + L.rows[6 + x], cu_seqlens, p->B, p->H, p->T, total_tokens, p->d, 2, out[x], st));
    return finish(LINSIMP_OP_BWD_PACKED, launched);
}

int linsimp_ring_fill_packed(const linsimp_params *p, const void *r, const void *u, const int32_t *cu_seqlens, int64_t total_tokens,
                             void *ring_r, void *ring_u, linsimp_stream stream)
{
    if (!params_ok(p, LINSIMP_OP_FWD) || !r || !u || !ring_r || !ring_u || !cu_seqlens || total_tokens < 0) return LINSIMP_EINVAL;
    if (p->W > 64) return LINSIMP_EUNSUPPORTED;
    if (!aligned16(r) || !aligned16(u) || !aligned16(ring_r) || !aligned16(ring_u) || ((uintptr_t)cu_seqlens & 3u)) return LINSIMP_EALIGN;
    return finish(LINSIMP_OP_STATE, packed_ring_fill_run(r, u, cu_seqlens, p->B, p->H, total_tokens, p->d, p->W,
                                                         p->io_dtype == LINSIMP_F32 ? 4 : 2, ring_r, ring_u, (cudaStream_t)stream));
}

int linsimp_ring_fill_padded(const linsimp_params *p, const void *r, const void *u, const int32_t *seq_lens, void *ring_r,
                             void *ring_u, linsimp_stream stream)
{
    if (!params_ok(p, LINSIMP_OP_FWD) || !r || !u || !ring_r || !ring_u || !seq_lens) return LINSIMP_EINVAL;
    if (p->W > 64) return LINSIMP_EUNSUPPORTED;
    if (!aligned16(r) || !aligned16(u) || !aligned16(ring_r) || !aligned16(ring_u) || ((uintptr_t)seq_lens & 3u)) return LINSIMP_EALIGN;
    return finish(LINSIMP_OP_STATE, ring_fill_run(p->B * p->H, p->T, p->d, p->W, p->io_dtype == LINSIMP_F32 ? 4 : 2, r, u, 0, ring_r,
                                                  ring_u, seq_lens, p->H, (cudaStream_t)stream));
}

int linsimp_bwd(const linsimp_params *p, const void *q, const void *k, const void *v, const void *r, const void *u,
                const float *omega, const void *o, const float *rowmax_L, const float *lse, const void *dO,
                void *dq, void *dk, void *dv, void *dr, void *du, void *workspace, size_t workspace_bytes,
                linsimp_stream stream)
{
    if (!params_ok(p, LINSIMP_OP_BWD, true)) return LINSIMP_EINVAL;
    if (!q || !k || !v || !r || !u || !omega || !o || !rowmax_L || !lse || !dO || !dq || !dk || !dv || !dr || !du)
        return LINSIMP_EINVAL;
    if (!shape_supported(p)) return LINSIMP_EUNSUPPORTED;
    const void *ptrs[] = {q, k, v, r, u, omega, o, dO, dq, dk, dv, dr, du};
    for (const void *x : ptrs)
        if (!aligned16(x)) return LINSIMP_EALIGN;
    if (own_value_width(p)) {
        int extra = 0;
        const int rc = value_width_bwd(p, q, k, v, r, u, omega, o, rowmax_L, lse, dO, dq, dk, dv, dr, du, workspace, workspace_bytes,
                                       stream, &extra);
        if (rc == LINSIMP_OK) g_launches[LINSIMP_OP_BWD] = g_launches[LINSIMP_OP_BWD] * ((p->dv + p->d - 1) / p->d) + extra;
        return rc;
    }
    if (p->flags & LINSIMP_FLAG_TWO_VIEWS) {
        if (!views_supported(p)) return LINSIMP_EUNSUPPORTED;
        return run_tc_views(LINSIMP_OP_BWD, p, q, k, v, r, u, omega, (void *)o, (float *)rowmax_L, (float *)lse, nullptr, nullptr,
                            dO, dq, dk, dv, dr, du, workspace, workspace_bytes, stream);
    }
    if (use_tc_blocks(p, LINSIMP_OP_BWD))
        return run_tc_blocks(LINSIMP_OP_BWD, p, q, k, v, r, u, omega, (void *)o, (float *)rowmax_L, (float *)lse, nullptr,
                             nullptr, dO, dq, dk, dv, dr, du, workspace, workspace_bytes, stream);
    if (use_tc(p, LINSIMP_OP_BWD))
        return run_tc_bwd(p, q, k, v, r, u, omega, o, rowmax_L, lse, dO, dq, dk, dv, dr, du, workspace, workspace_bytes, stream,
                          nullptr);
    const SimtLayout L = simt_layout(p, LINSIMP_OP_BWD);
    if (!workspace || workspace_bytes < L.total) return LINSIMP_EWORKSPACE;
    if ((uintptr_t)workspace & 255u) return LINSIMP_EALIGN;
    char *ws = (char *)workspace;
    SimtArgs a;
    memset(&a, 0, sizeof(a));
    a.B = p->B; a.H = p->H; a.T = p->T; a.d = p->d; a.m = p->m; a.W = p->W; a.C = kSimtChunk;
    a.omega_stride = p->omega_per_head ? (long)p->d * p->m : 0;
    a.log_eps_m = log_eps_m(p);
    a.q = q; a.k = k; a.v = v; a.r = r; a.u = u; a.omega = omega;
    a.o = (void *)o; a.L = (float *)rowmax_L; a.lse = (float *)lse; a.dO = dO;
    a.dq = dq; a.dk = dk; a.dv = dv; a.dr = dr; a.du = du;
    a.states = (float *)(ws + L.states);
    a.reuse_state = (p->flags & LINSIMP_FLAG_REUSE_FWD_STATE) && !use_tc(p, LINSIMP_OP_FWD);
    a.gstates = (float *)(ws + L.gstates);
    a.omegaT = (float *)(ws + L.omegaT);
    a.dz = (float *)(ws + L.dz);
    if (p->io_dtype == LINSIMP_F32) {
        a.dr_acc = (float *)dr;
        a.du_acc = (float *)du;
    } else {
        a.dr_acc = (float *)(ws + L.dr_acc);
        a.du_acc = (float *)(ws + L.du_acc);
    }
    return finish(LINSIMP_OP_BWD, simt_run(LINSIMP_OP_BWD, p->io_dtype, a, (cudaStream_t)stream));
}

int linsimp_decode_step(const linsimp_params *p, const void *q_t, const void *k_t, const void *v_t,
                        const void *r_t, const void *u_t, const float *omega, float *S, float *z, void *ring_r,
                        void *ring_u, const int32_t *pos, void *o_t, void *workspace, size_t workspace_bytes,
                        linsimp_stream stream)
{
    (void)workspace;
    (void)workspace_bytes;
    if (!params_ok(p, LINSIMP_OP_DECODE)) return LINSIMP_EINVAL;
    if (!q_t || !k_t || !v_t || !r_t || !u_t || !omega || !S || !z || !ring_r || !ring_u || !pos || !o_t)
        return LINSIMP_EINVAL;
    if (!shape_supported(p)) return LINSIMP_EUNSUPPORTED;
    const void *ptrs[] = {q_t, k_t, v_t, r_t, u_t, omega, S, z, ring_r, ring_u, o_t};
    for (const void *x : ptrs)
        if (!aligned16(x)) return LINSIMP_EALIGN;
    SimtArgs a;
    memset(&a, 0, sizeof(a));
    a.B = p->B; a.H = p->H; a.T = 0; a.d = p->d; a.m = p->m; a.W = p->W; a.C = kSimtChunk;
    a.omega_stride = p->omega_per_head ? (long)p->d * p->m : 0;
    a.log_eps_m = log_eps_m(p);
    a.q = q_t; a.k = k_t; a.v = v_t; a.r = r_t; a.u = u_t; a.omega = omega;
    a.o = o_t; a.S_final = S; a.z_final = z; a.ring_r = ring_r; a.ring_u = ring_u; a.pos = pos;
    if (p->io_dtype == LINSIMP_BF16 && p->algo == LINSIMP_ALGO_DEFAULT &&
        decode_mma_supported(p->d, p->m, p->W, decode_banks(p))) {
        const void *image = nullptr;
        if (p->flags & LINSIMP_FLAG_OMEGA_IMAGE) {
            if (!workspace || workspace_bytes < decode_mma_image_bytes(p->d, p->m, decode_banks(p))) return LINSIMP_EWORKSPACE;
            if ((uintptr_t)workspace & 255u) return LINSIMP_EALIGN;
            image = workspace;
        }
        return finish(LINSIMP_OP_DECODE, decode_mma_run(a, image, (cudaStream_t)stream));
    }
    return finish(LINSIMP_OP_DECODE, simt_run(LINSIMP_OP_DECODE, p->io_dtype, a, (cudaStream_t)stream));
}

int linsimp_qkr_normalize(const linsimp_params *p, const void *q, const void *k, const void *r, const float *tau,
                          void *q_hat, void *k_hat, void *r_hat, linsimp_stream stream)
{
    const int rc = norm_check(p, {q, k, r, q_hat, k_hat, r_hat}, {tau});
    if (rc != LINSIMP_OK) return rc;
    NormGateArgs a = norm_args(p);
    a.q = q; a.k = k; a.r = r; a.tau = tau; a.qh = q_hat; a.kh = k_hat; a.rh = r_hat;
    return finish(LINSIMP_OP_NORM, norm_gate_run(0, p->io_dtype == LINSIMP_F32, a, (cudaStream_t)stream));
}

int linsimp_qkr_normalize_bwd(const linsimp_params *p, const void *q, const void *k, const void *r, const float *tau,
                              const void *d_q_hat, const void *d_k_hat, const void *d_r_hat, void *dq, void *dk,
                              void *dr, float *dtau, void *workspace, size_t workspace_bytes, linsimp_stream stream)
{
    int rc = norm_check(p, {q, k, r, d_q_hat, d_k_hat, d_r_hat, dq, dk, dr}, {tau, dtau});
    if (rc != LINSIMP_OK) return rc;
    rc = norm_workspace_check(p, workspace, workspace_bytes);
    if (rc != LINSIMP_OK) return rc;
    NormGateArgs a = norm_args(p);
    a.q = q; a.k = k; a.r = r; a.tau = tau; a.dqh = d_q_hat; a.dkh = d_k_hat; a.drh = d_r_hat;
    a.dq = dq; a.dk = dk; a.dr = dr; a.dtau = dtau; a.partial = (float *)workspace;
    return finish(LINSIMP_OP_NORM, norm_gate_run(1, p->io_dtype == LINSIMP_F32, a, (cudaStream_t)stream));
}

int linsimp_gate_rmsnorm(const linsimp_params *p, const void *o, const float *gamma, float rms_eps, void *y,
                         linsimp_stream stream)
{
    const int rc = norm_check(p, {o, y}, {gamma});
    if (rc != LINSIMP_OK) return rc;
    if (!(rms_eps >= 0.f)) return LINSIMP_EINVAL;
    NormGateArgs a = norm_args(p);
    a.o = o; a.gamma = gamma; a.y = y; a.rms_eps = rms_eps;
    return finish(LINSIMP_OP_NORM, norm_gate_run(2, p->io_dtype == LINSIMP_F32, a, (cudaStream_t)stream));
}

int linsimp_gate_rmsnorm_bwd(const linsimp_params *p, const void *o, const float *gamma, float rms_eps, const void *dy,
                             void *d_o, float *dgamma, void *workspace, size_t workspace_bytes, linsimp_stream stream)
{
    int rc = norm_check(p, {o, dy, d_o}, {gamma, dgamma});
    if (rc != LINSIMP_OK) return rc;
    if (!(rms_eps >= 0.f)) return LINSIMP_EINVAL;
    rc = norm_workspace_check(p, workspace, workspace_bytes);
    if (rc != LINSIMP_OK) return rc;
    NormGateArgs a = norm_args(p);
    a.o = o; a.gamma = gamma; a.dy = dy; a.d_o = d_o; a.dgamma = dgamma; a.rms_eps = rms_eps;
    a.partial = (float *)workspace;
    return finish(LINSIMP_OP_NORM, norm_gate_run(3, p->io_dtype == LINSIMP_F32, a, (cudaStream_t)stream));
}

int linsimp_decode_prepare(const linsimp_params *p, const float *omega, void *workspace, size_t workspace_bytes,
                           linsimp_stream stream)
{
    if (!params_ok(p, LINSIMP_OP_DECODE) || !omega) return LINSIMP_EINVAL;
    if (!shape_supported(p)) return LINSIMP_EUNSUPPORTED;
    if (!aligned16(omega)) return LINSIMP_EALIGN;
    if (!(p->io_dtype == LINSIMP_BF16 && p->algo == LINSIMP_ALGO_DEFAULT &&
          decode_mma_supported(p->d, p->m, p->W, decode_banks(p))))
        return LINSIMP_OK;                                   // this shape's decode kernel reads omega itself
    if (!workspace || workspace_bytes < decode_mma_image_bytes(p->d, p->m, decode_banks(p))) return LINSIMP_EWORKSPACE;
    if ((uintptr_t)workspace & 255u) return LINSIMP_EALIGN;
    return finish(LINSIMP_OP_DECODE, decode_mma_prepare(omega, p->d, p->m, decode_banks(p), workspace, (cudaStream_t)stream));
}

int linsimp_prefill_state(const linsimp_params *p, const void *k, const void *v, const float *omega, float *S,
                          float *z, void *workspace, size_t workspace_bytes, linsimp_stream stream)
{
    if (!params_ok(p, LINSIMP_OP_STATE)) return LINSIMP_EINVAL;
    if (!k || !v || !omega || !S || !z) return LINSIMP_EINVAL;
    if (!shape_supported(p)) return LINSIMP_EUNSUPPORTED;
    if (!aligned16(k) || !aligned16(v) || !aligned16(omega) || !aligned16(S) || !aligned16(z)) return LINSIMP_EALIGN;
    if (use_tc_blocks(p, LINSIMP_OP_STATE))
        return run_tc_blocks(LINSIMP_OP_STATE, p, nullptr, k, v, nullptr, nullptr, omega, nullptr, nullptr, nullptr, S, z,
                             nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, workspace, workspace_bytes, stream);
    if (use_tc(p, LINSIMP_OP_STATE))
        return run_tc(p, nullptr, k, v, nullptr, nullptr, omega, nullptr, nullptr, nullptr, S, z, workspace,
                      workspace_bytes, stream, 1);
    const SimtLayout L = simt_layout(p, LINSIMP_OP_STATE);
    if (!workspace || workspace_bytes < L.total) return LINSIMP_EWORKSPACE;
    if ((uintptr_t)workspace & 255u) return LINSIMP_EALIGN;
    SimtArgs a;
    memset(&a, 0, sizeof(a));
    a.B = p->B; a.H = p->H; a.T = p->T; a.d = p->d; a.m = p->m; a.W = p->W; a.C = kSimtChunk;
    a.omega_stride = p->omega_per_head ? (long)p->d * p->m : 0;
    a.k = k; a.v = v; a.omega = omega; a.S_final = S; a.z_final = z;
    a.states = (float *)((char *)workspace + L.states);
    return finish(LINSIMP_OP_STATE, simt_run(LINSIMP_OP_STATE, p->io_dtype, a, (cudaStream_t)stream));
}

int linsimp_profile_enable(int on)
{
    for (auto &r : linsimp::g_records) {
        if (r.start) linsimp::g_event_pool.push_back(r.start);
        if (r.stop) linsimp::g_event_pool.push_back(r.stop);
    }
    linsimp::g_records.clear();
    linsimp::g_profile_error = false;
    linsimp::g_profile_on = on != 0;
    return LINSIMP_OK;
}

int linsimp_profile_read(int index, char *name, int name_len, float *total_ms, int *launches)
{
    if (linsimp::g_profile_error) return LINSIMP_ECUDA;
    std::vector<const char *> names;
    std::vector<float> ms;
    std::vector<int> cnt;
    for (auto &r : linsimp::g_records) {
        if (!r.start || !r.stop) return LINSIMP_ECUDA;
        if (cudaEventSynchronize(r.stop) != cudaSuccess) return LINSIMP_ECUDA;
        float t = 0.f;
        if (cudaEventElapsedTime(&t, r.start, r.stop) != cudaSuccess) return LINSIMP_ECUDA;
        size_t i = 0;
        for (; i < names.size(); ++i)
            if (strcmp(names[i], r.name) == 0) break;
        if (i == names.size()) {
            names.push_back(r.name);
            ms.push_back(0.f);
            cnt.push_back(0);
        }
        ms[i] += t;
        cnt[i] += 1;
    }
    if (index >= 0 && index < (int)names.size()) {
        if (name && name_len > 0) {
            strncpy(name, names[index], (size_t)name_len - 1);
            name[name_len - 1] = 0;
        }
        if (total_ms) *total_ms = ms[index];
        if (launches) *launches = cnt[index];
    }
    return (int)names.size();
}

int linsimp_read_status(const void *workspace, linsimp_stream stream)
{
    if (!workspace) return LINSIMP_EINVAL;
    int host = 0;
    if (cudaMemcpyAsync(&host, workspace, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess)
        return LINSIMP_ECUDA;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return LINSIMP_ECUDA;
    return host;
}

const char *linsimp_strerror(int code)
{
    switch (code) {
    case LINSIMP_OK: return "success";
    case LINSIMP_EINVAL: return "invalid argument (null pointer, non-positive size or bad enum)";
    case LINSIMP_EUNSUPPORTED: return "no kernel instance for this (d, m, W, io_dtype, algo)";
    case LINSIMP_EALIGN: return "pointer not sufficiently aligned";
    case LINSIMP_EWORKSPACE: return "workspace missing or too small";
    case LINSIMP_ECUDA: return "CUDA runtime or launch failure";
    case LINSIMP_ETOOLARGE: return "problem needs more scratch than the library's static array holds";
    default: return "unknown linsimp error code";
    }
}

int linsimp_version(void) { return LINSIMP_VERSION; }

int linsimp_last_launch_count(int op) { return (op >= 0 && op <= 6) ? g_launches[op] : 0; }

}  // extern "C"
