// Value streams of a width other than the key width: v, u in R^{D_v}, q, k, r in R^D (Sec. 3.1).
//
// Eqs. Ni, Zi treat every value channel on its own - N_i[e] uses only channel e of v and u, and Z_i none of them - so the
// layer with D_v channels is the layer with D channels applied to blocks of D value channels (the last block padded with
// zero channels): the outputs lie side by side, rowmax_L and lse are the same for every block, dv and du lie side by side,
// and dq, dk, dr are the sums of the blocks' (each block is a complete function of q, k, r).  This file holds the data
// movement and the driver; the estimator itself runs in the kernels linsimp_fwd / linsimp_bwd dispatch to.
#include <string.h>

#include "../../include/linsimp.h"
#include "common.cuh"
#include "launch.cuh"

namespace linsimp {

// rows x [w_src] -> rows x [w_dst] column window: dst[row][c] = src[row][c0 + c] for c0 + c < w_src, else zero (GATHER),
// or src[row][c] -> dst[row][c0 + c] for c0 + c < w_dst (scatter).  T = element type by size.
template <typename T, bool GATHER>
__global__ void __launch_bounds__(256) k_cols_move(const T *__restrict__ src, T *__restrict__ dst, long rows, int w_src, int w_dst, int c0)
{
    const int w = GATHER ? w_dst : w_src;
    for (long idx = (long)blockIdx.x * 256 + threadIdx.x; idx < rows * w; idx += (long)gridDim.x * 256) {
        const long row = idx / w;
        const int c = (int)(idx - row * w);
        if (GATHER) {
            T val;
            memset(&val, 0, sizeof(T));
            if (c0 + c < w_src) val = src[row * w_src + c0 + c];
            dst[idx] = val;
        } else if (c0 + c < w_dst) {
            dst[row * w_dst + c0 + c] = src[idx];
        }
    }
}

// acc (fp32) = (first ? 0 : acc) + x, x in the I/O type
template <typename T>
__global__ void __launch_bounds__(256) k_accumulate(const T *__restrict__ x, float *__restrict__ acc, long n, int first)
{
    for (long i = (long)blockIdx.x * 256 + threadIdx.x; i < n; i += (long)gridDim.x * 256) acc[i] = (first ? 0.f : acc[i]) + ldf(x + i);
}
template <typename T>
__global__ void __launch_bounds__(256) k_round_out(const float *__restrict__ acc, T *__restrict__ y, long n)
{
    for (long i = (long)blockIdx.x * 256 + threadIdx.x; i < n; i += (long)gridDim.x * 256) stf(y + i, acc[i]);
}

namespace {

size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }

struct DvLayout {
    size_t inner_bytes, v, u, dO, o, g[5], acc[3], S, z, total;
};

DvLayout dv_layout(const linsimp_params *p, int op, size_t inner)
{
    DvLayout L;
    memset(&L, 0, sizeof(L));
    const size_t esz = p->io_dtype == LINSIMP_F32 ? 4 : 2;
    const size_t n = up256((size_t)p->B * p->H * p->T * p->d * esz), n32 = up256((size_t)p->B * p->H * p->T * p->d * 4);
    L.inner_bytes = inner;
    size_t off = up256(inner);
    L.v = off; off += n;
    L.u = off; off += n;
    L.o = off; off += n;
    L.S = off; off += up256((size_t)p->B * p->H * p->m * p->d * 4);
    L.z = off; off += up256((size_t)p->B * p->H * p->m * 4);
    if (op == LINSIMP_OP_BWD) {
        L.dO = off; off += n;
        for (int x = 0; x < 5; ++x) { L.g[x] = off; off += n; }
        for (int x = 0; x < 3; ++x) { L.acc[x] = off; off += n32; }
    }
    L.total = off;
    return L;
}

template <bool GATHER>
int cols(LaunchScope &sc, int io_dtype, const void *src, void *dst, long rows, int w_src, int w_dst, int c0)
{
    const int w = GATHER ? w_dst : w_src;
    const unsigned grid = (unsigned)((rows * w + 255) / 256 < 4736 ? (rows * w + 255) / 256 : 4736);
    if (io_dtype == LINSIMP_F32)
        LS_LAUNCH(sc, GATHER ? "cols_gather" : "cols_scatter", k_cols_move<float, GATHER><<<grid, 256, 0, sc.stream>>>(
            (const float *)src, (float *)dst, rows, w_src, w_dst, c0));
    else
        LS_LAUNCH(sc, GATHER ? "cols_gather" : "cols_scatter", k_cols_move<bf16, GATHER><<<grid, 256, 0, sc.stream>>>(
            (const bf16 *)src, (bf16 *)dst, rows, w_src, w_dst, c0));
    return 0;
}

}  // namespace

size_t value_width_workspace_bytes(const linsimp_params *p, int op)
{
    linsimp_params pi = *p;
    pi.dv = 0;
    const size_t inner = linsimp_workspace_bytes(&pi, op);
    if (inner == 0) return 0;
    return dv_layout(p, op, inner).total;
}

// returns a LINSIMP_* code; *launched = kernels of this file (the inner calls count theirs)
int value_width_fwd(const linsimp_params *p, const void *q, const void *k, const void *v, const void *r, const void *u,
                    const float *omega, void *o, float *rowmax_L, float *lse, float *S_final, float *z_final, void *workspace,
                    size_t workspace_bytes, linsimp_stream stream, int *launched)
{
    linsimp_params pi = *p;
    pi.dv = 0;
    const size_t inner = linsimp_workspace_bytes(&pi, LINSIMP_OP_FWD);
    if (inner == 0) return LINSIMP_EUNSUPPORTED;
    const DvLayout L = dv_layout(p, LINSIMP_OP_FWD, inner);
    if (!workspace || workspace_bytes < L.total) return LINSIMP_EWORKSPACE;
    if ((uintptr_t)workspace & 255u) return LINSIMP_EALIGN;
    char *ws = (char *)workspace;
    LaunchScope sc = {(cudaStream_t)stream, 0};
    const long rows = (long)p->B * p->H * p->T, srows = (long)p->B * p->H * p->m;
    const int nb = (p->dv + p->d - 1) / p->d;
    for (int b = 0; b < nb; ++b) {
        cols<true>(sc, p->io_dtype, v, ws + L.v, rows, p->dv, p->d, b * p->d);
        cols<true>(sc, p->io_dtype, u, ws + L.u, rows, p->dv, p->d, b * p->d);
        // the shift and the log-normaliser do not depend on the values: every block writes the same numbers
        const int rc = linsimp_fwd(&pi, q, k, ws + L.v, r, ws + L.u, omega, ws + L.o, rowmax_L, lse, S_final ? (float *)(ws + L.S) : nullptr,
                                   S_final ? (float *)(ws + L.z) : nullptr, ws, inner, stream);
        if (rc != LINSIMP_OK) return rc;
        cols<false>(sc, p->io_dtype, ws + L.o, o, rows, p->d, p->dv, b * p->d);
        if (S_final) {
            cols<false>(sc, LINSIMP_F32, ws + L.S, S_final, srows, p->d, p->dv, b * p->d);
            if (b == 0 && cudaMemcpyAsync(z_final, ws + L.z, sizeof(float) * srows, cudaMemcpyDeviceToDevice, sc.stream) != cudaSuccess)
                return LINSIMP_ECUDA;
        }
    }
    *launched = sc.count;
    return sc.result() < 0 ? LINSIMP_ECUDA : LINSIMP_OK;
}

int value_width_bwd(const linsimp_params *p, const void *q, const void *k, const void *v, const void *r, const void *u,
                    const float *omega, const void *o, const float *rowmax_L, const float *lse, const void *dO, void *dq, void *dk,
                    void *dv, void *dr, void *du, void *workspace, size_t workspace_bytes, linsimp_stream stream, int *launched)
{
    linsimp_params pi = *p;
    pi.dv = 0;
    pi.flags &= ~LINSIMP_FLAG_REUSE_FWD_STATE;           // every block runs its own pre-pass
    const size_t inner = linsimp_workspace_bytes(&pi, LINSIMP_OP_BWD);
    if (inner == 0) return LINSIMP_EUNSUPPORTED;
    const DvLayout L = dv_layout(p, LINSIMP_OP_BWD, inner);
    if (!workspace || workspace_bytes < L.total) return LINSIMP_EWORKSPACE;
    if ((uintptr_t)workspace & 255u) return LINSIMP_EALIGN;
    char *ws = (char *)workspace;
    LaunchScope sc = {(cudaStream_t)stream, 0};
    const long rows = (long)p->B * p->H * p->T, n = rows * p->d;
    const int nb = (p->dv + p->d - 1) / p->d;
    const unsigned grid = (unsigned)((n + 255) / 256 < 4736 ? (n + 255) / 256 : 4736);
    void *sums[3] = {dq, dk, dr};
    const size_t gsrc[3] = {L.g[0], L.g[1], L.g[3]};
    for (int b = 0; b < nb; ++b) {
        cols<true>(sc, p->io_dtype, v, ws + L.v, rows, p->dv, p->d, b * p->d);
        cols<true>(sc, p->io_dtype, u, ws + L.u, rows, p->dv, p->d, b * p->d);
        cols<true>(sc, p->io_dtype, dO, ws + L.dO, rows, p->dv, p->d, b * p->d);
        // (the output argument of the backward is not read by the kernels that recompute it; the fp32 kernels read it:
        // give them the block's own columns)
        cols<true>(sc, p->io_dtype, o, ws + L.o, rows, p->dv, p->d, b * p->d);
        const int rc = linsimp_bwd(&pi, q, k, ws + L.v, r, ws + L.u, omega, ws + L.o, rowmax_L, lse, ws + L.dO, ws + L.g[0], ws + L.g[1],
                                   ws + L.g[2], ws + L.g[3], ws + L.g[4], ws, inner, stream);
        if (rc != LINSIMP_OK) return rc;
        cols<false>(sc, p->io_dtype, ws + L.g[2], dv, rows, p->d, p->dv, b * p->d);
        cols<false>(sc, p->io_dtype, ws + L.g[4], du, rows, p->d, p->dv, b * p->d);
        for (int x = 0; x < 3; ++x) {
            if (p->io_dtype == LINSIMP_F32)
                LS_LAUNCH(sc, "accumulate", k_accumulate<float><<<grid, 256, 0, sc.stream>>>((const float *)(ws + gsrc[x]), (float *)(ws + L.acc[x]), n, b == 0));
            else
                LS_LAUNCH(sc, "accumulate", k_accumulate<bf16><<<grid, 256, 0, sc.stream>>>((const bf16 *)(ws + gsrc[x]), (float *)(ws + L.acc[x]), n, b == 0));
        }
    }
    for (int x = 0; x < 3; ++x) {
        if (p->io_dtype == LINSIMP_F32)
            LS_LAUNCH(sc, "round_out", k_round_out<float><<<grid, 256, 0, sc.stream>>>((const float *)(ws + L.acc[x]), (float *)sums[x], n));
        else
            LS_LAUNCH(sc, "round_out", k_round_out<bf16><<<grid, 256, 0, sc.stream>>>((const float *)(ws + L.acc[x]), (bf16 *)sums[x], n));
    }
    *launched = sc.count;
    return sc.result() < 0 ? LINSIMP_ECUDA : LINSIMP_OK;
}

}  // namespace linsimp
