/*
 * linsimp.h - C ABI of the B200 (sm_100a) LinSimp hot path.
 *
 * LinSimp = linearized 2-simplicial attention.  For one head, with streams
 * q, k, r (width d) and v, u (width d as well), a feature matrix Omega and the
 * feature map  phi(x) = exp(Omega x - |x|^2/2)/sqrt(m)  (Eq. prf):
 *
 *     M_i = sum_{j<=i} phi(k_j) v_j^T ,  a_i = sum_{j<=i} phi(k_j)   (Eqs. Mstate, astate)
 *     C_i = { max(0, i-W+1), ..., i }                               (Sec. 3.3)
 *     N_i = sum_{c in C_i} [phi(q_i*r_c)^T M_i] * u_c               (Eq. Ni)
 *     Z_i = sum_{c in C_i}  phi(q_i*r_c)^T a_i                      (Eq. Zi)
 *     o_i = N_i / (Z_i + eps)                                       (Eq. linearized-output)
 *
 * ('*' between vectors is the coordinatewise product.)  linsimp_fwd, linsimp_bwd and
 * linsimp_decode_step use their inputs as given; the L2 normalisation with the
 * temperature of Sec. 3.1 and the gated RMSNorm of Eq. gated-output are entry points
 * of their own (linsimp_qkr_normalize, linsimp_gate_rmsnorm and their backward).
 *
 * Conventions shared by all entry points
 *   - Every pointer is a DEVICE pointer unless stated otherwise.  The library
 *     never allocates, frees or synchronises; all work is enqueued on `stream`
 *     (a cudaStream_t passed as void*; NULL = the default stream).  The caller
 *     owns every buffer, including the workspace, for the duration of the work.
 *   - Token tensors are contiguous [B, H, T, d] (decode: [B, H, d]) in
 *     `io_dtype`; they must be 16-byte aligned.
 *   - Omega is fp32, contiguous [d, m] (column p is the paper's feature row
 *     omega_p), shared by all heads, or [H, d, m] when omega_per_head != 0.
 *     It is read-only and gets no gradient (non-trainable buffer, App. B.1).
 *   - The library evaluates the features in log space with a per-row shift
 *     (App. B.2): psi' = exp(l - L_i), L_i = max over the row's anchors and
 *     features; key features are unshifted.  Internally neither feature carries
 *     the 1/sqrt(m) factor; the guard eps is rescaled to match, so the result
 *     equals N_i/(Z_i+eps) of Eq. linearized-output with eps on the unscaled
 *     Z_i.  If both the shifted normaliser and the shifted eps underflow fp32
 *     the row's output is 0.
 *   - State tensors S [B, H, m, d] and z [B, H, m] are fp32 and hold
 *     sum_j exp(l(k_j)) v_j^T and sum_j exp(l(k_j)): the paper's M and a times
 *     sqrt(m).
 *   - Return value: 0 on success, a negative LINSIMP_E* code otherwise.  All
 *     argument checks happen on the host before anything is launched; on error
 *     nothing has been enqueued.  Launch failures are reported as
 *     LINSIMP_ECUDA (the CUDA error is left readable via cudaGetLastError's
 *     sticky state only if it is a sticky error).
 */
#ifndef LINSIMP_H
#define LINSIMP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LINSIMP_VERSION 6

enum {
    LINSIMP_OK = 0,
    LINSIMP_EINVAL = -1,      /* null pointer, non-positive size, bad enum           */
    LINSIMP_EUNSUPPORTED = -2,/* (d, m, W, io_dtype, algo) has no kernel instance     */
    LINSIMP_EALIGN = -3,      /* a pointer is not 16-byte aligned                     */
    LINSIMP_EWORKSPACE = -4,  /* workspace null or smaller than linsimp_workspace_bytes */
    LINSIMP_ECUDA = -5,       /* a CUDA runtime call or kernel launch failed          */
    LINSIMP_ETOOLARGE = -6    /* problem needs more scratch than the built-in static array holds */
};

enum { LINSIMP_F32 = 0, LINSIMP_BF16 = 1 };          /* io_dtype */
enum { LINSIMP_OP_FWD = 0, LINSIMP_OP_BWD = 1, LINSIMP_OP_DECODE = 2, LINSIMP_OP_STATE = 3, LINSIMP_OP_NORM = 4,
       LINSIMP_OP_FWD_PACKED = 5, LINSIMP_OP_BWD_PACKED = 6 };
enum {
    LINSIMP_ALGO_DEFAULT = 0, /* fp32 I/O: fp32 CUDA-core kernels; bf16 I/O: tensor-core kernels */
    LINSIMP_ALGO_FP32 = 1     /* force the fp32 CUDA-core kernels (any io_dtype)      */
};

enum {
    /* linsimp_bwd only: the workspace is the one the preceding linsimp_fwd call (same
     * parameters, same k, v, omega, same stream) was given and nothing has written to it
     * since, so the chunk-boundary states of Eqs. Mstate/astate it still holds are used
     * instead of being recomputed.  The workspace must have the size linsimp_bwd asks for.
     * Without the bit the backward recomputes the states and depends on no earlier call. */
    LINSIMP_FLAG_REUSE_FWD_STATE = 1,
    /* linsimp_decode_step only: the workspace holds the image of omega that linsimp_decode_prepare
     * wrote (same parameters, same omega, untouched since); the step then copies it instead of
     * converting omega again.  Ignored by kernels that keep omega in fp32. */
    LINSIMP_FLAG_OMEGA_IMAGE = 2,
    /* linsimp_fwd and linsimp_bwd: both orientations of the trilinear score (Eq. two-views) kernelised and averaged
     * (App. E, first item), in the windowed form of this operator.  View 1 is the estimator as defined (composite
     * query q_i * r_c over the window, keys k_j over the prefix); view 2 exchanges the two key streams and their
     * values (composite query q_i * k_j over the window, keys r_c over the prefix).  Numerators and normalisers
     * are added before the division: o_i = (N1_i + N2_i) / (Z1_i + Z2_i + 2 eps).  rowmax_L and lse then describe
     * the combined estimator (lse = log(m (Z1 + Z2 + 2 eps))), S_final / z_final the state of view 1.  Costs two
     * passes of the kernels.  bf16 I/O on the tensor-core kernels with m <= 128 only (LINSIMP_EUNSUPPORTED
     * otherwise); LINSIMP_FLAG_REUSE_FWD_STATE has no effect together with it. */
    LINSIMP_FLAG_TWO_VIEWS = 4,
    /* linsimp_bwd (and the forward whose states it reuses), tensor-core kernels: the chunk-boundary states enter the
     * backward's products as two bf16 terms instead of one.  The backward recomputes the output (App. C) from a
     * bf16 operand image of M_b (Eq. Mstate); dZ_i sees that output, while every key's own value enters its gradient
     * exactly, and the two cancel in dk (d l / d z = omega - z, App. C): the image's rounding is the largest part of
     * the error of dk (up to 2.3e-2 of max|dk| on a few of 170 surveyed seeds; below 1e-2 with this bit).  Costs a
     * second image per chunk in the workspace (linsimp_workspace_bytes accounts for it) and about a sixth more time in
     * the backward's tile kernel.  A forward that is to leave its states for LINSIMP_FLAG_REUSE_FWD_STATE must be
     * given the bit as well.  No effect on the fp32 kernels, whose state is exact. */
    LINSIMP_FLAG_STATE_TWO_TERMS = 8
};

typedef struct {
    int32_t B, H;             /* batch (decode: sequences) and heads                  */
    int32_t T;                /* tokens per sequence (ignored by decode)              */
    int32_t d;                /* head width of q,k,r and of v,u: 32, 64 or 128        */
    int32_t m;                /* feature rank: 32, 64, 128 or 256                     */
    int32_t W;                /* anchor window, 1..64                                 */
    int32_t io_dtype;         /* LINSIMP_F32 or LINSIMP_BF16                          */
    int32_t omega_per_head;   /* 0: Omega [d,m]; else [H,d,m]                         */
    int32_t algo;             /* LINSIMP_ALGO_*                                       */
    float   eps;              /* guard of Eq. linearized-output, 1e-30 in the paper   */
    int32_t flags;            /* LINSIMP_FLAG_* bits, 0 for none                      */
    int32_t dv;               /* width D_v of v, u (and o, dO, dv, du, S) when it differs from d (Sec. 3.1: q,k,r in
                               * R^D, v,u in R^{D_v}); 0 or d: the same width.  Any D_v >= 1 with D_v * element size a
                               * multiple of 16 bytes; taken by linsimp_fwd and linsimp_bwd only, where the layer runs
                               * as ceil(D_v / d) blocks of d value channels (every value channel is an estimator of
                               * its own that shares Z_i), at that many times the cost.  Other calls: LINSIMP_EINVAL. */
} linsimp_params;

typedef void *linsimp_stream;

/* Bytes of device workspace the given operation needs for these parameters
 * (0 for an invalid parameter set).  The workspace needs 256-byte alignment
 * and may be reused between calls on the same stream; its contents after a
 * call are unspecified, except that linsimp_fwd leaves the chunk-boundary
 * states at the start of the workspace in the form LINSIMP_FLAG_REUSE_FWD_STATE
 * describes.  Host function, no CUDA call. */
size_t linsimp_workspace_bytes(const linsimp_params *p, int op);

/*
 * Forward (Eqs. Mstate, astate, Ni, Zi, linearized-output; Algorithm 1 in
 * chunked form with exclusive chunk-boundary states, Sec. 4.2).
 *   in : q,k,v,r,u [B,H,T,d] io_dtype; omega fp32
 *   out: o [B,H,T,d] io_dtype
 *        rowmax_L [B,H,T] fp32   L_i of App. B.2
 *        lse      [B,H,T] fp32   L_i + log(Z'_i + eps'_i), where Z' is the shifted
 *                                normaliser without 1/m and eps' = eps*m*exp(-L_i);
 *                                i.e. log(m*(Z_i + eps)).  rowmax_L is the per-row
 *                                shift of App. B.2 and lse the log-normaliser; with
 *                                the inputs they are all the backward needs
 *                                (Sec. 4.2 "Backward").
 *        S_final [B,H,m,d], z_final [B,H,m] fp32, nullable (both or neither):
 *                                prefix state after the last token, in the
 *                                decode convention above.
 */
int linsimp_fwd(const linsimp_params *p,
                const void *q, const void *k, const void *v, const void *r, const void *u,
                const float *omega,
                void *o, float *rowmax_L, float *lse,
                float *S_final, float *z_final,
                void *workspace, size_t workspace_bytes, linsimp_stream stream);

/*
 * Forward of a segment that continues a sequence (Theorem 1: the state M, a and the last
 * W-1 anchors are all the past the layer needs; chunked prefill and prefill after a cached
 * prefix).  As linsimp_fwd, with
 *   S_init [B,H,m,d], z_init [B,H,m] fp32 (both or neither null): the prefix state before
 *        the segment's first token, in the decode convention (what S_final, z_final of the
 *        previous segment, linsimp_prefill_state or linsimp_decode_step hold);
 *   hist_r, hist_u [B,H,n_hist,d] io_dtype, 0 <= n_hist <= W-1 (null when 0): r and u of
 *        the n_hist tokens before the segment, oldest first; they act only as anchors.
 * Outputs cover the segment's T tokens.  Available where the tensor-core forward is
 * (bf16 I/O, default algo, d in {64,128}, m in {32,64,128}); LINSIMP_EUNSUPPORTED otherwise.
 * Its backward is linsimp_bwd_continue.
 */
int linsimp_fwd_continue(const linsimp_params *p,
                         const void *q, const void *k, const void *v, const void *r, const void *u,
                         const float *omega,
                         const float *S_init, const float *z_init,
                         const void *hist_r, const void *hist_u, int32_t n_hist,
                         void *o, float *rowmax_L, float *lse,
                         float *S_final, float *z_final,
                         void *workspace, size_t workspace_bytes, linsimp_stream stream);

/*
 * Backward of a continued segment (Theorem 1 read backwards: the only paths between a segment
 * and the rest of the sequence are the state M, a it starts from and ends with and the W-1
 * anchor rows before it; App. C for the sweeps themselves).  For a loss
 *     sum(dO * o_segment) + f(S_final, z_final)
 * with dS_final = df/dS_final and dz_final = df/dz_final known, it returns the gradients with
 * respect to the segment's own q, k, v, r, u, to the history anchors and to the state the
 * segment started from.  Chunked training over a long sequence walks the segments last to
 * first: dS_init, dz_init of one call are dS_final, dz_final of the call for the segment
 * before, and d_hist_r, d_hist_u are added by the caller to dr, du of the last n_hist rows
 * before the segment (the rows hist_r, hist_u were copied from).
 *   in : q,k,v,r,u [B,H,T,d], omega, S_init, z_init, hist_r, hist_u, n_hist as in
 *        linsimp_fwd_continue; rowmax_L, lse [B,H,T] from that call; dO [B,H,T,d];
 *        dS_final [B,H,m,d], dz_final [B,H,m] fp32 (both or neither null: null = zero)
 *   out: dq,dk,dv,dr,du [B,H,T,d] io_dtype (overwritten);
 *        d_hist_r, d_hist_u [B,H,n_hist,d] io_dtype (overwritten; null when n_hist = 0);
 *        dS_init [B,H,m,d], dz_init [B,H,m] fp32 (both or neither null), in the convention of
 *        the state tensors (gradient with respect to those very numbers)
 *   workspace: linsimp_workspace_bytes(p, LINSIMP_OP_BWD).  LINSIMP_FLAG_REUSE_FWD_STATE is not
 *        accepted here (LINSIMP_EINVAL): the segment's pre-pass always runs.
 * Available where linsimp_fwd_continue is; LINSIMP_EUNSUPPORTED otherwise.
 */
int linsimp_bwd_continue(const linsimp_params *p,
                         const void *q, const void *k, const void *v, const void *r, const void *u,
                         const float *omega,
                         const float *S_init, const float *z_init,
                         const void *hist_r, const void *hist_u, int32_t n_hist,
                         const float *rowmax_L, const float *lse, const void *dO,
                         const float *dS_final, const float *dz_final,
                         void *dq, void *dk, void *dv, void *dr, void *du,
                         void *d_hist_r, void *d_hist_u, float *dS_init, float *dz_init,
                         void *workspace, size_t workspace_bytes, linsimp_stream stream);

/*
 * Anchor ring of the decode step from token rows (the hand-off from prefill; data movement
 * only, no counterpart in the paper): for t in [max(0, T-W), T) the rows r[t], u[t] go to slot
 * (t_first + t) % W of ring_r, ring_u [B,H,W,d].  p->T = T tokens in r, u [B,H,T,d];
 * t_first = position of r[0] in the sequence.  Calling it segment by segment keeps the ring
 * current; the decode position after a prefix of n tokens is pos = n.
 */
int linsimp_ring_fill(const linsimp_params *p, const void *r, const void *u, int64_t t_first,
                      void *ring_r, void *ring_u, linsimp_stream stream);

/*
 * Backward of sum(dO*o) w.r.t. q, k, v, r, u (App. C, backward query sweep and
 * backward state sweep).  Everything except the inputs, o, rowmax_L and lse is
 * recomputed.  d l/d z = omega - z.
 *   in : q,k,v,r,u, omega as in forward; o, rowmax_L, lse from linsimp_fwd on
 *        the same inputs; dO [B,H,T,d] io_dtype
 *   out: dq,dk,dv,dr,du [B,H,T,d] io_dtype (overwritten)
 * The anchor gradients dr, du are accumulated with floating-point atomics,
 * so their last bits may differ between runs; dq, dk, dv of the tensor-core
 * kernels (and o, rowmax_L, lse of the forward) are bit-reproducible.
 */
int linsimp_bwd(const linsimp_params *p,
                const void *q, const void *k, const void *v, const void *r, const void *u,
                const float *omega,
                const void *o, const float *rowmax_L, const float *lse, const void *dO,
                void *dq, void *dk, void *dv, void *dr, void *du,
                void *workspace, size_t workspace_bytes, linsimp_stream stream);

/*
 * One autoregressive step for B sequences (Theorem 1: persistent M, a and a
 * rolling buffer of the last W (r, u) pairs).  For each (sequence, head):
 *   S += exp(l(k_t)) v_t^T ; z += exp(l(k_t)) ; ring slot pos % W <- (r_t, u_t);
 *   then o_t from the min(pos+1, W) most recent anchors and the updated state.
 *   in    : q_t,k_t,v_t,r_t,u_t [B,H,d] io_dtype; omega fp32;
 *           pos [B] int32 (device): tokens seen so far by each sequence
 *   in/out: S [B,H,m,d] fp32, z [B,H,m] fp32,
 *           ring_r, ring_u [B,H,W,d] io_dtype (slot s holds the token t with t % W == s)
 *   out   : o_t [B,H,d] io_dtype
 * `pos` is not modified; the caller advances it.  p->T is ignored.
 */
int linsimp_decode_step(const linsimp_params *p,
                        const void *q_t, const void *k_t, const void *v_t,
                        const void *r_t, const void *u_t, const float *omega,
                        float *S, float *z, void *ring_r, void *ring_u,
                        const int32_t *pos, void *o_t,
                        void *workspace, size_t workspace_bytes, linsimp_stream stream);

/*
 * Optional companion of linsimp_decode_step (no counterpart in the paper: a layout
 * conversion of the constant feature matrix, done once instead of in every step).
 * Writes the image of omega the decode kernel works from (fp16 high and low parts,
 * transposed) into `workspace` (device, 256-byte aligned,
 * linsimp_workspace_bytes(p, LINSIMP_OP_DECODE) bytes; that is 0 for shapes whose
 * decode kernel has no such image, and the call is then a no-op).  Pass the same
 * workspace to linsimp_decode_step with LINSIMP_FLAG_OMEGA_IMAGE set.
 */
int linsimp_decode_prepare(const linsimp_params *p, const float *omega,
                           void *workspace, size_t workspace_bytes, linsimp_stream stream);

/*
 * Prefix state only (Eqs. Mstate, astate; the chunk-state + scan kernels of the
 * forward without the query side): S [B,H,m,d] = sum_{j<T} exp(l(k_j)) v_j^T,
 * z [B,H,m] = sum_{j<T} exp(l(k_j)), fp32, overwritten.  This is the
 * prefill-to-decode hand-off: its outputs are the decode state after T tokens.
 *   in : k, v [B,H,T,d] io_dtype; omega fp32
 *   workspace: linsimp_workspace_bytes(p, LINSIMP_OP_STATE)
 */
int linsimp_prefill_state(const linsimp_params *p, const void *k, const void *v, const float *omega,
                          float *S, float *z, void *workspace, size_t workspace_bytes,
                          linsimp_stream stream);

/*
 * Batches of sequences of different lengths, padded to a common T (Theorem 1: the layer is
 * causal, so padding placed after a sequence cannot reach its tokens; what has to know the
 * true lengths is the state, the decode ring and the backward).  seq_lens [B] int32 (device):
 * sequence b holds seq_lens[b] tokens (clamped to [0, T]) followed by padding rows, whose
 * contents are read but have no effect.
 *   linsimp_fwd_padded: as linsimp_fwd; padding keys add nothing to the prefix state, so
 *        S_final, z_final hold each sequence's state after its own last token.  o, rowmax_L,
 *        lse of padding rows are finite but unspecified.
 *   linsimp_bwd_padded: as linsimp_bwd with dO of padding rows taken as zero (whatever the
 *        buffer holds there); all five gradients of padding rows come out as zero.
 *        LINSIMP_FLAG_REUSE_FWD_STATE refers to a linsimp_fwd_padded call with the same seq_lens.
 *   linsimp_ring_fill_padded: the decode ring of each sequence from its own last
 *        min(seq_lens[b], W) rows (token t in slot t mod W); continue decoding sequence b with
 *        pos[b] = seq_lens[b].
 * Available where the tensor-core kernels are (bf16 I/O, default algo, d in {64,128},
 * m in {32,64,128}); LINSIMP_EUNSUPPORTED otherwise.  A sequence starts at row 0 of its batch
 * entry here; the *_packed calls below take sequences laid end to end.
 */
int linsimp_fwd_padded(const linsimp_params *p,
                       const void *q, const void *k, const void *v, const void *r, const void *u,
                       const float *omega, const int32_t *seq_lens,
                       void *o, float *rowmax_L, float *lse, float *S_final, float *z_final,
                       void *workspace, size_t workspace_bytes, linsimp_stream stream);
int linsimp_bwd_padded(const linsimp_params *p,
                       const void *q, const void *k, const void *v, const void *r, const void *u,
                       const float *omega, const int32_t *seq_lens,
                       const void *o, const float *rowmax_L, const float *lse, const void *dO,
                       void *dq, void *dk, void *dv, void *dr, void *du,
                       void *workspace, size_t workspace_bytes, linsimp_stream stream);
int linsimp_ring_fill_padded(const linsimp_params *p, const void *r, const void *u, const int32_t *seq_lens,
                             void *ring_r, void *ring_u, linsimp_stream stream);

/*
 * Exact windowed 2-simplicial attention, forward (the comparison layer of Sec. 4.3 "Baselines" and Table layouts: one
 * joint softmax over a w1 x w2 pair plane, 512 x 32 in the paper's runs; Eq. exact-window-app with a window on the first
 * key stream as well).  No random features, no state:
 *     s_ijc = sum_a q_i[a] k_j[a] r_c[a],    o_i = sum_{j,c} exp(s_ijc) (v_j * u_c) / sum_{j,c} exp(s_ijc)
 * over j in [max(0, i-w1+1), i] and c in [max(0, i-w2+1), i].  Inputs are used as given (normalisation and temperature
 * are the caller's, as for linsimp_fwd).
 *   in : q,k,v,r,u [B,H,T,d] bf16; p->W = w2 (1..32); w1 >= 1; p->d in {64,128}; p->m, p->eps unused
 *   out: o [B,H,T,d] bf16; lse [B,H,T] fp32 (nullable): log of the normaliser
 * No workspace.  fp32 streams, other widths or w2 > 32: LINSIMP_EUNSUPPORTED.
 */
int linsimp_winsimp_fwd(const linsimp_params *p, int32_t w1,
                        const void *q, const void *k, const void *v, const void *r, const void *u,
                        void *o, float *lse, linsimp_stream stream);

/*
 * Packed batches (Theorem 1 again: sequences are independent, so how they share a buffer is
 * data layout only; the paper has no counterpart).  The token streams are [H, total_tokens, d]:
 * for every head the sequences lie end to end, sequence b in rows [cu_seqlens[b], cu_seqlens[b+1]).
 * cu_seqlens [B+1] int32 (device), non-decreasing, cu_seqlens[0] >= 0, cu_seqlens[B] <= total_tokens
 * (the library does not check the values; rows outside every sequence are neither read nor written).
 * p->B = number of sequences, p->T = an upper bound on the longest sequence (a longer one is cut at T).
 *   linsimp_fwd_packed: o [H,total_tokens,d], rowmax_L, lse [H,total_tokens] for the sequences' rows;
 *        S_final [B,H,m,d], z_final [B,H,m] (nullable) per sequence after its own last token.
 *   linsimp_bwd_packed: rowmax_L, lse from linsimp_fwd_packed, dO and the five gradients [H,total_tokens,d].
 *   linsimp_ring_fill_packed: decode ring [B,H,W,d] of each sequence from its own last min(len, W) rows
 *        (token t in slot t mod W); continue decoding sequence b with pos[b] = its length.
 * The sequences are moved into the padded form inside the workspace, run through the padded-batch
 * kernels and gathered back, so the cost is that of a padded batch of B x T tokens plus the copies.
 * workspace: linsimp_workspace_bytes(p, LINSIMP_OP_FWD_PACKED / LINSIMP_OP_BWD_PACKED).
 * LINSIMP_FLAG_REUSE_FWD_STATE is not accepted (LINSIMP_EINVAL).  bf16 I/O on the tensor-core kernels
 * only; LINSIMP_EUNSUPPORTED otherwise.
 */
int linsimp_fwd_packed(const linsimp_params *p,
                       const void *q, const void *k, const void *v, const void *r, const void *u,
                       const float *omega, const int32_t *cu_seqlens, int64_t total_tokens,
                       void *o, float *rowmax_L, float *lse, float *S_final, float *z_final,
                       void *workspace, size_t workspace_bytes, linsimp_stream stream);
int linsimp_bwd_packed(const linsimp_params *p,
                       const void *q, const void *k, const void *v, const void *r, const void *u,
                       const float *omega, const int32_t *cu_seqlens, int64_t total_tokens,
                       const float *rowmax_L, const float *lse, const void *dO,
                       void *dq, void *dk, void *dv, void *dr, void *du,
                       void *workspace, size_t workspace_bytes, linsimp_stream stream);
int linsimp_ring_fill_packed(const linsimp_params *p, const void *r, const void *u, const int32_t *cu_seqlens,
                             int64_t total_tokens, void *ring_r, void *ring_u, linsimp_stream stream);

/*
 * Input side of a head (Sec. 3.1, the definitions before the trilinear score): the streams
 * the estimator consumes are
 *     q^ = tau_h q / |q|_2,   k^ = k / |k|_2,   r^ = r / |r|_2
 * with one learned temperature per head on the query only (the paper initialises tau = sqrt(d)).
 * One streaming kernel normalises the three streams; arithmetic in fp32, outputs rounded to
 * io_dtype.  A row whose norm is below LINSIMP_NORM_FLOOR is divided by the floor instead
 * (a zero row stays zero; the paper does not treat the case).
 *   in : q, k, r [B,H,T,d] io_dtype; tau [H] fp32 (device)
 *   out: q_hat, k_hat, r_hat [B,H,T,d] io_dtype (may alias their inputs)
 * Uses p->B, H, T, d, io_dtype; d must be a multiple of 4, at most 512 (LINSIMP_EUNSUPPORTED
 * otherwise).  No workspace.
 */
#define LINSIMP_NORM_FLOOR 1e-12f
int linsimp_qkr_normalize(const linsimp_params *p, const void *q, const void *k, const void *r, const float *tau,
                          void *q_hat, void *k_hat, void *r_hat, linsimp_stream stream);

/*
 * Backward of linsimp_qkr_normalize: given the gradients of the normalised streams (what
 * linsimp_bwd returns as dq, dk, dr when it was fed q^, k^, r^) and the raw streams,
 *     dx = s/|x| (g - e (e . g)),  e = x/|x|,  s = tau_h for q and 1 for k, r;
 *     dtau_h = sum over b, t of e_q . g_q
 * (a floored row: dx = s/floor g).  The norms are recomputed from the raw rows; the per-head
 * sum is taken in a fixed order (bit-reproducible).
 *   in : q, k, r, d_q_hat, d_k_hat, d_r_hat [B,H,T,d] io_dtype; tau [H] fp32
 *   out: dq, dk, dr [B,H,T,d] io_dtype (may alias the d_*_hat inputs); dtau [H] fp32, overwritten
 *   workspace: linsimp_workspace_bytes(p, LINSIMP_OP_NORM), 256-byte aligned
 */
int linsimp_qkr_normalize_bwd(const linsimp_params *p, const void *q, const void *k, const void *r, const float *tau,
                              const void *d_q_hat, const void *d_k_hat, const void *d_r_hat,
                              void *dq, void *dk, void *dr, float *dtau,
                              void *workspace, size_t workspace_bytes, linsimp_stream stream);

/*
 * Output side of a head (Eq. gated-output): y_i = sigmoid(gamma_h) RMSNorm(o_i) with
 * RMSNorm(x) = x / sqrt(mean_e x_e^2 + rms_eps), one learned scalar gate per head (the paper
 * initialises gamma = -2), no learned weight inside the norm (the paper names none; its
 * model-wide RMSNorm epsilon is 1e-6).
 *   in : o [B,H,T,d] io_dtype; gamma [H] fp32 (device); rms_eps >= 0
 *   out: y [B,H,T,d] io_dtype (may alias o)
 * Shape limits as linsimp_qkr_normalize.  No workspace.
 */
int linsimp_gate_rmsnorm(const linsimp_params *p, const void *o, const float *gamma, float rms_eps, void *y,
                         linsimp_stream stream);

/*
 * Backward of linsimp_gate_rmsnorm: with s = (mean(o^2) + rms_eps)^(-1/2), n = o s, g = sigmoid(gamma_h),
 *     d_o = g s (dy - n mean_e(dy n)),   dgamma_h = g (1 - g) sum over b, t of dy . n
 * (per-head sum in a fixed order).
 *   in : o, dy [B,H,T,d] io_dtype; gamma [H] fp32
 *   out: d_o [B,H,T,d] io_dtype (may alias dy): the dO argument of linsimp_bwd; dgamma [H] fp32, overwritten
 *   workspace: linsimp_workspace_bytes(p, LINSIMP_OP_NORM), 256-byte aligned
 */
int linsimp_gate_rmsnorm_bwd(const linsimp_params *p, const void *o, const float *gamma, float rms_eps,
                             const void *dy, void *d_o, float *dgamma,
                             void *workspace, size_t workspace_bytes, linsimp_stream stream);

/*
 * Device-side health word of the last call that used `workspace` (the paper has no
 * counterpart).  Every wait inside the kernels (on an mbarrier fed by a bulk copy or by the
 * tensor cores) is bounded; a wait that gives up records a positive code in the first word
 * of the workspace and the kernel runs to its end with undefined results instead of
 * hanging.  This call copies the word to the host and SYNCHRONISES `stream`.
 * Returns 0 (healthy), a positive wait code, or a negative LINSIMP_E* code.
 * CUDA-core-only calls never write the word.
 */
int linsimp_read_status(const void *workspace, linsimp_stream stream);

/* Static description of an error code.  Host function. */
const char *linsimp_strerror(int code);

/* LINSIMP_VERSION the library was built with.  Host function. */
int linsimp_version(void);

/* Number of kernels the last successful call of the given op enqueued on this
 * host thread's behalf (for launch accounting in benchmarks).  Host function. */
int linsimp_last_launch_count(int op);

/*
 * Forward without a workspace argument, for callers that cannot allocate device memory (the
 * paper has no counterpart).  Hosts that must not call cudaMalloc - a real-time loop where an
 * allocation could stall on the driver, a plug-in that is handed tensors and a stream but no
 * allocator, a process whose device memory was budgeted once at start-up - cannot provide the
 * workspace linsimp_fwd asks for.  This variant keeps that scratch in a fixed array inside the
 * library image (LINSIMP_STATIC_SCRATCH_BYTES, 32 MiB, resident on every GPU that loads the
 * library until the process exits) and calls no cudaMalloc, cudaFree or any allocating routine.
 *   - It runs the fp32 CUDA-core forward (as LINSIMP_ALGO_FP32) for either io_dtype; inputs,
 *     outputs and their meaning are exactly those of linsimp_fwd.
 *   - Problems whose workspace (linsimp_workspace_bytes with algo = LINSIMP_ALGO_FP32, op =
 *     LINSIMP_OP_FWD: B*H*ceil(T/32)*(m*d+m)*4 bytes) exceeds the array are refused with
 *     LINSIMP_ETOOLARGE before anything is launched.
 *   - The first call on each device looks up the array's device address (with that device
 *     current).  With CUDA's lazy module loading that look-up is also what loads the part of
 *     the library that holds the array, so the driver reserves the 32 MiB - and may stall for
 *     it - inside that first call.  Make it once at start-up, outside any time-critical loop
 *     and before starting any stream capture; later calls only read a cached address.
 *   - All calls on a device share the one array.  It keeps the previous call's contents, which
 *     is harmless: every element a call reads it has written first, so nothing needs clearing.
 *     But two calls whose kernels overlap in time on the GPU (different streams, no ordering)
 *     race on it; order such calls yourself.
 */
#define LINSIMP_STATIC_SCRATCH_BYTES (32u << 20)
int linsimp_fwd_static(const linsimp_params *p,
                       const void *q, const void *k, const void *v, const void *r, const void *u,
                       const float *omega,
                       void *o, float *rowmax_L, float *lse,
                       float *S_final, float *z_final, linsimp_stream stream);

/*
 * Per-kernel timing for benchmarks (the paper has no counterpart).  While
 * enabled on the calling host thread, every kernel the library launches from
 * that thread is bracketed by CUDA events on the launching stream.
 * linsimp_profile_enable(1) clears earlier records; linsimp_profile_read
 * synchronises on the recorded events and returns the number of distinct
 * kernel names; for 0 <= index < that number it fills name (NUL-terminated,
 * truncated to name_len), the summed device time in ms and the launch count.
 * Any output pointer may be NULL.  Returns a negative code on a CUDA error.
 */
int linsimp_profile_enable(int on);
int linsimp_profile_read(int index, char *name, int name_len, float *total_ms, int *launches);

#ifdef __cplusplus
}
#endif
#endif /* LINSIMP_H */
