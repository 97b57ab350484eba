/*
 * linsimp_debug.h - test-support entry points of liblinsimp.so (the paper has no counterpart).
 *
 * They exist so that the GPU tests can pin two things the production kernels rely on and that
 * no public call exposes: the tcgen05 descriptor encodings / swizzled operand layouts, and the
 * behaviour of a bounded device-side wait that runs out.  Plain device pointers and sizes; the
 * caller owns every buffer; nothing is allocated; all work is enqueued on `stream`.
 */
#ifndef LINSIMP_DEBUG_H
#define LINSIMP_DEBUG_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* One accumulation chain of tensor-core products D[128][N] = sum_k A_k . B_k^T on caller-built
 * operand images, described the way the kernels describe theirs. */
typedef struct linsimp_umma_probe {
    uint32_t idesc;                 /* instruction descriptor (kind::f16) */
    uint32_t a_lbo, a_sbo, a_layout;/* shared-memory descriptor fields of A: byte strides, swizzle code */
    uint32_t b_lbo, b_sbo, b_layout;/* same for B */
    int32_t nk;                     /* K steps of 16, 1..16 */
    int32_t a_koff[16], b_koff[16]; /* per K step: byte offset into the image (A from tensor memory: column offset) */
    int32_t a_bytes, b_bytes;       /* image sizes, multiples of 16 */
    int32_t n_out;                  /* accumulator columns to read back, a multiple of 16, <= N */
    int32_t a_from_tmem;            /* 1: the A image is [128][a_bytes/512] 32-bit words per row, held in tensor memory */
} linsimp_umma_probe;

/*
 * Runs the chain on device images a_img, b_img (16-byte aligned) and writes the fp32
 * accumulator to out [128][n_out].  Only descriptors of the forms the library's own kernels
 * build are accepted (kind::f16, fp32 accumulator, fp16 or bf16 for both operands, M = 128,
 * N a multiple of 16 up to 256, 32/64/128-byte swizzle, K steps inside the image); anything
 * else returns -2 before a launch.  -1: null pointer or size out of range; -5: CUDA error.
 * `status` (two device ints, nullable): [0] receives code 1 if the kernel's wait on the product gives up, [1] the
 * clock ticks from the first issue to the completion of the chain.
 */
int linsimp_debug_umma(const void *a_img, const void *b_img, const linsimp_umma_probe *probe, float *out,
                       int *status, void *stream);

/*
 * Launches a one-warp kernel that waits, for at most `limit` polls (1..65536), on a barrier
 * nothing ever arrives at.  The wait gives up, the kernel writes `code` (> 0) to *status
 * (device int) and 1 to *gave_up (device int, nullable) and returns normally: the path a
 * production kernel takes when a copy or a product it waits for never completes (see
 * linsimp_read_status).  No fault, trap or endless loop is involved; the context stays usable.
 * Returns 0, -1 (bad argument) or -5 (CUDA error).
 */
int linsimp_debug_wait_expiry(int *status, int code, unsigned limit, int *gave_up, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* LINSIMP_DEBUG_H */
