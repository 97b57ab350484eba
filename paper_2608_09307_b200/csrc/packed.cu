// Packed (cu_seqlens) batches: sequences of different lengths laid end to end in one token buffer.  The estimator's
// kernels walk one (batch, head) unit as a contiguous run of T rows, so a packed batch is brought into the padded form
// [B][H][T][d] (T = the longest sequence), run through the padded-batch kernels, and the results are gathered back.
// Only data movement lives here; the rows are copied in 16-byte pieces where the row size allows it.
#include "packed.h"

#include <string.h>

#include <type_traits>

#include "common.cuh"
#include "launch.cuh"

namespace linsimp {

__global__ void k_packed_lens(const int32_t *__restrict__ cu, int B, int T, int32_t *__restrict__ lens)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B) lens[b] = min(max(cu[b + 1] - cu[b], 0), T);
}

// grid (ceil(T * pieces / 256), H, B); VEC = bytes per piece (16 or the element size for odd rows)
template <int VEC, bool UNPACK>
__global__ void __launch_bounds__(256) k_packed_move(const uint8_t *__restrict__ src, uint8_t *__restrict__ dst,
                                                     const int32_t *__restrict__ cu, int H, int T, long total, int row_bytes)
{
    const int b = blockIdx.z, h = blockIdx.y;
    const int pieces = row_bytes / VEC;
    const long idx = (long)blockIdx.x * 256 + threadIdx.x;
    if (idx >= (long)T * pieces) return;
    const int t = (int)(idx / pieces), pc = (int)(idx - (long)t * pieces);
    const long first = cu[b];
    const int len = min(max(cu[b + 1] - cu[b], 0), T);
    const long padded_off = (((long)b * H + h) * T + t) * row_bytes + (long)pc * VEC;
    const long packed_off = ((long)h * total + first + t) * row_bytes + (long)pc * VEC;
    typedef typename std::conditional<VEC == 16, uint4, typename std::conditional<VEC == 4, uint32_t, uint16_t>::type>::type V;
    if (UNPACK) {
        V val;
        memset(&val, 0, sizeof(V));
        if (t < len) val = *(const V *)(src + packed_off);
        *(V *)(dst + padded_off) = val;
    } else if (t < len) {
        *(V *)(dst + packed_off) = *(const V *)(src + padded_off);
    }
}

// grid (W, H, B), one block per ring slot; row_bytes a multiple of 4
__global__ void __launch_bounds__(64) k_packed_ring_fill(const uint8_t *__restrict__ r, const uint8_t *__restrict__ u,
                                                         const int32_t *__restrict__ cu, int H, long total, int W, int row_bytes,
                                                         uint8_t *__restrict__ ring_r, uint8_t *__restrict__ ring_u)
{
    const int slot = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const long first = cu[b];
    const int len = max(cu[b + 1] - cu[b], 0);
    if (len <= slot && len <= W) return;                   // fewer tokens than this slot's index: the slot stays as it is
    // the latest token t < len with t % W == slot
    const int t = slot + ((len - 1 - slot) / W) * W;
    if (t < 0 || t < len - W) return;
    const long src = ((long)h * total + first + t) * row_bytes;
    const long dst = (((long)b * H + h) * W + slot) * row_bytes;
    for (int x = threadIdx.x * 4; x < row_bytes; x += 64 * 4) {
        *(uint32_t *)(ring_r + dst + x) = *(const uint32_t *)(r + src + x);
        *(uint32_t *)(ring_u + dst + x) = *(const uint32_t *)(u + src + x);
    }
}

int packed_ring_fill_run(const void *r, const void *u, const int32_t *cu_seqlens, int B, int H, long total, int d, int W,
                         int elem_bytes, void *ring_r, void *ring_u, cudaStream_t st)
{
    LaunchScope sc = {st, 0};
    LS_LAUNCH(sc, "packed_ring_fill", k_packed_ring_fill<<<dim3(W, H, B), 64, 0, st>>>(
        (const uint8_t *)r, (const uint8_t *)u, cu_seqlens, H, total, W, d * elem_bytes, (uint8_t *)ring_r, (uint8_t *)ring_u));
    return sc.result();
}

int packed_lens_run(const int32_t *cu_seqlens, int B, int T, int32_t *seq_lens, cudaStream_t st)
{
    LaunchScope sc = {st, 0};
    LS_LAUNCH(sc, "packed_lens", k_packed_lens<<<(B + 255) / 256, 256, 0, st>>>(cu_seqlens, B, T, seq_lens));
    return sc.result();
}

template <bool UNPACK>
static int move_run(const void *src, void *dst, const int32_t *cu, int B, int H, int T, long total, int width, int elem_bytes,
                    cudaStream_t st)
{
    LaunchScope sc = {st, 0};
    const int row_bytes = width * elem_bytes;
    const char *name = UNPACK ? "packed_unpack" : "packed_pack";
    if (row_bytes % 16 == 0) {
        const long n = (long)T * (row_bytes / 16);
        LS_LAUNCH(sc, name, k_packed_move<16, UNPACK><<<dim3((unsigned)((n + 255) / 256), H, B), 256, 0, st>>>(
            (const uint8_t *)src, (uint8_t *)dst, cu, H, T, total, row_bytes));
    } else if (elem_bytes == 4) {
        const long n = (long)T * width;
        LS_LAUNCH(sc, name, k_packed_move<4, UNPACK><<<dim3((unsigned)((n + 255) / 256), H, B), 256, 0, st>>>(
            (const uint8_t *)src, (uint8_t *)dst, cu, H, T, total, row_bytes));
    } else {
        const long n = (long)T * width;
        LS_LAUNCH(sc, name, k_packed_move<2, UNPACK><<<dim3((unsigned)((n + 255) / 256), H, B), 256, 0, st>>>(
            (const uint8_t *)src, (uint8_t *)dst, cu, H, T, total, row_bytes));
    }
    return sc.result();
}

int packed_unpack_run(const void *packed, const int32_t *cu_seqlens, int B, int H, int T, long total, int width, int elem_bytes,
                      void *padded, cudaStream_t st)
{
    return move_run<true>(packed, padded, cu_seqlens, B, H, T, total, width, elem_bytes, st);
}

int packed_pack_run(const void *padded, const int32_t *cu_seqlens, int B, int H, int T, long total, int width, int elem_bytes,
                    void *packed, cudaStream_t st)
{
    return move_run<false>(padded, packed, cu_seqlens, B, H, T, total, width, elem_bytes, st);
}

}  // namespace linsimp
