// Host-side interface of the packed-batch (cu_seqlens) data movement kernels (internal to the library).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace linsimp {

// seq_lens[b] = cu_seqlens[b + 1] - cu_seqlens[b] (clamped to [0, T]); one launch
int packed_lens_run(const int32_t *cu_seqlens, int B, int T, int32_t *seq_lens, cudaStream_t st);
// rows of `elem_bytes`-sized elements, `width` elements per row: packed [H][total][width] -> padded [B][H][T][width]
// (rows at or beyond a sequence's length are zero), and back (only the sequences' own rows are written)
int packed_unpack_run(const void *packed, const int32_t *cu_seqlens, int B, int H, int T, long total, int width, int elem_bytes,
                      void *padded, cudaStream_t st);
int packed_pack_run(const void *padded, const int32_t *cu_seqlens, int B, int H, int T, long total, int width, int elem_bytes,
                    void *packed, cudaStream_t st);

// decode ring from a packed batch: for t in [max(0, len_b - W), len_b) the rows r[h][cu[b] + t], u[...] go to slot t % W
int packed_ring_fill_run(const void *r, const void *u, const int32_t *cu_seqlens, int B, int H, long total, int d, int W,
                         int elem_bytes, void *ring_r, void *ring_u, cudaStream_t st);

}  // namespace linsimp
