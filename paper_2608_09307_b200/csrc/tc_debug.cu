// Bring-up probe for the tcgen05 path: runs one accumulation chain of UMMA instructions on
// operand images and descriptors supplied by the caller and returns the fp32 accumulator.
// Used by the GPU tests to pin the descriptor encodings and the swizzled operand layouts
// the production kernels rely on.  Only the encodings those kernels build are accepted: anything
// else is refused on the host, so that no unchecked descriptor ever reaches the tensor cores.
// A second probe exercises the give-up path of the bounded waits.  Declared in linsimp_debug.h.
#include "../../include/linsimp_debug.h"
#include "common.cuh"
#include "tc_common.cuh"

namespace linsimp {

typedef linsimp_umma_probe UmmaProbe;

__global__ void __launch_bounds__(128) k_umma_probe(const uint4 *__restrict__ a_img, const uint4 *__restrict__ b_img,
                                                    UmmaProbe pr, float *__restrict__ out, int *status)
{
    using namespace tc;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *base = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *a_s = base;
    uint8_t *b_s = base + ((pr.a_bytes + 1023) & ~1023);
    __shared__ uint64_t bar;
    __shared__ uint32_t tmem_base_s;
    const int warp = threadIdx.x >> 5;
    if (warp == 0) {
        tmem_alloc(&tmem_base_s, 512);
        tmem_relinquish();
    }
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        fence_barrier_init();
    }
    if (!pr.a_from_tmem)
        for (int i = threadIdx.x; i < pr.a_bytes / 16; i += 128) ((uint4 *)a_s)[i] = a_img[i];
    for (int i = threadIdx.x; i < pr.b_bytes / 16; i += 128) ((uint4 *)b_s)[i] = b_img[i];
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = tmem_base_s;
    const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
    if (pr.a_from_tmem) {
        const int words = pr.a_bytes / 512;              // 32-bit words per row
        const uint32_t *arow = (const uint32_t *)a_img + (size_t)threadIdx.x * words;
        for (int c0 = 0; c0 < words; c0 += 32) {
            uint32_t r[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) r[j] = arow[c0 + j];
            tmem_st32(tbase + lane_off + 256 + c0, r);
        }
        tmem_st_wait();
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
    }
    long long t_issue = 0;
    if (threadIdx.x == 0) {
        t_issue = clock64();
        for (int k = 0; k < pr.nk; ++k) {
            const uint64_t bd = make_smem_desc(smem_u32(b_s) + pr.b_koff[k], pr.b_lbo, pr.b_sbo, pr.b_layout);
            if (pr.a_from_tmem) {
                mma_f16_ts(tbase, tbase + 256 + pr.a_koff[k], bd, pr.idesc, k > 0);
            } else {
                const uint64_t ad = make_smem_desc(smem_u32(a_s) + pr.a_koff[k], pr.a_lbo, pr.a_sbo, pr.a_layout);
                mma_f16_ss(tbase, ad, bd, pr.idesc, k > 0);
            }
        }
        tc_commit(&bar);
    }
    mbar_wait(&bar, 0, status, 1);
    // clock ticks from the first issue to the completion of the chain as thread 0 sees it (second word of `status`)
    if (threadIdx.x == 0 && status) status[1] = (int)(clock64() - t_issue);
    tc_fence_after();
    for (int c0 = 0; c0 < pr.n_out; c0 += 16) {
        uint32_t r[16];
        tmem_ld16(tbase + lane_off + c0, r);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j) out[(size_t)threadIdx.x * pr.n_out + c0 + j] = __uint_as_float(r[j]);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tbase, 512);
}

}  // namespace linsimp

namespace linsimp {

// A test-only kernel whose single wait can never succeed: the barrier expects one arrival and nothing arrives.  After
// `limit` polls the wait gives up, records `code` in *status and the kernel returns without touching the barrier,
// tensor memory or any copy engine again - the path every production kernel takes when one of its waits runs out.
__global__ void k_wait_expiry(int *status, int code, uint32_t limit, int *polled)
{
    using namespace tc;
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        fence_barrier_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const bool ok = mbar_wait_limit(&bar, 0, status, code, limit);
        if (polled) *polled = ok ? 0 : 1;
    }
}

namespace {
// the instruction descriptors the production kernels build: kind::f16 with an fp32 accumulator, both operands of the
// same 16-bit format, M = 128, N a multiple of 16 up to 256, either operand K-major or MN-major
bool idesc_known(uint32_t d)
{
    const uint32_t fa = (d >> 7) & 7u, fb = (d >> 10) & 7u, n8 = (d >> 17) & 0x3Fu, m16 = (d >> 24) & 0x1Fu;
    const uint32_t known = (1u << 4) | (7u << 7) | (7u << 10) | (1u << 15) | (1u << 16) | (0x3Fu << 17) | (0x1Fu << 24);
    if (d & ~known) return false;
    if (!(d & (1u << 4))) return false;
    if (fa != fb || fa > 1u) return false;
    if (m16 != 8u) return false;
    return n8 >= 2u && n8 <= 32u && (n8 & 1u) == 0u;
}
// shared-memory operands: a swizzled layout the kernels use, strides in whole 16-byte units, every K step inside the image
bool operand_known(uint32_t lbo, uint32_t sbo, uint32_t layout, const int *koff, int nk, int bytes)
{
    if (!(layout == tc::kSw128 || layout == tc::kSw64 || layout == tc::kSw32)) return false;
    if ((lbo & 15u) || (sbo & 15u) || lbo > (1u << 18) || sbo > (1u << 18) || sbo == 0) return false;
    if (bytes < 512 || (bytes & 15)) return false;
    for (int k = 0; k < nk; ++k)
        if (koff[k] < 0 || (koff[k] & 15) || koff[k] >= bytes) return false;
    return true;
}
}  // namespace
}  // namespace linsimp

extern "C" int linsimp_debug_wait_expiry(int *status, int code, unsigned limit, int *gave_up, void *stream)
{
    using namespace linsimp;
    if (!status || code <= 0 || limit < 1 || limit > (1u << 16)) return -1;
    k_wait_expiry<<<1, 32, 0, (cudaStream_t)stream>>>(status, code, limit, gave_up);
    return cudaPeekAtLastError() == cudaSuccess ? 0 : -5;
}

extern "C" int linsimp_debug_umma(const void *a_img, const void *b_img, const linsimp_umma_probe *probe, float *out,
                                  int *status, void *stream)
{
    using namespace linsimp;
    if (!a_img || !b_img || !probe || !out) return -1;
    if (probe->nk < 1 || probe->nk > 16 || probe->n_out < 16 || probe->n_out > 256 || probe->n_out % 16) return -1;
    if (probe->a_bytes < 512 || probe->b_bytes < 512 || (probe->a_bytes & 15) || (probe->b_bytes & 15)) return -1;
    if (!idesc_known(probe->idesc)) return -2;
    if ((int)(((probe->idesc >> 17) & 0x3Fu) << 3) < probe->n_out) return -2;     // reads only columns the product wrote
    if (!operand_known(probe->b_lbo, probe->b_sbo, probe->b_layout, probe->b_koff, probe->nk, probe->b_bytes)) return -2;
    if (probe->a_from_tmem) {
        // A is [128][words] 32-bit words stored to tensor memory behind the accumulator: K-major only, steps inside it
        const int words = probe->a_bytes / 512;
        if ((probe->idesc >> 15) & 1u) return -2;
        if (words < 8 || words > 256 || (words & 31)) return -2;
        for (int k = 0; k < probe->nk; ++k)
            if (probe->a_koff[k] < 0 || probe->a_koff[k] + 8 > words) return -2;
    } else if (!operand_known(probe->a_lbo, probe->a_sbo, probe->a_layout, probe->a_koff, probe->nk, probe->a_bytes)) {
        return -2;
    }
    const size_t smem = 1024 + ((probe->a_bytes + 1023) & ~1023) + ((probe->b_bytes + 1023) & ~1023);
    if (smem > 200 * 1024) return -1;
    if (cudaFuncSetAttribute(k_umma_probe, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return -5;
    k_umma_probe<<<1, 128, smem, (cudaStream_t)stream>>>((const uint4 *)a_img, (const uint4 *)b_img, *probe, out, status);
    return cudaPeekAtLastError() == cudaSuccess ? 0 : -5;
}
