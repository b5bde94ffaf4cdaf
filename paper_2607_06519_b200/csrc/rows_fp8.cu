// 8-bit row streams: the composition with quantisation mentioned after Eq. 3 (the paper fixes no scheme; this build's
// reading is stated in fdkv.h): the dense rows a committed unit streams at decode time (Z0 of shared / residual units,
// the original rows of exact units) become e4m3 codes with one float32 scale per channel of each stored tensor,
//     scale_c = max_t |R[t][c]| / 448 (float32 division; 1 when the maximum is 0),
//     code    = e4m3(R[t][c] / scale_c) (float32 division, nearest even, saturating).
// bf16 storage, head_dim 128.
#include <cuda_fp8.h>
#include <cuda_fp16.h>

#include "fdkv_internal.h"

namespace fdkv {

namespace {

constexpr int kD = 128;

// grid (token chunks): per-channel maximum of |x| over the chunk, merged with atomicMax on the bit patterns
// (non-negative floats order like their bits).  amax must start at zero.
__global__ void __launch_bounds__(256) absmax_kernel(const __nv_bfloat16* src, int64_t stride_t, int T, int rows_per_cta,
                                                     uint32_t* amax_bits) {
    __shared__ uint32_t s_max[2][kD];
    const int c = threadIdx.x & (kD - 1), half = threadIdx.x >> 7;
    const int t0 = blockIdx.x * rows_per_cta, t1 = min(T, t0 + rows_per_cta);
    uint32_t m = 0;
    for (int t = t0 + half; t < t1; t += 2) {
        const uint32_t b = (uint32_t)__bfloat16_as_ushort(src[(int64_t)t * stride_t + c]) << 16;
        m = max(m, b & 0x7FFFFFFFu);
    }
    s_max[half][c] = m;
    __syncthreads();
    if (half == 0) atomicMax(&amax_bits[c], max(s_max[0][c], s_max[1][c]));
}

// one thread per 8 channels of a token: scale from the maxima, codes out (8 bytes per store)
__global__ void __launch_bounds__(256) quantise_kernel(const __nv_bfloat16* src, int64_t stride_t, int T, const uint32_t* amax_bits,
                                                       uint8_t* codes, float* scale_out) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int t = (int)(i >> 4), c8 = (int)(i & 15) * 8;
    if (t >= T) return;
    const uint4 raw = *reinterpret_cast<const uint4*>(src + (int64_t)t * stride_t + c8);
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
    uint32_t out[2] = {0u, 0u};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const float amax = __uint_as_float(amax_bits[c8 + j]);
        const float sc = amax > 0.f ? __fdiv_rn(amax, 448.f) : 1.f;
        const float x = __uint_as_float((j & 1) ? (w[j >> 1] & 0xFFFF0000u) : (w[j >> 1] << 16));
        const uint32_t code = (uint32_t)__nv_cvt_float_to_fp8(__fdiv_rn(x, sc), __NV_SATFINITE, __NV_E4M3);
        out[j >> 2] |= code << (8 * (j & 3));
        if (t == 0) scale_out[c8 + j] = sc;
    }
    *reinterpret_cast<uint2*>(codes + (int64_t)t * kD + c8) = make_uint2(out[0], out[1]);
}

// Position of channel c inside its 16-channel group as the decode kernel's converted fragments see it.
// K: a 4-byte register holds channels 4j..4j+3 of a token; its low pair feeds k-slots (2j, 2j+1), its high pair
//    (2j+8, 2j+9) of the m16n8k16 A operand.
// V: a 2-byte unit holds channels (2j, 2j+1) of a token; after the transposing load they become rows j and j + 8.
__device__ __forceinline__ int slot_k(int c) { return 2 * (c >> 2) + (c & 1) + 8 * ((c >> 1) & 1); }
__device__ __forceinline__ int slot_v(int c) { return (c >> 1) + 8 * (c & 1); }

__global__ void __launch_bounds__(256) repack_entries_f8_kernel(uint32_t* dst, const uint32_t* src, int64_t n, const float* scale,
                                                                int is_v) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const uint32_t w = src[i];
    // undo the pair-path offset: byte offset / 2 = half << 10 | row << 6 | (chunk ^ row) << 3 | ch & 7
    const uint32_t off2 = w >> 16;
    const int row = (off2 >> 6) & 15, half = off2 >> 10, chunk = ((off2 >> 3) ^ (off2 >> 6)) & 7, ch = half * 64 + chunk * 8 + (off2 & 7);
    const int g = ch & ~15, cs = g + (is_v ? slot_v(ch & 15) : slot_k(ch & 15));
    const uint32_t off = (uint32_t)((cs >> 6) * 2048 + row * 128 + ((((cs >> 3) & 7) ^ (row & 7)) << 4) + (cs & 7) * 2);
    const float v = __uint_as_float((w & 0xFFFFu) << 16);
    const __half hv = __float2half_rn(__fdiv_rn(v, scale[ch]));
    dst[i] = (uint32_t)__half_as_ushort(hv) | ((off >> 1) << 16);
}

}  // namespace

cudaError_t launch_quantise_rows(const void* src, int64_t stride_t, int T, uint8_t* codes, float* scale, cudaStream_t st) {
    if (T <= 0) return cudaSuccess;
    // the caller's scale slot is 1 KiB: [0, 512) the float32 scales, [512, 1024) the channel maxima (bit patterns)
    uint32_t* amax = reinterpret_cast<uint32_t*>(scale) + kD;
    cudaError_t e = cudaMemsetAsync(amax, 0, kD * sizeof(uint32_t), st);
    if (e != cudaSuccess) return e;
    const int rows_per_cta = 256;
    absmax_kernel<<<(T + rows_per_cta - 1) / rows_per_cta, 256, 0, st>>>(reinterpret_cast<const __nv_bfloat16*>(src), stride_t, T,
                                                                         rows_per_cta, amax);
    const int64_t threads = (int64_t)T * 16;
    quantise_kernel<<<(unsigned)((threads + 255) / 256), 256, 0, st>>>(reinterpret_cast<const __nv_bfloat16*>(src), stride_t, T, amax,
                                                                        codes, scale);
    count_launch(2);
    return cudaGetLastError();
}

cudaError_t launch_repack_entries_f8(uint32_t* dst, const uint32_t* src, int64_t n, const float* scale, int is_v, cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    repack_entries_f8_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(dst, src, n, scale, is_v);
    count_launch(1);
    return cudaGetLastError();
}

}  // namespace fdkv
