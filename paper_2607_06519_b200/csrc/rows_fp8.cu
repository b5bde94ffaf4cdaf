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

// All row streams of a commit are quantised by four launches over a job table (one job per stored tensor).
// grid (token chunks, jobs): per-channel maximum of |x| over the chunk, merged with atomicMax on the bit patterns
// (non-negative floats order like their bits); the maxima live in the second half of the job's 1 KiB scale slot.
__global__ void __launch_bounds__(128) zero_amax_kernel(const QuantJob* jobs) {
    reinterpret_cast<uint32_t*>(jobs[blockIdx.x].scale)[kD + threadIdx.x] = 0u;
}
__global__ void __launch_bounds__(256) absmax_kernel(const QuantJob* jobs, int rows_per_cta) {
    __shared__ uint32_t s_max[16][kD];
    const QuantJob jb = jobs[blockIdx.y];
    const __nv_bfloat16* src = reinterpret_cast<const __nv_bfloat16*>(jb.src);
    // a thread takes 8 channels (16 bytes) of every 16th row of the chunk
    const int c8 = (threadIdx.x & 15) * 8, rg = threadIdx.x >> 4;
    const int t0 = blockIdx.x * rows_per_cta, t1 = min(jb.T, t0 + rows_per_cta);
    if (t0 >= jb.T) return;
    uint32_t m[4] = {0u, 0u, 0u, 0u};  // two 15-bit magnitudes per word
    for (int t = t0 + rg; t < t1; t += 16) {
        const uint4 raw = *reinterpret_cast<const uint4*>(src + (int64_t)t * jb.stride_t + c8);
        m[0] = __vmaxu2(m[0], raw.x & 0x7FFF7FFFu);
        m[1] = __vmaxu2(m[1], raw.y & 0x7FFF7FFFu);
        m[2] = __vmaxu2(m[2], raw.z & 0x7FFF7FFFu);
        m[3] = __vmaxu2(m[3], raw.w & 0x7FFF7FFFu);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        s_max[rg][c8 + 2 * j] = (m[j] & 0xFFFFu) << 16;  // as float32 bit patterns
        s_max[rg][c8 + 2 * j + 1] = m[j] & 0xFFFF0000u;
    }
    __syncthreads();
    if (threadIdx.x < kD) {
        uint32_t v = 0;
#pragma unroll
        for (int r = 0; r < 16; ++r) v = max(v, s_max[r][threadIdx.x]);
        atomicMax(reinterpret_cast<uint32_t*>(jb.scale) + kD + threadIdx.x, v);
    }
}

// one CTA per job: the channel scales from the maxima
__global__ void __launch_bounds__(128) scale_kernel(const QuantJob* jobs) {
    const QuantJob jb = jobs[blockIdx.x];
    const float amax = __uint_as_float(reinterpret_cast<const uint32_t*>(jb.scale)[kD + threadIdx.x]);
    jb.scale[threadIdx.x] = amax > 0.f ? __fdiv_rn(amax, 448.f) : 1.f;
}

// grid (ceil(T * 16 / 256), jobs): one thread per 8 channels of a token: codes out (8 bytes)
__global__ void __launch_bounds__(256) quantise_kernel(const QuantJob* jobs) {
    const QuantJob jb = jobs[blockIdx.y];
    const __nv_bfloat16* src = reinterpret_cast<const __nv_bfloat16*>(jb.src);
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int t = (int)(i >> 4), c8 = (int)(i & 15) * 8;
    if (t >= jb.T) return;
    const uint4 raw = *reinterpret_cast<const uint4*>(src + (int64_t)t * jb.stride_t + c8);
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
    const float4 s0 = *reinterpret_cast<const float4*>(jb.scale + c8), s1 = *reinterpret_cast<const float4*>(jb.scale + c8 + 4);
    const float scv[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
    uint32_t out[2] = {0u, 0u};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const float sc = scv[j];
        const float x = __uint_as_float((j & 1) ? (w[j >> 1] & 0xFFFF0000u) : (w[j >> 1] << 16));
        const uint32_t code = (uint32_t)__nv_cvt_float_to_fp8(__fdiv_rn(x, sc), __NV_SATFINITE, __NV_E4M3);
        out[j >> 2] |= code << (8 * (j & 3));
    }
    *reinterpret_cast<uint2*>(jb.codes + (int64_t)t * kD + c8) = make_uint2(out[0], out[1]);
}

// Position of channel c inside its 16-channel group as the decode kernel's converted fragments see it.
// K: a 4-byte register holds channels 4j..4j+3 of a token; its low pair feeds k-slots (2j, 2j+1), its high pair
//    (2j+8, 2j+9) of the m16n8k16 A operand.
// V: a 2-byte unit holds channels (2j, 2j+1) of a token; after the transposing load they become rows j and j + 8.
__device__ __forceinline__ int slot_k(int c) { return 2 * (c >> 2) + (c & 1) + 8 * ((c >> 1) & 1); }
__device__ __forceinline__ int slot_v(int c) { return (c >> 1) + 8 * (c & 1); }

// grid (ceil(n / 256), jobs)
__global__ void __launch_bounds__(256) repack_entries_f8_kernel(const RepackJob* jobs) {
    const RepackJob jb = jobs[blockIdx.y];
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (jb.rows) {
        // token rule: one warp per kept row, a lane per four channels; the whole row is read before any of it is written
        const int64_t row = i >> 5;
        if (row >= jb.n) return;  // (warp-uniform)
        const int lane = threadIdx.x & 31;
        uint16_t* const r16 = reinterpret_cast<uint16_t*>(jb.dst) + row * kD;
        const uint2 in = *reinterpret_cast<const uint2*>(r16 + 4 * lane);
        const uint32_t w2[2] = {in.x, in.y};
        __syncwarp();
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int ch = 4 * lane + j;
            const float v = __uint_as_float((j & 1) ? (w2[j >> 1] & 0xFFFF0000u) : (w2[j >> 1] << 16));
            const int cs = (ch & ~15) + (jb.is_v ? slot_v(ch & 15) : slot_k(ch & 15));
            r16[cs] = __half_as_ushort(__float2half_rn(__fdiv_rn(v, jb.scale[ch])));
        }
        return;
    }
    if (i >= jb.n) return;
    const uint32_t w = jb.src[i];
    // undo the pair-path offset: byte offset / 2 = half << 10 | row << 6 | (chunk ^ row) << 3 | ch & 7
    const uint32_t off2 = w >> 16;
    const int row = (off2 >> 6) & 15, half = off2 >> 10, chunk = ((off2 >> 3) ^ (off2 >> 6)) & 7, ch = half * 64 + chunk * 8 + (off2 & 7);
    const int g = ch & ~15, cs = g + (jb.is_v ? slot_v(ch & 15) : slot_k(ch & 15));
    const uint32_t off = (uint32_t)((cs >> 6) * 2048 + row * 128 + ((((cs >> 3) & 7) ^ (row & 7)) << 4) + (cs & 7) * 2);
    const float v = __uint_as_float((w & 0xFFFFu) << 16);
    const __half hv = __float2half_rn(__fdiv_rn(v, jb.scale[ch]));
    jb.dst[i] = (uint32_t)__half_as_ushort(hv) | ((off >> 1) << 16);
}

}  // namespace

cudaError_t launch_quantise_jobs(const QuantJob* jobs_dev, int njobs, int T_max, cudaStream_t st) {
    if (njobs <= 0 || T_max <= 0) return cudaSuccess;
    const int rows_per_cta = 1024;
    zero_amax_kernel<<<njobs, kD, 0, st>>>(jobs_dev);
    absmax_kernel<<<dim3((T_max + rows_per_cta - 1) / rows_per_cta, njobs), 256, 0, st>>>(jobs_dev, rows_per_cta);
    scale_kernel<<<njobs, kD, 0, st>>>(jobs_dev);
    const int64_t threads = (int64_t)T_max * 16;
    quantise_kernel<<<dim3((unsigned)((threads + 255) / 256), njobs), 256, 0, st>>>(jobs_dev);
    count_launch(4);
    return cudaGetLastError();
}

cudaError_t launch_repack_jobs(const RepackJob* jobs_dev, int njobs, int64_t n_max, cudaStream_t st) {
    if (njobs <= 0 || n_max <= 0) return cudaSuccess;
    repack_entries_f8_kernel<<<dim3((unsigned)((n_max + 255) / 256), njobs), 256, 0, st>>>(jobs_dev);
    count_launch(1);
    return cudaGetLastError();
}

}  // namespace fdkv
