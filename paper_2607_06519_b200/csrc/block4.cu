// Depth blocks of four layers (Eq. 1 with B = 4, the orthonormal DCT-II of size 4).
//
// The first row of F_4 is (1/2, 1/2, 1/2, 1/2): the shared coefficient is Z0 = (x0 + x1 + x2 + x3) / 2 and its
// contribution to every layer is Z0 / 2, the block mean.  Because F_4 is orthonormal the three high-frequency
// coefficients of a position contribute x_l - mean to layer l and their squared sum equals sum_l (x_l - mean)^2.
// The library therefore stages, per position, Z0, the four layer-space deviations dev_l = x_l - Z0 / 2 and the
// energy e = sum_l dev_l^2; the three high-frequency groups share one kept set per tensor (Eq. 3), the k positions
// of largest energy (ties to the lowest index), found by the float32 radix select of compress.cu on e.
// A decode call for layer l then reads one value per kept position (dev_l) instead of three coefficients.
//
// Stored arithmetic (float32, never contracted):  s = (x0 + x1) + (x2 + x3);  z0 = rs(0.5 s);
// dev_l = rs(x_l - 0.5 z0);  e = (dev_0^2 + dev_1^2) + (dev_2^2 + dev_3^2)  with rs = rounding to the storage type.
#include <algorithm>

#include "fdkv_internal.h"

namespace fdkv {

namespace {

template <typename T>
struct Vec;
template <>
struct Vec<float> {
    static constexpr int N = 4;
    using raw = float4;
    __device__ static void unpack(const raw& v, float (&f)[N]) { f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w; }
    __device__ static raw pack(const float (&f)[N]) { return make_float4(f[0], f[1], f[2], f[3]); }
    __device__ static float rs(float x) { return x; }
};
template <>
struct Vec<__nv_bfloat16> {
    static constexpr int N = 8;
    using raw = uint4;
    __device__ static void unpack(const raw& v, float (&f)[N]) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    __device__ static raw pack(const float (&f)[N]) {  // values already representable in bf16
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) w[i] = (__float_as_uint(f[2 * i]) >> 16) | (__float_as_uint(f[2 * i + 1]) & 0xFFFF0000u);
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
    __device__ static float rs(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }
};

// grid (chunks, Hkv * 2): each CTA owns a token range of one unit-tensor and a private histogram of the energies'
// top 15 magnitude bits (the first pass of the float32 radix select).
template <typename T>
__global__ void __launch_bounds__(512) split4_hist_kernel(Split4Args a, int tokens_per_cta) {
    extern __shared__ uint32_t s_hist[];
    using V = Vec<T>;
    constexpr int N = V::N;
    for (int b = threadIdx.x; b < kHistBins; b += blockDim.x) s_hist[b] = 0;
    __syncthreads();
    const int h = blockIdx.y >> 1, is_v = blockIdx.y & 1;
    const int ut = a.ut_base + blockIdx.y;
    const T* x[4];
#pragma unroll
    for (int l = 0; l < 4; ++l) x[l] = reinterpret_cast<const T*>(is_v ? a.v[l] : a.k[l]) + (int64_t)h * a.stride_h;
    T* z0 = reinterpret_cast<T*>(a.z0) + (int64_t)ut * a.unit_stride;
    T* dev = reinterpret_cast<T*>(a.dev) + (int64_t)ut * 4 * a.unit_stride;
    float* en = a.energy + (int64_t)ut * a.unit_stride;
    T* drop = (a.drop && !is_v) ? reinterpret_cast<T*>(a.drop) + (int64_t)(ut >> 1) * 4 * a.unit_stride : nullptr;

    const int t_begin = blockIdx.x * tokens_per_cta;
    const int t_end = min(a.T, t_begin + tokens_per_cta);
    const int vpr = a.d / N;
    const int64_t nvec = (int64_t)max(0, t_end - t_begin) * vpr;
    for (int64_t v = threadIdx.x; v < nvec; v += blockDim.x) {
        const int t = t_begin + (int)(v / vpr);
        const int cv = (int)(v % vpr) * N;
        const int64_t off_in = (int64_t)t * a.stride_t + cv, off_out = (int64_t)t * a.d + cv;
        typename V::raw r[4];
#pragma unroll
        for (int l = 0; l < 4; ++l) r[l] = *reinterpret_cast<const typename V::raw*>(x[l] + off_in);
        float f[4][N], z[N], e[N], dv[4][N];
#pragma unroll
        for (int l = 0; l < 4; ++l) V::unpack(r[l], f[l]);
#pragma unroll
        for (int i = 0; i < N; ++i) {
            const float s = __fadd_rn(__fadd_rn(f[0][i], f[1][i]), __fadd_rn(f[2][i], f[3][i]));
            z[i] = V::rs(__fmul_rn(0.5f, s));
            const float half = __fmul_rn(0.5f, z[i]);  // exact
#pragma unroll
            for (int l = 0; l < 4; ++l) dv[l][i] = V::rs(__fsub_rn(f[l][i], half));
            e[i] = __fadd_rn(__fadd_rn(__fmul_rn(dv[0][i], dv[0][i]), __fmul_rn(dv[1][i], dv[1][i])),
                             __fadd_rn(__fmul_rn(dv[2][i], dv[2][i]), __fmul_rn(dv[3][i], dv[3][i])));
        }
        *reinterpret_cast<typename V::raw*>(z0 + off_out) = V::pack(z);
#pragma unroll
        for (int l = 0; l < 4; ++l) {
            const typename V::raw pk = V::pack(dv[l]);
            *reinterpret_cast<typename V::raw*>(dev + (int64_t)l * a.unit_stride + off_out) = pk;
            if (drop) *reinterpret_cast<typename V::raw*>(drop + (int64_t)l * a.unit_stride + off_out) = pk;
        }
#pragma unroll
        for (int i = 0; i < N; i += 4)
            *reinterpret_cast<float4*>(en + off_out + i) = make_float4(e[i], e[i + 1], e[i + 2], e[i + 3]);
#pragma unroll
        for (int i = 0; i < N; ++i) atomicAdd(&s_hist[(__float_as_uint(e[i]) & 0x7FFFFFFFu) >> 16], 1u);
    }
    __syncthreads();
    uint32_t* gh = a.hist + (int64_t)ut * kHistBins;
    for (int b = threadIdx.x; b < kHistBins; b += blockDim.x) {
        const uint32_t c = s_hist[b];
        if (c) atomicAdd(&gh[b], c);
    }
}

// Packed entry of the bf16 / head_dim 128 decode kernel (same format as the pair path writes): low half = value
// bits, high half = (byte offset / 2) of the position inside a 16-token x 128-channel tile of two 64-channel halves
// with 128-byte rows whose 16-byte chunks are XOR-swizzled with the row.
__device__ __forceinline__ uint32_t packed_entry_bf16(float v, int flat) {
    const int row = (flat >> 7) & 15, ch = flat & 127;
    const uint32_t off = (uint32_t)((ch >> 6) * 2048 + row * 128 + ((((ch >> 3) & 7) ^ (row & 7)) << 4) + (ch & 7) * 2);
    return (__float_as_uint(v) >> 16) | ((off >> 1) << 16);
}

// grid (ceil(k / 256), unit-tensors): the four layers' values at the kept positions, in list order
template <typename T>
__global__ void __launch_bounds__(256) gather4_kernel(Gather4Args a) {
    const int ut = a.ut_begin + blockIdx.y;
    const int64_t w = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (w >= a.k) return;
    const int i = a.idx[(int64_t)ut * a.kcap + w];
    const T* dev = reinterpret_cast<const T*>(a.dev) + (int64_t)ut * 4 * a.unit_stride;
    T* val = reinterpret_cast<T*>(a.val) + (int64_t)ut * 4 * a.kcap;
    // K tensors: the copy of the deviations that the residual candidate of the probe misses loses its kept positions
    T* drop = (a.drop && !(ut & 1)) ? reinterpret_cast<T*>(a.drop) + (int64_t)(ut >> 1) * 4 * a.unit_stride : nullptr;
#pragma unroll
    for (int l = 0; l < 4; ++l) {
        const T v = dev[(int64_t)l * a.unit_stride + i];
        val[(int64_t)l * a.kcap + w] = v;
        if (drop) drop[(int64_t)l * a.unit_stride + i] = T(0.f);
        if constexpr (sizeof(T) == 2) {
            // the decode kernel scales the rows by 1/2 and the residual by the same factor: store twice the deviation
            if (a.packed) a.packed[((int64_t)ut * 4 + l) * a.kcap + w] = packed_entry_bf16(2.f * __bfloat162float(v), i);
        }
    }
}

}  // namespace

cudaError_t launch_split4_hist(const Split4Args& a, int dtype, cudaStream_t st) {
    static PerDevice once;
    const size_t smem = (size_t)kHistBins * sizeof(uint32_t);
    cudaError_t e0 = once.ensure([&]() {
        cudaError_t e = cudaFuncSetAttribute(split4_hist_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        return cudaFuncSetAttribute(split4_hist_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    });
    if (e0 != cudaSuccess) return e0;
    if (a.T <= 0) return cudaSuccess;
    const int tokens_per_cta = 2048 * 128 / a.d / (dtype == FDKV_BF16 ? 1 : 2);
    dim3 grid((a.T + tokens_per_cta - 1) / tokens_per_cta, a.Hkv * 2);
    if (dtype == FDKV_BF16)
        split4_hist_kernel<__nv_bfloat16><<<grid, 512, smem, st>>>(a, tokens_per_cta);
    else
        split4_hist_kernel<float><<<grid, 512, smem, st>>>(a, tokens_per_cta);
    count_launch(1);
    return cudaGetLastError();
}

cudaError_t launch_gather4(const Gather4Args& a, int dtype, cudaStream_t st) {
    if (a.ut_count <= 0 || a.k <= 0) return cudaSuccess;
    dim3 grid((unsigned)((a.k + 255) / 256), a.ut_count);
    if (dtype == FDKV_BF16)
        gather4_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(a);
    else
        gather4_kernel<float><<<grid, 256, 0, st>>>(a);
    count_launch(1);
    return cudaGetLastError();
}

}  // namespace fdkv
