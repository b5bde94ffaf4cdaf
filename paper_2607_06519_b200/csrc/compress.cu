// Prefill compression kernels: depth split (Eq. 1, B = 2) fused with the magnitude histogram and the
// radix-select threshold of the sparse residual (Eq. 3, entry form); the index-ordered compaction that follows
// is select_fused.cu.
#include <algorithm>
#include <mutex>

#include "fdkv_internal.h"

namespace fdkv {

namespace {

__device__ __forceinline__ uint32_t key_of(float x) { return __float_as_uint(x) & 0x7FFFFFFFu; }

// ----- storage traits -------------------------------------------------------------------------------
template <typename T>
struct Store;
template <>
struct Store<float> {
    static constexpr int VEC = 4;
    using vec_t = float4;
    __device__ static void unpack(const vec_t& v, float* f) { f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w; }
    __device__ static vec_t pack(const float* f) { return make_float4(f[0], f[1], f[2], f[3]); }
};
template <>
struct Store<__nv_bfloat16> {
    static constexpr int VEC = 8;
    using vec_t = uint4;
    __device__ static void unpack(const vec_t& v, float* f) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    // f holds float32 values; round each to nearest-even bf16
    __device__ static vec_t pack(const float* f) {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint32_t lo = __bfloat16_as_ushort(__float2bfloat16_rn(f[2 * i]));
            uint32_t hi = __bfloat16_as_ushort(__float2bfloat16_rn(f[2 * i + 1]));
            w[i] = lo | (hi << 16);
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
};

// value as stored, widened back to float32 (exact)
template <typename T>
__device__ __forceinline__ float stored(float x);
template <>
__device__ __forceinline__ float stored<float>(float x) { return x; }
template <>
__device__ __forceinline__ float stored<__nv_bfloat16>(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

// ----- C1: depth split + histogram of the top 15 magnitude bits of z1 ---------------------------------
// grid (chunks, Hkv*tensors, pairs); each CTA owns a token range of one unit-tensor and a private 128 KiB histogram.
template <typename T>
__global__ void __launch_bounds__(1024) split_hist_kernel(CompressArgs a, int tokens_per_cta) {
    extern __shared__ uint32_t s_hist[];
    using S = Store<T>;
    constexpr int VEC = S::VEC;
    for (int b = threadIdx.x; b < kHistBins; b += blockDim.x) s_hist[b] = 0;
    __syncthreads();

    const int h = blockIdx.y / a.tensors, is_v = blockIdx.y % a.tensors, pj = blockIdx.z;
    const int ut = a.ut_base + pj * a.Hkv * a.tensors + blockIdx.y;
    const T* x0 = reinterpret_cast<const T*>(is_v ? a.v0[pj] : a.k0[pj]) + (int64_t)h * a.stride_h;
    const T* x1 = reinterpret_cast<const T*>(is_v ? a.v1[pj] : a.k1[pj]) + (int64_t)h * a.stride_h;
    T* z0 = reinterpret_cast<T*>(a.z0) + (int64_t)ut * a.unit_stride;
    T* z1 = reinterpret_cast<T*>(a.z1) + (int64_t)ut * a.unit_stride;
    const float c32 = __uint_as_float(0x3F3504F3u);

    const int t_begin = blockIdx.x * tokens_per_cta;
    const int t_end = min(a.T, t_begin + tokens_per_cta);
    const int vpr = a.d / VEC;
    const int64_t nvec = (int64_t)max(0, t_end - t_begin) * vpr;
    // two vector pairs in flight per thread: all four loads are issued before the first is used
    for (int64_t v0 = threadIdx.x; v0 < nvec; v0 += 2 * (int64_t)blockDim.x) {
        typename S::vec_t va[2], vb[2];
        int64_t off_in[2], off_out[2];
        bool live[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int64_t v = v0 + (int64_t)u * blockDim.x;
            live[u] = v < nvec;
            const int t = t_begin + (int)(v / vpr);
            const int cv = (int)(v % vpr) * VEC;
            off_in[u] = (int64_t)t * a.stride_t + cv;
            off_out[u] = (int64_t)t * a.d + cv;
            if (live[u]) {
                va[u] = *reinterpret_cast<const typename S::vec_t*>(x0 + off_in[u]);
                vb[u] = *reinterpret_cast<const typename S::vec_t*>(x1 + off_in[u]);
            }
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            if (!live[u]) continue;
            float fa[VEC], fb[VEC], f0[VEC], f1[VEC];
            S::unpack(va[u], fa);
            S::unpack(vb[u], fb);
#pragma unroll
            for (int i = 0; i < VEC; ++i) {
                // one float32 add (subtract), one float32 multiply: never contracted into an FMA
                f0[i] = __fmul_rn(__fadd_rn(fa[i], fb[i]), c32);
                f1[i] = __fmul_rn(__fsub_rn(fa[i], fb[i]), c32);
            }
            *reinterpret_cast<typename S::vec_t*>(z0 + off_out[u]) = S::pack(f0);
            *reinterpret_cast<typename S::vec_t*>(z1 + off_out[u]) = S::pack(f1);
#pragma unroll
            for (int i = 0; i < VEC; ++i) atomicAdd(&s_hist[key_of(stored<T>(f1[i])) >> 16], 1u);
        }
    }
    __syncthreads();
    uint32_t* gh = a.hist + (int64_t)ut * kHistBins;
    for (int b = threadIdx.x; b < kHistBins; b += blockDim.x) {
        const uint32_t c = s_hist[b];
        if (c) atomicAdd(&gh[b], c);
    }
}

// ----- C2: threshold from a histogram --------------------------------------------------------------
// One CTA per unit-tensor.  Scans `nbins` bins from the top: finds the bin where the running count of larger
// keys first reaches k_rem, appends the bin to the prefix and lowers k_rem.  Clears the bins it read.
// On the last pass writes tau (prefix left-aligned to 31 bits) and need.
__global__ void __launch_bounds__(1024) threshold_kernel(uint32_t* hist, SelState* sel, int ut_begin, int nbins,
                                                         int bits, int first, int last, int shift_final,
                                                         uint32_t k_init) {
    __shared__ uint32_t s_tot[32];
    __shared__ uint32_t s_found_bin, s_found_above;
    const int ut = ut_begin + blockIdx.x;
    uint32_t* h = hist + (int64_t)ut * kHistBins;
    SelState st = sel[ut];
    if (first) { st.prefix = 0; st.k_rem = k_init; }
    // Warp w owns the segment of nbins / nwarps bins below nbins - w * seg (warp 0 the largest keys) and reads it in
    // rows of 32 consecutive bins, largest first: lane l of row i holds bin hi - 1 - 32 i - l.
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int seg = nbins / nwarps, rows = seg / 32;  // nbins is a multiple of 32 * nwarps (32768 / 1024 threads, 256 / 256)
    const int hi = nbins - warp * seg;
    uint32_t mine = 0;
    for (int i = 0; i < rows; ++i) mine += h[hi - 1 - 32 * i - lane];
#pragma unroll
    for (int o = 16; o; o >>= 1) mine += __shfl_xor_sync(0xFFFFFFFFu, mine, o);
    if (lane == 0) s_tot[warp] = mine;
    if (threadIdx.x == 0) { s_found_bin = 0xFFFFFFFFu; s_found_above = 0; }
    __syncthreads();
    uint32_t above = 0;  // keys in the segments of larger keys
    for (int w = 0; w < warp; ++w) above += s_tot[w];
    if (st.k_rem > 0 && above < st.k_rem && st.k_rem <= above + mine) {
        // the k-th key lies in this warp's segment: walk its rows with a warp scan (the condition is warp-uniform)
        for (int i = 0; i < rows; ++i) {
            const int b = hi - 1 - 32 * i - lane;
            const uint32_t c = h[b];
            uint32_t incl = c;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += v;
            }
            const uint32_t before = above + incl - c;  // keys larger than bin b
            const uint32_t hit = __ballot_sync(0xFFFFFFFFu, before < st.k_rem && st.k_rem <= before + c);
            if (hit) {
                if (lane == __ffs((int)hit) - 1) { s_found_bin = (uint32_t)b; s_found_above = before; }
                break;
            }
            above += __shfl_sync(0xFFFFFFFFu, incl, 31);
        }
    }
    __syncthreads();
    for (int i = 0; i < rows; ++i) h[hi - 1 - 32 * i - lane] = 0;
    if (threadIdx.x == 0) {
        if (st.k_rem == 0 || s_found_bin == 0xFFFFFFFFu) {
            // nothing (left) to take: a threshold above every key
            st.prefix = 0xFFFFFFFFu;
            st.k_rem = 0;
            if (last) { st.tau = 0xFFFFFFFFu; st.need = 0; }
        } else {
            st.prefix = (st.prefix << bits) | s_found_bin;
            st.k_rem -= s_found_above;
            if (last) { st.tau = st.prefix << shift_final; st.need = st.k_rem; }
        }
        sel[ut] = st;
    }
}

// ----- C2b (float32 only): histogram of the next 8 key bits among entries that match the prefix ------
// The first refinement (prefix = the 15 bits of the split's histogram) also collects the low 16 bits of every matching
// key in the unit-tensor's index list, which nothing has written yet (`cap` entries); the histogram holds the bins in
// words [0, 256), the candidate count in word 256 and an overflow flag in word 257.  The second refinement then reads
// those candidates instead of the whole tensor; only if they did not fit does the full pass run again.
constexpr int kCandCount = 256, kCandOverflow = 257;
constexpr int kCandBlock = 2048;  // candidates a thread block of the first refinement gathers before its one reservation in the list
__global__ void __launch_bounds__(256) refine_hist_kernel(const float* z1, int64_t unit_stride, int64_t n,
                                                          int ut_begin, const SelState* sel, uint32_t* hist,
                                                          int shift_prefix, int shift_digit, int32_t* cand_all, int64_t cap,
                                                          int only_on_overflow) {
    __shared__ uint32_t s_h[256];
    __shared__ uint16_t s_c[kCandBlock];
    __shared__ uint32_t s_n, s_base;
    const int ut = ut_begin + blockIdx.y;
    uint32_t* const h = hist + (int64_t)ut * kHistBins;
    if (only_on_overflow && !h[kCandOverflow]) return;  // (block-uniform: the candidates served this pass)
    s_h[threadIdx.x] = 0;
    if (threadIdx.x == 0) s_n = 0;
    __syncthreads();
    const uint32_t prefix = sel[ut].prefix;
    if (prefix != 0xFFFFFFFFu) {
        const float* z = z1 + (int64_t)ut * unit_stride;
        for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
            const uint32_t key = key_of(z[i]);
            if ((key >> shift_prefix) == prefix) {
                atomicAdd(&s_h[(key >> shift_digit) & 0xFFu], 1u);
                if (cand_all) {
                    const uint32_t pos = atomicAdd(&s_n, 1u);
                    if (pos < (uint32_t)kCandBlock) s_c[pos] = (uint16_t)(key & 0xFFFFu);
                }
            }
        }
    }
    __syncthreads();
    if (s_h[threadIdx.x]) atomicAdd(&h[threadIdx.x], s_h[threadIdx.x]);
    if (cand_all) {
        const uint32_t mine = s_n;
        if (threadIdx.x == 0) {
            s_base = atomicAdd(&h[kCandCount], mine);
            if (mine > (uint32_t)kCandBlock) h[kCandOverflow] = 1u;  // more than the block could hold: the full pass runs again
        }
        __syncthreads();
        const uint32_t base = s_base;
        for (uint32_t i = threadIdx.x; i < min(mine, (uint32_t)kCandBlock); i += blockDim.x)
            if ((int64_t)(base + i) < cap) cand_all[(int64_t)ut * cap + base + i] = (int32_t)s_c[i];
    }
}
// second refinement from the collected candidates: one thread block per unit-tensor
__global__ void __launch_bounds__(256) refine_candidates_kernel(int ut_begin, const SelState* sel, uint32_t* hist, const int32_t* cand_all,
                                                                int64_t cap) {
    __shared__ uint32_t s_h[256];
    const int ut = ut_begin + blockIdx.x;
    uint32_t* const h = hist + (int64_t)ut * kHistBins;
    const uint32_t count = h[kCandCount];
    if ((int64_t)count > cap || h[kCandOverflow]) {  // they did not fit: the full pass that follows does the work
        if (threadIdx.x == 0) h[kCandOverflow] = 1u;
        return;
    }
    s_h[threadIdx.x] = 0;
    __syncthreads();
    const uint32_t prefix = sel[ut].prefix;  // 23 bits by now: the candidates share its upper 15
    if (prefix != 0xFFFFFFFFu)
        for (uint32_t i = threadIdx.x; i < count; i += blockDim.x) {
            const uint32_t c = (uint32_t)cand_all[(int64_t)ut * cap + i];
            if ((c >> 8) == (prefix & 0xFFu)) atomicAdd(&s_h[c & 0xFFu], 1u);
        }
    __syncthreads();
    if (s_h[threadIdx.x]) h[threadIdx.x] = s_h[threadIdx.x];
}

// (C3-C5, the index-ordered compaction, live in select_fused.cu.)

template <typename T>
__global__ void strided_copy_kernel(const T* src, int64_t stride_t, T* dst, int T_, int d) {
    using S = Store<T>;
    constexpr int VEC = S::VEC;
    const int vpr = d / VEC;
    const int64_t n = (int64_t)T_ * vpr;
    for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < n; v += (int64_t)gridDim.x * blockDim.x) {
        const int64_t t = v / vpr;
        const int cv = (int)(v % vpr) * VEC;
        *reinterpret_cast<typename S::vec_t*>(dst + t * d + cv) =
            *reinterpret_cast<const typename S::vec_t*>(src + t * stride_t + cv);
    }
}

}  // namespace

cudaError_t launch_split_hist(const CompressArgs& a, int dtype, cudaStream_t st) {
    static PerDevice once;
    const size_t smem = (size_t)kHistBins * sizeof(uint32_t);
    cudaError_t e0 = once.ensure([&]() {
        cudaError_t e = cudaFuncSetAttribute(split_hist_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        return cudaFuncSetAttribute(split_hist_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    });
    if (e0 != cudaSuccess) return e0;
    if (a.T <= 0 || a.n_pairs <= 0) return cudaSuccess;
    const int tokens_per_cta = 4096 * 128 / a.d / (dtype == FDKV_BF16 ? 1 : 2);
    dim3 grid((a.T + tokens_per_cta - 1) / tokens_per_cta, a.Hkv * a.tensors, a.n_pairs);
    if (dtype == FDKV_BF16)
        split_hist_kernel<__nv_bfloat16><<<grid, 1024, smem, st>>>(a, tokens_per_cta);
    else
        split_hist_kernel<float><<<grid, 1024, smem, st>>>(a, tokens_per_cta);
    count_launch(1);
    return cudaGetLastError();
}

cudaError_t launch_select_and_compact(const SelectArgs& a, int dtype, cudaStream_t st) {
    if (a.ut_count <= 0) return cudaSuccess;
    const uint32_t k = (uint32_t)a.k;
    const int64_t n = (int64_t)a.T * a.d;
    if (dtype == FDKV_BF16) {
        threshold_kernel<<<a.ut_count, 1024, 0, st>>>(a.hist, a.sel, a.ut_begin, kHistBins, 15, 1, 1, 16, k);
        count_launch(1);
    } else {
        threshold_kernel<<<a.ut_count, 1024, 0, st>>>(a.hist, a.sel, a.ut_begin, kHistBins, 15, 1, 0, 0, k);
        const int chunks = (int)std::min<int64_t>(64, (n + 256 * 16 - 1) / (256 * 16));
        refine_hist_kernel<<<dim3(chunks, a.ut_count), 256, 0, st>>>(reinterpret_cast<const float*>(a.z1), a.unit_stride,
                                                                     n, a.ut_begin, a.sel, a.hist, 16, 8, a.idx, a.kcap, 0);
        threshold_kernel<<<a.ut_count, 256, 0, st>>>(a.hist, a.sel, a.ut_begin, 256, 8, 0, 0, 0, k);
        refine_candidates_kernel<<<a.ut_count, 256, 0, st>>>(a.ut_begin, a.sel, a.hist, a.idx, a.kcap);
        refine_hist_kernel<<<dim3(chunks, a.ut_count), 256, 0, st>>>(reinterpret_cast<const float*>(a.z1), a.unit_stride,
                                                                     n, a.ut_begin, a.sel, a.hist, 8, 0, nullptr, 0, 1);
        threshold_kernel<<<a.ut_count, 256, 0, st>>>(a.hist, a.sel, a.ut_begin, 256, 8, 0, 1, 0, k);
        count_launch(6);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (a.T <= 0) return cudaSuccess;
    return launch_select_fused(a, dtype, st);
}

// grid (chunks of 32 KiB, jobs): the device-to-device copies of a commit (row streams, strided source rows of exact
// units, residual lists, offset tables) as one launch instead of several hundred copy calls
constexpr int kCopyChunk = 32 * 1024;
__global__ void __launch_bounds__(256) copy_jobs_kernel(const CopyJob* jobs) {
    const CopyJob jb = jobs[blockIdx.y];
    const int64_t c0 = (int64_t)blockIdx.x * kCopyChunk;
    if (c0 >= jb.bytes) return;
    const int64_t c1 = min(jb.bytes, c0 + kCopyChunk);
    const bool plain = jb.src_pitch == jb.row_bytes;
    auto src_of = [&](int64_t o) {
        if (plain) return o;
        const int64_t r = o / jb.row_bytes;
        return r * jb.src_pitch + (o - r * jb.row_bytes);
    };
    // 16-byte vectors when both sides allow it (offset tables of later unit-tensors start on 4-byte boundaries only)
    const bool vec_ok = (((uintptr_t)jb.src | (uintptr_t)jb.dst) & 15) == 0;
    const int64_t v1 = vec_ok ? (c1 & ~(int64_t)15) : c0;
#pragma unroll 4
    for (int64_t o = c0 + threadIdx.x * 16; o < v1; o += 256 * 16)
        *reinterpret_cast<uint4*>(jb.dst + o) = *reinterpret_cast<const uint4*>(jb.src + src_of(o));
    for (int64_t o = v1 + threadIdx.x * 4; o < c1; o += 256 * 4)
        *reinterpret_cast<uint32_t*>(jb.dst + o) = *reinterpret_cast<const uint32_t*>(jb.src + src_of(o));
}
cudaError_t launch_copy_jobs(const CopyJob* jobs_dev, int njobs, int64_t bytes_max, cudaStream_t st) {
    if (njobs <= 0 || bytes_max <= 0) return cudaSuccess;
    copy_jobs_kernel<<<dim3((unsigned)((bytes_max + kCopyChunk - 1) / kCopyChunk), njobs), 256, 0, st>>>(jobs_dev);
    count_launch(1);
    return cudaGetLastError();
}

__global__ void offset_copy_kernel(int32_t* dst, const int32_t* src, int n, int add) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) dst[i] = src[i] + add;
}
cudaError_t launch_offset_copy(int32_t* dst, const int32_t* src, int n, int add, cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    offset_copy_kernel<<<(n + 255) / 256, 256, 0, st>>>(dst, src, n, add);
    count_launch(1);
    return cudaGetLastError();
}

cudaError_t launch_strided_copy(const void* src, int64_t stride_t, void* dst, int T, int d, int esize, cudaStream_t st) {
    if (T <= 0) return cudaSuccess;
    const int vec = esize == 2 ? 8 : 4;
    const int64_t n = (int64_t)T * (d / vec);
    const int blocks = (int)std::min<int64_t>(148 * 8, (n + 255) / 256);
    if (esize == 2)
        strided_copy_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(reinterpret_cast<const __nv_bfloat16*>(src), stride_t,
                                                                  reinterpret_cast<__nv_bfloat16*>(dst), T, d);
    else
        strided_copy_kernel<float><<<blocks, 256, 0, st>>>(reinterpret_cast<const float*>(src), stride_t,
                                                           reinterpret_cast<float*>(dst), T, d);
    count_launch(1);
    return cudaGetLastError();
}

}  // namespace fdkv

// ---------------------------------------------------------------------------------------------------------------
// Allocation-free compression of one [T][d] tensor pair (declared in fdkv.h as fdkv_compress_unit_noalloc).
// Same kernels as fdkv_compress_prefill; the scratch they need (the Z1 temporary, the magnitude histogram, the
// select state, the look-back records and the tile offsets) lives in the file-scope device array below instead of a
// caller-provided workspace.  Every GPU that loads this library holds the array until the process exits.
// ---------------------------------------------------------------------------------------------------------------
namespace fdkv {
namespace {

constexpr int64_t kNoAllocMaxElems = FDKV_NOALLOC_MAX_ELEMS;                    // T * head_dim
constexpr int64_t kNoAllocMaxTiles = kNoAllocMaxElems / 64 / fdkv::kResTile;    // head_dim >= 64
constexpr size_t kNaZ1 = 0;                                                     // Z1 temporary, float32 worst case
constexpr size_t kNaHist = kNaZ1 + (size_t)kNoAllocMaxElems * 4;
constexpr size_t kNaSel = kNaHist + (size_t)fdkv::kHistBins * 4;
constexpr size_t kNaStatus = kNaSel + 256;
constexpr size_t kNaRecords = kNaStatus + 256;
constexpr size_t kNaTicket = kNaRecords + (size_t)kNoAllocMaxTiles * 8;
constexpr size_t kNaOff = kNaTicket + 256;
constexpr size_t kNaBytes = (kNaOff + (size_t)(kNoAllocMaxTiles + 1) * 4 + 255) / 256 * 256;

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNaBytes];

// In host code the array's name is only a handle: the device address comes from cudaGetSymbolAddress, once per
// device, with that device current.
constexpr int kMaxDevices = 64;
void* g_noalloc_ptr[kMaxDevices] = {};
std::mutex g_noalloc_mutex;

cudaError_t noalloc_scratch(char** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess) return e;
        g_noalloc_ptr[dev] = p;
    }
    *out = static_cast<char*>(g_noalloc_ptr[dev]);
    return cudaSuccess;
}

}  // namespace
}  // namespace fdkv

extern "C" fdkv_status fdkv_compress_unit_noalloc(const void* x0, const void* x1, int64_t stride_t, int32_t T,
                                                  int32_t head_dim, int32_t dtype, int32_t keep_num, int32_t keep_den,
                                                  void* z0_out, int32_t* idx_out, void* val_out, int32_t* count_host,
                                                  void* stream) {
    using namespace fdkv;
    if (!x0 || !x1 || !z0_out || T < 1) return FDKV_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128) return FDKV_ERR_UNSUPPORTED;
    if (dtype != FDKV_F32 && dtype != FDKV_BF16) return FDKV_ERR_UNSUPPORTED;
    if (keep_den <= 0 || keep_num < 0 || keep_num > keep_den) return FDKV_ERR_INVALID_ARG;
    if (stride_t < head_dim || (stride_t % 8)) return FDKV_ERR_INVALID_ARG;
    if ((int64_t)T * head_dim > kNoAllocMaxElems) return FDKV_ERR_TOO_LARGE;  // the static scratch cannot hold it
    const int64_t k = (int64_t)T * head_dim * keep_num / keep_den;
    if (k > 0 && (!idx_out || !val_out)) return FDKV_ERR_INVALID_ARG;
    for (const void* p : {x0, x1, (const void*)z0_out, (const void*)idx_out, (const void*)val_out})
        if (reinterpret_cast<uintptr_t>(p) % 16) return FDKV_ERR_INVALID_ARG;
    if (count_host) *count_host = (int32_t)k;

    char* sc = nullptr;
    cudaError_t e = noalloc_scratch(&sc);
    if (e != cudaSuccess) return record_cuda_error(e);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    // the array keeps the previous call's contents: the histogram and the status word must start at zero
    e = cudaMemsetAsync(sc + kNaHist, 0, (size_t)kHistBins * 4 + 512, st);
    if (e != cudaSuccess) return record_cuda_error(e);

    CompressArgs a;
    a.k0[0] = x0; a.k1[0] = x1; a.v0[0] = x0; a.v1[0] = x1;
    a.n_pairs = 1;
    a.stride_t = stride_t; a.stride_h = 0;
    a.T = T; a.d = head_dim; a.Hkv = 1; a.tensors = 1;
    a.ut_base = 0; a.unit_stride = 0;
    a.z0 = z0_out; a.z1 = sc + kNaZ1;
    a.hist = reinterpret_cast<uint32_t*>(sc + kNaHist);
    if ((e = launch_split_hist(a, dtype, st)) != cudaSuccess) return record_cuda_error(e);

    SelectArgs sa;
    sa.ut_begin = 0; sa.ut_count = 1;
    sa.T = T; sa.d = head_dim; sa.k = k;
    sa.unit_stride = 0; sa.kcap = 0; sa.ntiles_max = (int)kNoAllocMaxTiles;
    sa.z1 = sc + kNaZ1;
    sa.hist = reinterpret_cast<uint32_t*>(sc + kNaHist);
    sa.sel = reinterpret_cast<SelState*>(sc + kNaSel);
    sa.lb_records = reinterpret_cast<unsigned long long*>(sc + kNaRecords);
    sa.lb_ticket = reinterpret_cast<uint32_t*>(sc + kNaTicket);
    sa.tile_off = reinterpret_cast<int32_t*>(sc + kNaOff);
    sa.idx = idx_out; sa.val = val_out; sa.packed = nullptr; sa.z1drop = nullptr;
    sa.status = reinterpret_cast<int32_t*>(sc + kNaStatus);
    if ((e = launch_select_and_compact(sa, dtype, st)) != cudaSuccess) return record_cuda_error(e);
    return FDKV_OK;
}
