// Decode attention over the compressed cache (the fused reconstruct-and-attend step after Eq. 3):
// tail append, split-K partial attention with per-mode reconstruction, split-K combine.
// This file holds the portable kernel (float32 or bf16 storage, head_dim 64/128, any group size up to 8);
// the bulk-copy / tensor-core kernel for bf16, head_dim 128 lives in decode_fast.cu.
#include "fdkv_internal.h"

namespace fdkv {

namespace {

template <typename T, int EPL>
__device__ __forceinline__ void load_row(const T* row, int lane, float* f);
template <>
__device__ __forceinline__ void load_row<float, 4>(const float* row, int lane, float* f) {
    const float4 v = *reinterpret_cast<const float4*>(row + lane * 4);
    f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
}
template <>
__device__ __forceinline__ void load_row<float, 2>(const float* row, int lane, float* f) {
    const float2 v = *reinterpret_cast<const float2*>(row + lane * 2);
    f[0] = v.x; f[1] = v.y;
}
template <>
__device__ __forceinline__ void load_row<__nv_bfloat16, 4>(const __nv_bfloat16* row, int lane, float* f) {
    const uint2 v = *reinterpret_cast<const uint2*>(row + lane * 4);
    f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xFFFF0000u);
    f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xFFFF0000u);
}
template <>
__device__ __forceinline__ void load_row<__nv_bfloat16, 2>(const __nv_bfloat16* row, int lane, float* f) {
    const uint32_t v = *reinterpret_cast<const uint32_t*>(row + lane * 2);
    f[0] = __uint_as_float(v << 16); f[1] = __uint_as_float(v & 0xFFFF0000u);
}
template <typename T>
__device__ __forceinline__ float ldf(const T* p);
template <>
__device__ __forceinline__ float ldf<float>(const float* p) { return *p; }
template <>
__device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }

// Appends k_new / v_new rows of every sequence to the layer's tail and bumps the tail length.
template <typename T>
__global__ void append_tail_kernel(DecodeArgs a) {
    // Programmatic dependent launch: the kernel may become resident, and let the decode kernel behind it start its
    // own prologue, while the kernel ahead of it in the stream still runs.  Everything it reads was possibly written by
    // that kernel -- k_new / v_new come from the caller's projection, the tail length from the previous step's append,
    // and the previous step's decode kernel of this layer may still be reading the length -- so the dependency wait
    // comes before the first read.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int b = blockIdx.x;
    int32_t* len = a.tail_len + a.layer * a.max_batch + b;
    const int n = *len;
    if (n >= a.max_tail) {
        if (threadIdx.x == 0) atomicMax(a.status, (int32_t)kFlagTailFull);
        return;
    }
    const int row = a.Hkv * a.d;
    const T* kn = reinterpret_cast<const T*>(a.k_new) + (int64_t)b * row;
    const T* vn = reinterpret_cast<const T*>(a.v_new) + (int64_t)b * row;
    T* tk = reinterpret_cast<T*>(a.tail_k);
    T* tv = reinterpret_cast<T*>(a.tail_v);
    for (int i = threadIdx.x; i < row; i += blockDim.x) {
        const int h = i / a.d, c = i % a.d;
        const int64_t o = ((((int64_t)a.layer * a.max_batch + b) * a.Hkv + h) * a.tail_rows + n) * a.d + c;
        tk[o] = kn[i];
        tv[o] = vn[i];
    }
    __syncthreads();
    if (threadIdx.x == 0) *len = n + 1;
}

constexpr int kWarps = 4;
constexpr int kGTile = 32;                  // tokens per warp tile of the portable kernel
constexpr int kSub = kGTile / kResTile;     // residual-offset tiles per warp tile

// grid (splits, Hkv, batch); 4 warps; each warp owns whole 32-token tiles and a private online-softmax state.
template <typename T, int D, int G>
__global__ void __launch_bounds__(kWarps * 32) decode_generic_kernel(DecodeArgs a, int splits) {
    constexpr int EPL = D / 32;
    __shared__ float qs[G][D];
    __shared__ float s_corr[kWarps][G][32];
    __shared__ float s_p[kWarps][G][32];
    __shared__ float s_vacc[kWarps][G][D];
    __shared__ float s_m[kWarps][G], s_l[kWarps][G];

    const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const UnitDesc u = a.desc[((int64_t)b * a.L + a.layer) * a.Hkv + h];
    const T* qg = reinterpret_cast<const T*>(a.q) + ((int64_t)b * a.Hq + h * G) * D;
    for (int i = threadIdx.x; i < G * D; i += blockDim.x) qs[i / D][i % D] = ldf<T>(qg + i);
    for (int i = threadIdx.x; i < kWarps * G * D; i += blockDim.x) (&s_vacc[0][0][0])[i] = 0.f;
    __syncthreads();

    float q[G][EPL], acc[G][EPL], m[G], l[G];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        m[g] = -INFINITY;
        l[g] = 0.f;
#pragma unroll
        for (int i = 0; i < EPL; ++i) { q[g][i] = qs[g][lane * EPL + i]; acc[g][i] = 0.f; }
    }

    const float inv_sqrt_d = rsqrtf((float)D);
    const float c = u.scale;  // what the stored rows are multiplied by (1/sqrt 2 for a pair, 1/2 for a block of four)
    const bool coef = u.mode != FDKV_MODE_EXACT;
    const bool resid = u.mode == FDKV_MODE_RESIDUAL;

    const int nres = (u.T + kResTile - 1) / kResTile;
    // ---- one 32-token tile: rows [row0, row0 + nrows) of kbase / vbase ----
    auto tile = [&](const T* kbase, const T* vbase, int nrows, float kscale, float vscale, bool with_res, int jt) {
        float s[G];
#pragma unroll
        for (int g = 0; g < G; ++g) s[g] = 0.f;
        for (int tt = 0; tt < nrows; ++tt) {
            float kf[EPL];
            load_row<T, EPL>(kbase + (int64_t)tt * D, lane, kf);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                float p = 0.f;
#pragma unroll
                for (int i = 0; i < EPL; ++i) p = fmaf(q[g][i], kf[i], p);
#pragma unroll
                for (int o = 16; o; o >>= 1) p += __shfl_xor_sync(0xFFFFFFFFu, p, o);
                if (lane == tt) s[g] = p;
            }
        }
        if (with_res && u.res_kind == 1) {
            // token rule: the tile's selected tokens carry whole high-frequency rows (k_idx = ascending token list, k_off =
            // tokens kept before every 16-token slice, k_val / v_val = their rows, densely packed)
            const T* rows = reinterpret_cast<const T*>(u.k_val);
            const int j1 = u.k_off[min(nres, (jt + 1) * kSub)];
            for (int j = u.k_off[jt * kSub]; j < j1; ++j) {
                const int tt = u.k_idx[j] - jt * kGTile;
                float kf[EPL];
                load_row<T, EPL>(rows + (int64_t)j * D, lane, kf);
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    float p = 0.f;
#pragma unroll
                    for (int i = 0; i < EPL; ++i) p = fmaf(q[g][i], kf[i], p);
#pragma unroll
                    for (int o = 16; o; o >>= 1) p += __shfl_xor_sync(0xFFFFFFFFu, p, o);
                    if (lane == tt) s[g] = fmaf(u.sign, p, s[g]);
                }
            }
        } else if (with_res) {
            // sparse correction in the logit domain: q . z1 over this tile's kept K entries
#pragma unroll
            for (int g = 0; g < G; ++g) s_corr[warp][g][lane] = 0.f;
            __syncwarp();
            const int64_t base = (int64_t)jt * kGTile * D;
            const T* val = reinterpret_cast<const T*>(u.k_val);
            const int ke1 = u.k_off[min(nres, (jt + 1) * kSub)];
            for (int e = u.k_off[jt * kSub] + lane; e < ke1; e += 32) {
                const int f = (int)(u.k_idx[e] - base);
                const float v = ldf<T>(val + e);
#pragma unroll
                for (int g = 0; g < G; ++g) atomicAdd(&s_corr[warp][g][f / D], qs[g][f % D] * v);
            }
            __syncwarp();
#pragma unroll
            for (int g = 0; g < G; ++g) s[g] = fmaf(u.sign, s_corr[warp][g][lane], s[g]);
        }
        float p[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const float sg = lane < nrows ? s[g] * kscale : -INFINITY;
            float mx = sg;
#pragma unroll
            for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
            const float m_new = fmaxf(m[g], mx);
            const float alpha = __expf(m[g] - m_new);  // m_new is finite here (nrows >= 1)
            p[g] = lane < nrows ? __expf(sg - m_new) : 0.f;
            float ps = p[g];
#pragma unroll
            for (int o = 16; o; o >>= 1) ps += __shfl_xor_sync(0xFFFFFFFFu, ps, o);
            l[g] = l[g] * alpha + ps;
            m[g] = m_new;
#pragma unroll
            for (int i = 0; i < EPL; ++i) acc[g][i] *= alpha;
            p[g] *= vscale;
        }
        for (int tt = 0; tt < nrows; ++tt) {
            float vf[EPL];
            load_row<T, EPL>(vbase + (int64_t)tt * D, lane, vf);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const float pg = __shfl_sync(0xFFFFFFFFu, p[g], tt);
#pragma unroll
                for (int i = 0; i < EPL; ++i) acc[g][i] = fmaf(pg, vf[i], acc[g][i]);
            }
        }
        if (with_res && u.res_kind == 1) {
            const T* rows = reinterpret_cast<const T*>(u.v_val);
            const int j1 = u.k_off[min(nres, (jt + 1) * kSub)];
            for (int j = u.k_off[jt * kSub]; j < j1; ++j) {
                const int tt = u.k_idx[j] - jt * kGTile;
                float vf[EPL];
                load_row<T, EPL>(rows + (int64_t)j * D, lane, vf);
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const float pg = u.sign * __shfl_sync(0xFFFFFFFFu, p[g], tt);
#pragma unroll
                    for (int i = 0; i < EPL; ++i) acc[g][i] = fmaf(pg, vf[i], acc[g][i]);
                }
            }
        } else if (with_res) {
#pragma unroll
            for (int g = 0; g < G; ++g) s_p[warp][g][lane] = p[g];
            __syncwarp();
            const int64_t base = (int64_t)jt * kGTile * D;
            const T* val = reinterpret_cast<const T*>(u.v_val);
            const int e0 = u.v_off[jt * kSub], e1 = u.v_off[min(nres, (jt + 1) * kSub)];
            for (int e = e0 + lane; e < e1; e += 32) {
                const int f = (int)(u.v_idx[e] - base);
                const float v = ldf<T>(val + e);
#pragma unroll
                for (int g = 0; g < G; ++g) atomicAdd(&s_vacc[warp][g][f % D], s_p[warp][g][f / D] * v);
            }
            __syncwarp();
            if (e1 > e0) {
#pragma unroll
                for (int g = 0; g < G; ++g)
#pragma unroll
                    for (int i = 0; i < EPL; ++i) {
                        acc[g][i] = fmaf(u.sign, s_vacc[warp][g][lane * EPL + i], acc[g][i]);
                        s_vacc[warp][g][lane * EPL + i] = 0.f;
                    }
            }
            __syncwarp();
        }
    };

    // ---- prefill rows of this split ----
    {
        const int ntiles = (u.T + kGTile - 1) / kGTile;
        const int tiles_per_split = (ntiles + splits - 1) / splits;
        const int j0 = split * tiles_per_split, j1 = min(ntiles, j0 + tiles_per_split);
        const T* kr = reinterpret_cast<const T*>(u.k_rows);
        const T* vr = reinterpret_cast<const T*>(u.v_rows);
        const float kscale = coef ? c * inv_sqrt_d : inv_sqrt_d;
        const float vscale = coef ? c : 1.f;
        for (int jt = j0 + warp; jt < j1; jt += kWarps) {
            const int t0 = jt * kGTile;
            tile(kr + (int64_t)t0 * D, vr + (int64_t)t0 * D, min(kGTile, u.T - t0), kscale, vscale, resid, jt);
        }
    }
    // ---- uncompressed tail rows (last split only) ----
    if (split == splits - 1) {
        const int n = min(a.tail_len[a.layer * a.max_batch + b], a.max_tail);
        const int64_t o = (((int64_t)a.layer * a.max_batch + b) * a.Hkv + h) * a.tail_rows * D;
        const T* tk = reinterpret_cast<const T*>(a.tail_k) + o;
        const T* tv = reinterpret_cast<const T*>(a.tail_v) + o;
        for (int t0 = warp * 32; t0 < n; t0 += kWarps * 32)
            tile(tk + (int64_t)t0 * D, tv + (int64_t)t0 * D, min(32, n - t0), inv_sqrt_d, 1.f, false, 0);
    }

    // ---- merge the warps' states and write the split's partial ----
    if (lane == 0)
#pragma unroll
        for (int g = 0; g < G; ++g) { s_m[warp][g] = m[g]; s_l[warp][g] = l[g]; }
    __syncthreads();
#pragma unroll
    for (int g = 0; g < G; ++g) {
        float M = -INFINITY;
        for (int w = 0; w < kWarps; ++w) M = fmaxf(M, s_m[w][g]);
        const float f = M == -INFINITY ? 0.f : __expf(m[g] - M);
#pragma unroll
        for (int i = 0; i < EPL; ++i) s_vacc[warp][g][lane * EPL + i] = acc[g][i] * f;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < G * D; i += blockDim.x) {
        const int g = i / D, ch = i % D;
        float M = -INFINITY;
        for (int w = 0; w < kWarps; ++w) M = fmaxf(M, s_m[w][g]);
        float L = 0.f, A = 0.f;
        for (int w = 0; w < kWarps; ++w) {
            L += M == -INFINITY ? 0.f : s_l[w][g] * __expf(s_m[w][g] - M);
            A += s_vacc[w][g][ch];
        }
        float* part = a.partials + (((int64_t)b * a.Hq + h * G + g) * kMaxSplits + split) * (D + 4);
        if (ch == 0) { part[0] = M; part[1] = L; }
        part[4 + ch] = A;
    }
}

// out = sum_s e^{m_s - M} acc_s / sum_s e^{m_s - M} l_s.  grid (Hq, batch), D threads.
template <int D>
__global__ void combine_kernel(const float* partials, int Hq, int splits, void* out, int out_dtype) {
    const int i = blockIdx.x, b = blockIdx.y, ch = threadIdx.x;
    const float* p = partials + ((int64_t)b * Hq + i) * kMaxSplits * (D + 4);
    float M = -INFINITY;
    for (int s = 0; s < splits; ++s) M = fmaxf(M, p[s * (D + 4)]);
    float L = 0.f, A = 0.f;
    for (int s = 0; s < splits; ++s) {
        const float ms = p[s * (D + 4)];
        if (ms == -INFINITY) continue;
        const float f = __expf(ms - M);
        L = fmaf(p[s * (D + 4) + 1], f, L);
        A = fmaf(p[s * (D + 4) + 4 + ch], f, A);
    }
    const float r = L > 0.f ? A / L : 0.f;
    const int64_t o = ((int64_t)b * Hq + i) * D + ch;
    if (out_dtype == FDKV_BF16)
        reinterpret_cast<__nv_bfloat16*>(out)[o] = __float2bfloat16_rn(r);
    else
        reinterpret_cast<float*>(out)[o] = r;
}

template <typename T, int D>
cudaError_t launch_generic(const DecodeArgs& a, int splits, cudaStream_t st) {
    dim3 grid(splits, a.Hkv, a.batch);
    switch (a.G) {
        case 1: decode_generic_kernel<T, D, 1><<<grid, kWarps * 32, 0, st>>>(a, splits); break;
        case 2: decode_generic_kernel<T, D, 2><<<grid, kWarps * 32, 0, st>>>(a, splits); break;
        case 4: decode_generic_kernel<T, D, 4><<<grid, kWarps * 32, 0, st>>>(a, splits); break;
        case 8: decode_generic_kernel<T, D, 8><<<grid, kWarps * 32, 0, st>>>(a, splits); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

}  // namespace

__global__ void set_tail_len_kernel(int32_t* tail_len, int L, int max_batch, int seq, int n) {
    for (int l = threadIdx.x; l < L; l += blockDim.x) tail_len[l * max_batch + seq] = n;
}
cudaError_t launch_set_tail_len(int32_t* tail_len, int L, int max_batch, int seq, int n, cudaStream_t st) {
    set_tail_len_kernel<<<1, 128, 0, st>>>(tail_len, L, max_batch, seq, n);
    count_launch(1);
    return cudaGetLastError();
}

cudaError_t launch_decode_fast(const DecodeArgs& a, cudaStream_t st, bool* handled);

cudaError_t launch_decode(const DecodeArgs& a, int dtype, cudaStream_t st) {
    cudaError_t e;
    bool handled = false;
    if ((e = launch_decode_fast(a, st, &handled)) != cudaSuccess) return e;  // (appends k_new / v_new itself)
    if (handled) return cudaSuccess;
    if (a.k_new) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(a.batch);
        cfg.blockDim = dim3(128);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (dtype == FDKV_BF16)
            e = cudaLaunchKernelEx(&cfg, append_tail_kernel<__nv_bfloat16>, a);
        else
            e = cudaLaunchKernelEx(&cfg, append_tail_kernel<float>, a);
        if (e != cudaSuccess) return e;
        count_launch(1);
    }
    if (a.packed_lists) return cudaErrorNotSupported;  // packed residual lists are only read by the kernel above

    const int ntiles = (a.Tmax_batch + kGTile - 1) / kGTile;
    int splits = (2 * 148 + a.Hkv * a.batch - 1) / (a.Hkv * a.batch);
    splits = max(1, min(min(splits, kMaxSplits), (ntiles + 7) / 8));
    if (dtype == FDKV_BF16)
        e = a.d == 128 ? launch_generic<__nv_bfloat16, 128>(a, splits, st) : launch_generic<__nv_bfloat16, 64>(a, splits, st);
    else
        e = a.d == 128 ? launch_generic<float, 128>(a, splits, st) : launch_generic<float, 64>(a, splits, st);
    if (e != cudaSuccess) return e;
    dim3 cgrid(a.Hq, a.batch);
    if (a.d == 128)
        combine_kernel<128><<<cgrid, 128, 0, st>>>(a.partials, a.Hq, splits, a.out, a.out_dtype);
    else
        combine_kernel<64><<<cgrid, 64, 0, st>>>(a.partials, a.Hq, splits, a.out, a.out_dtype);
    count_launch(2);
    count_kernel(FDKV_KERNEL_DECODE_PORTABLE);
    return cudaGetLastError();
}

}  // namespace fdkv
