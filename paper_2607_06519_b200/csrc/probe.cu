// Routing probe (Eq. 2 and the argmin of Eq. 3): logit-error of the shared and residual candidates over the
// probe window, then the mode rule.  This file holds the portable float32-FMA kernel (any dtype / head_dim);
// the tcgen05 tensor-core kernel for bf16 lives in probe_tc.cu.
#include "fdkv_internal.h"

namespace fdkv {

namespace {

template <typename T>
__device__ __forceinline__ float ldf(const T* p);
template <>
__device__ __forceinline__ float ldf<float>(const float* p) { return *p; }
template <>
__device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }

constexpr int kRowsBlk = 16;

// grid (probe tiles, units).  Each CTA: 64 tokens of one unit, all 2*G*W probe rows, both candidates.
template <typename T>
__global__ void __launch_bounds__(256) probe_tile_kernel(ProbeArgs a) {
    extern __shared__ float smem[];
    const int d = a.d, ld = d + 1;
    float* full = smem;                      // [64][d+1]  Z1 of K: what the shared candidate drops
    float* drop = full + kProbeTile * ld;    // [64][d+1]  Z1 of K minus the kept entries: what residual drops
    float* qs = drop + kProbeTile * ld;      // [16][d]
    __shared__ double s_red[2][8];

    const int unit = a.unit_begin + blockIdx.y;
    const int t0 = blockIdx.x * kProbeTile;
    const int nt = min(kProbeTile, a.T - t0);
    const int h = unit % a.Hkv, pair = unit / a.Hkv;
    const int ut = unit * 2;  // K
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int j = (warp & 1) * 32 + lane;  // token within the tile
    const int rg = warp >> 1;              // 4 row groups
    // A pair has one high-frequency operand (Z1) that both layers' queries see; a block of four layers has one
    // operand per layer (its deviation from the block mean), seen by that layer's queries only.
    const int n_ops = a.B == 4 ? 4 : 1;
    const int M = (a.B == 4 ? 1 : 2) * a.G * a.W;  // probe rows per operand
    float sum_f = 0.f, sum_d = 0.f;
    for (int op = 0; op < n_ops; ++op) {
        const T* z1 = reinterpret_cast<const T*>(a.z1) + ((int64_t)ut * n_ops + op) * a.unit_stride + (int64_t)t0 * d;
        for (int i = threadIdx.x; i < kProbeTile * d; i += blockDim.x) {
            const int t = i / d, c = i % d;
            const float v = t < nt ? ldf<T>(z1 + i) : 0.f;
            full[t * ld + c] = v;
            drop[t * ld + c] = v;
        }
        __syncthreads();
        if (a.tok_flag) {
            // token rule: the residual candidate keeps whole rows -- the selected tokens drop nothing
            const uint8_t* flag = a.tok_flag + (int64_t)unit * a.Tmax + t0;
            for (int i = threadIdx.x; i < nt * d; i += blockDim.x)
                if (flag[i / d]) drop[(i / d) * ld + (i % d)] = 0.f;
        } else {
            const int32_t* off = a.tile_off + (int64_t)ut * (a.ntiles_max + 1);
            const int ntiles = (a.T + kResTile - 1) / kResTile;
            const int j0 = t0 / kResTile, j1 = min(ntiles, (t0 + kProbeTile) / kResTile);
            const int32_t* idx = a.idx + (int64_t)ut * a.kcap;
            for (int e = off[j0] + threadIdx.x; e < off[j1]; e += blockDim.x) {
                const int f = idx[e] - t0 * d;
                drop[(f / d) * ld + (f % d)] = 0.f;
            }
        }
        __syncthreads();
        for (int rb = 0; rb < M; rb += kRowsBlk) {
            // stage 16 probe rows: row r = (layer*G + g)*W + qi  ->  Q[layer][qi][h*G + g][:]
            for (int i = threadIdx.x; i < kRowsBlk * d; i += blockDim.x) {
                const int r = rb + i / d, c = i % d;
                float v = 0.f;
                if (r < M) {
                    const int layer = a.B == 4 ? op : r / (a.G * a.W), g = (r / a.W) % a.G, qi = r % a.W;
                    const T* q = reinterpret_cast<const T*>(a.q_layers_dev[a.B * pair + layer]);
                    v = ldf<T>(q + ((int64_t)qi * a.Hq + h * a.G + g) * d + c);
                }
                qs[i] = v;
            }
            __syncthreads();
            float af[4] = {0.f, 0.f, 0.f, 0.f}, ad[4] = {0.f, 0.f, 0.f, 0.f};
            const float* zf = full + j * ld;
            const float* zd = drop + j * ld;
            const float* qr = qs + rg * 4 * d;
            for (int c = 0; c < d; ++c) {
                const float vf = zf[c], vd = zd[c];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float qv = qr[i * d + c];
                    af[i] = fmaf(qv, vf, af[i]);
                    ad[i] = fmaf(qv, vd, ad[i]);
                }
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int r = rb + rg * 4 + i;
                if (r < M && j < nt && t0 + j <= a.pos[r % a.W]) {  // causal: keys at or before the probe position
                    sum_f = fmaf(af[i], af[i], sum_f);
                    sum_d = fmaf(ad[i], ad[i], sum_d);
                }
            }
            __syncthreads();
        }
    }
    double df = sum_f, dd = sum_d;
#pragma unroll
    for (int o = 16; o; o >>= 1) {
        df += __shfl_xor_sync(0xFFFFFFFFu, df, o);
        dd += __shfl_xor_sync(0xFFFFFFFFu, dd, o);
    }
    if (lane == 0) { s_red[0][warp] = df; s_red[1][warp] = dd; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double tf = 0, td = 0;
        for (int w = 0; w < 8; ++w) { tf += s_red[0][w]; td += s_red[1][w]; }
        double* p = a.part + ((int64_t)unit * a.nptiles_max + blockIdx.x) * 2;
        p[0] = tf;
        p[1] = td;
    }
}

}  // namespace

// Sums the per-tile partials in a fixed order, applies the (c/sqrt d)^2 / (2 G W) factor and the mode rule.
__global__ void __launch_bounds__(256) probe_finalize_kernel(ProbeArgs a, int nparts) {
    __shared__ double s0[256], s1[256];
    const int unit = a.unit_begin + blockIdx.x;
    const double* p = a.part + (int64_t)unit * a.nptiles_max * 2;
    double x0 = 0, x1 = 0;
    for (int i = threadIdx.x; i < nparts; i += blockDim.x) { x0 += p[2 * i]; x1 += p[2 * i + 1]; }
    s0[threadIdx.x] = x0;
    s1[threadIdx.x] = x1;
    __syncthreads();
    for (int o = 128; o; o >>= 1) {
        if (threadIdx.x < o) { s0[threadIdx.x] += s0[threadIdx.x + o]; s1[threadIdx.x] += s1[threadIdx.x + o]; }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        // (c / sqrt d)^2 over 2 G W rows for a pair's Z1; (1 / sqrt d)^2 over 4 G W rows for a block's deviations
        const double norm = a.B == 4 ? 1.0 / (double)a.d / (double)(4 * a.G * a.W) : 0.5 / (double)a.d / (double)(2 * a.G * a.W);
        const double e_sh = s0[0] * norm, e_rs = s1[0] * norm;
        a.scores[2 * unit] = e_sh;
        a.scores[2 * unit + 1] = e_rs;
        const double L0 = e_sh + a.lambda * a.omega[0];
        const double L1 = e_rs + a.lambda * a.omega[1];
        const double L2 = a.lambda * a.omega[2];
        int m = 0;
        double best = L0;
        if (L1 < best) { best = L1; m = 1; }
        if (L2 < best) { best = L2; m = 2; }
        a.modes[unit] = m;
        if (a.modes_out) a.modes_out[blockIdx.x] = m;
        if (a.scores_out) {
            a.scores_out[2 * blockIdx.x] = (float)e_sh;
            a.scores_out[2 * blockIdx.x + 1] = (float)e_rs;
        }
    }
}

cudaError_t launch_probe_tc(const ProbeArgs& a, int dtype, cudaStream_t st, bool* handled, int* nparts);

cudaError_t launch_probe(const ProbeArgs& a, int dtype, cudaStream_t st) {
    if (a.unit_count <= 0) return cudaSuccess;
    int nparts = (a.T + kProbeTile - 1) / kProbeTile;
    bool handled = false;
    cudaError_t e = launch_probe_tc(a, dtype, st, &handled, &nparts);
    if (e != cudaSuccess) return e;
    if (!handled) {
        const size_t smem = (size_t)(2 * kProbeTile * (a.d + 1) + kRowsBlk * a.d) * sizeof(float);
        static PerDevice once;
        e = once.ensure([&]() {
            cudaError_t e2 = cudaFuncSetAttribute(probe_tile_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
            if (e2 != cudaSuccess) return e2;
            return cudaFuncSetAttribute(probe_tile_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
        });
        if (e != cudaSuccess) return e;
        dim3 grid(nparts, a.unit_count);
        if (dtype == FDKV_BF16)
            probe_tile_kernel<__nv_bfloat16><<<grid, 256, smem, st>>>(a);
        else
            probe_tile_kernel<float><<<grid, 256, smem, st>>>(a);
        count_launch(1);
        count_kernel(FDKV_KERNEL_PROBE_PORTABLE);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    probe_finalize_kernel<<<a.unit_count, 256, 0, st>>>(a, nparts);
    count_launch(1);
    return cudaGetLastError();
}

}  // namespace fdkv
