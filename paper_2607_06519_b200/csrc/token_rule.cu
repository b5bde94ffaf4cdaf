// Token-granular sparse residual (the paper's rule, Method between Eq. 2 and Eq. 3).  The tensor-core kernels below
// serve bf16 storage with head_dim 128; other storage types and head dimensions take token_score_tile_kernel, a plain
// float32 product, and the same selection.
//
//   s_t = max over (layer of the depth block, group query head, probe query q with pos[q] >= t) | Q_l . (K_l[t,:] - Khat_l^shared[t,:]) |
//       = | Q_l . (+-c Z1K[t,:]) | for a pair, | Q_l . dev_l[t,:] | for a block of four (dev_l = layer l's deviation from the block mean);
//   keep the k_tok tokens with the largest s_t (ties: lowest t); they keep all 128 high-frequency values of K and of V
//   (of every layer of a block of four).
//
// 1. token_score_kernel (tcgen05): the transposed probe product D[token][probe row] = Z1K . Q^T, so that a thread
//    of the epilogue owns one token (TMEM lane) and takes the maximum over its row's columns in registers.  A = 128
//    tokens of Z1K per tile (TMA ring, shared memory), B = the item's 256 Q rows (shared memory, resident),
//    M = 128, N = 256, K = 16, two accumulator sets of 256 TMEM columns.  Items of the two layers / row blocks of a
//    unit merge with atomicMax on the (non-negative) float bit patterns, which is order-independent.
// 2. token_select_kernel: per unit an MSB-first radix select (4 x 8 bits) of the k_tok-th largest score and an
//    index-ordered compaction: ascending token list, per-token flags, per-16-token-slice counts.
// 3. token_drop_kernel: Z1K with the selected rows zeroed (the residual candidate's B operand in the probe).
// 4. token_gather_kernel (commit): the selected rows of Z1, densely packed.
#include <cuda.h>

#include <algorithm>
#include <cstdlib>

#include "fdkv_internal.h"
#include "mbar_wait.cuh"

namespace fdkv {

namespace {

constexpr int kTM = 128;                    // tokens per tile (M of the MMA)
constexpr int kTN = 256;                    // probe rows per item (N of the MMA)
constexpr int kTStages = 4;
constexpr int kTAHalf = kTM * 128;          // one 64-channel half of a token tile: 16 KiB
constexpr int kTAStage = 2 * kTAHalf;       // 32 KiB
constexpr int kTBHalf = kTN * 128;          // one 64-channel half of the Q block: 32 KiB
constexpr int kTBBytes = 2 * kTBHalf;       // 64 KiB
constexpr int kTHdr = 2048;                 // barriers, TMEM slot, abort flag, probe position of every column
constexpr int kTSmem = kTHdr + kTBBytes + kTStages * kTAStage;  // 194 KiB
constexpr int kTThreads = 6 * 32;
constexpr int tFull = 0, tEmpty = 32, tTFull = 64, tTEmpty = 80, tSlot = 96, tAbort = 100, tPosCol = 1024;  // pos_col: 256 ints

__device__ __forceinline__ uint32_t s_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mb_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mb_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mb_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mb_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, int32_t* status) {
    mbar_wait_bounded(bar, parity, abort_flag, status);
}
__device__ __forceinline__ void tma_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
// shared-memory matrix descriptor: K-major operand, 128-byte swizzle, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// instruction descriptor: D = f32, A = B = bf16, both K-major, M = 128, N = 256
constexpr uint32_t kTIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTN >> 3) << 17) | ((uint32_t)(kTM >> 4) << 24);

template <int ACC>
__device__ __forceinline__ void umma_ss(uint32_t tmem_d, uint64_t da, uint64_t db) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
        "l"(da), "l"(db), "r"(kTIdesc), "n"(ACC)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
          "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
          "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
}

struct ScorePlan {
    int items_per_unit, mblocks, nsplits, ntiles, tiles_per_split, pos_min;
};

__global__ void __launch_bounds__(kTThreads, 1)
token_score_kernel(const __grid_constant__ CUtensorMap tmap, TokenArgs a, ScorePlan pl) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t sm0 = s_u32(smem);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + tAbort);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (sm0 & 1023u) {
        if (threadIdx.x == 0) atomicMax(a.status, (int32_t)kFlagCountMismatch);
        return;
    }
    int it = blockIdx.x;
    const int unit = a.unit_begin + it / pl.items_per_unit;
    it %= pl.items_per_unit;
    const int split = it % pl.nsplits; it /= pl.nsplits;
    const int mblock = it % pl.mblocks; it /= pl.mblocks;
    const int layer = it;
    const int h = unit % a.Hkv, pair = unit / a.Hkv;
    const int tile0 = split * pl.tiles_per_split;
    const int ntile = max(0, min(pl.ntiles, tile0 + pl.tiles_per_split) - tile0);
    const int rows_layer = a.G * a.W;
    int* const pos_col = reinterpret_cast<int*>(smem + tPosCol);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kTStages; ++s) { mb_init(sm0 + tFull + 8 * s, 1); mb_init(sm0 + tEmpty + 8 * s, 1); }
        for (int s = 0; s < 2; ++s) { mb_init(sm0 + tTFull + 8 * s, 1); mb_init(sm0 + tTEmpty + 8 * s, 4); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // ---- B: probe rows r = mblock*256 + i of this layer, r = g*W + qi -> Q[layer][qi][h*G+g][:]; padding rows zero ----
    {
        const __nv_bfloat16* q = reinterpret_cast<const __nv_bfloat16*>(a.q_layers_dev[a.B * pair + layer]);
        for (int v = threadIdx.x; v < kTN * 16; v += kTThreads) {
            const int i = v >> 4, chunk = v & 15;
            const int r = mblock * kTN + i;
            uint4 val = make_uint4(0u, 0u, 0u, 0u);
            if (r < rows_layer)
                val = *reinterpret_cast<const uint4*>(q + ((int64_t)(r % a.W) * a.Hq + h * a.G + r / a.W) * 128 + chunk * 8);
            *reinterpret_cast<uint4*>(smem + kTHdr + (chunk >> 3) * kTBHalf + i * 128 + (((chunk & 7) ^ (i & 7)) << 4)) = val;
        }
        for (int i = threadIdx.x; i < kTN; i += kTThreads) {
            const int r = mblock * kTN + i;
            pos_col[i] = r < rows_layer ? a.pos[r % a.W] : -1;
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sm0 + tSlot), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(smem + tSlot);
    const uint32_t b_base = sm0 + kTHdr, a_base = b_base + kTBBytes;

    if (warp == 0) {
        if (lane == 0) {
            // K high-frequency rows of the unit: unit-tensor 2*unit (a block of four stages one operand per layer)
            const int64_t row0 = a.B == 4 ? ((int64_t)unit * 2 * 4 + layer) * a.Tmax : (int64_t)unit * 2 * a.Tmax;
            for (int i = 0; i < ntile; ++i) {
                const int s = i % kTStages;
                mb_wait(sm0 + tEmpty + 8 * s, ((uint32_t)(i / kTStages) & 1u) ^ 1u, abort_flag, a.status);
                if (*abort_flag) break;
                const uint32_t full = sm0 + tFull + 8 * s, dst = a_base + s * kTAStage;
                const int y = (int)(row0 + (int64_t)(tile0 + i) * kTM);
                mb_expect_tx(full, kTAStage);
                tma_2d(dst, &tmap, 0, y, full);
                tma_2d(dst + kTAHalf, &tmap, 64, y, full);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint64_t db0 = smem_desc(b_base);
            for (int i = 0; i < ntile; ++i) {
                const int s = i % kTStages, as = i & 1;
                mb_wait(sm0 + tTEmpty + 8 * as, (((uint32_t)i >> 1) & 1u) ^ 1u, abort_flag, a.status);
                mb_wait(sm0 + tFull + 8 * s, (uint32_t)(i / kTStages) & 1u, abort_flag, a.status);
                if (*abort_flag) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint64_t da0 = smem_desc(a_base + s * kTAStage);
                const uint32_t d_tmem = tmem_base + (uint32_t)(as * kTN);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const uint64_t da = da0 + (uint64_t)(((k >> 2) * kTAHalf + (k & 3) * 32) >> 4);
                    const uint64_t db = db0 + (uint64_t)(((k >> 2) * kTBHalf + (k & 3) * 32) >> 4);
                    if (k == 0) umma_ss<0>(d_tmem, da, db);
                    else umma_ss<1>(d_tmem, da, db);
                }
                umma_commit(sm0 + tEmpty + 8 * s);
                umma_commit(sm0 + tTFull + 8 * as);
            }
        }
    } else {
        // ---- epilogue: thread = token (TMEM lane); maximum of |D| over the probe rows that can see the token ----
        const int lq = warp & 3;
        const float c32 = a.B == 4 ? 1.f : __uint_as_float(0x3F3504F3u);  // a pair's rows are Z1: K - Khat^shared = +-c Z1
        uint32_t* score = a.score + (int64_t)unit * a.Tmax;
        for (int i = 0; i < ntile; ++i) {
            const int as = i & 1;
            const int t = (tile0 + i) * kTM + lq * 32 + lane;
            mb_wait(sm0 + tTFull + 8 * as, ((uint32_t)i >> 1) & 1u, abort_flag, a.status);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            float m = 0.f;
            if (!*abort_flag) {
                const bool all_visible = (tile0 + i) * kTM + kTM - 1 <= pl.pos_min;
#pragma unroll
                for (int cp = 0; cp < 4; ++cp) {
                    uint32_t r0[32], r1[32];
                    const uint32_t ta = tmem_base + ((uint32_t)(lq * 32) << 16) + (uint32_t)(as * kTN + cp * 64);
                    tmem_ld32(ta, r0);
                    tmem_ld32(ta + 32, r1);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    if (all_visible) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) m = fmaxf(m, fmaxf(fabsf(__uint_as_float(r0[j])), fabsf(__uint_as_float(r1[j]))));
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            if (pos_col[cp * 64 + j] >= t) m = fmaxf(m, fabsf(__uint_as_float(r0[j])));
                            if (pos_col[cp * 64 + 32 + j] >= t) m = fmaxf(m, fabsf(__uint_as_float(r1[j])));
                        }
                    }
                }
            }
            if (t < a.T && m > 0.f && !*abort_flag) atomicMax(score + t, __float_as_uint(m * c32));
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mb_arrive(sm0 + tTEmpty + 8 * as);
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (*abort_flag)
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
}

// ---- block-wide helpers for the select kernel (1024 threads) ----
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t* s_warp, uint32_t* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t x = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += x;
    }
    __syncthreads();  // s_warp may still be read from the previous call
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        uint32_t w = s_warp[lane];
        uint32_t wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t x = __shfl_up_sync(0xFFFFFFFFu, wi, o);
            if (lane >= o) wi += x;
        }
        s_warp[lane] = wi - w;
        if (lane == 31) s_warp[32] = wi;
    }
    __syncthreads();
    *total = s_warp[32];
    return s_warp[warp] + incl - v;
}

// One CTA per unit: threshold of the k-th largest score (32-bit patterns of non-negative floats order like the
// floats), then the ascending list of kept tokens (score above the threshold, or equal and among the first `need`
// such tokens), their flags and the number of kept tokens before every 16-token slice.
__global__ void __launch_bounds__(1024) token_select_kernel(TokenArgs a) {
    __shared__ uint32_t s_hist[256];
    __shared__ uint32_t s_warp[33];
    __shared__ uint32_t s_prefix, s_krem;
    const int unit = a.unit_begin + blockIdx.x;
    const uint32_t* key = a.score + (int64_t)unit * a.Tmax;
    uint8_t* flag = a.flag + (int64_t)unit * a.Tmax;
    int32_t* list = a.list + (int64_t)unit * a.ktok_cap;
    int32_t* off = a.off + (int64_t)unit * (a.ntiles_max + 1);
    const int T = a.T;
    const int nslice = (T + kResTile - 1) / kResTile;
    uint32_t tau = 0xFFFFFFFFu, need = 0;
    if (a.k_tok > 0) {
        if (threadIdx.x == 0) { s_prefix = 0; s_krem = (uint32_t)a.k_tok; }
        for (int pass = 0; pass < 4; ++pass) {
            const int shift = 24 - 8 * pass;
            if (threadIdx.x < 256) s_hist[threadIdx.x] = 0;
            __syncthreads();
            const uint32_t prefix = s_prefix;
            for (int t = threadIdx.x; t < T; t += blockDim.x) {
                const uint32_t k = key[t];
                if (pass == 0 || (k >> (shift + 8)) == prefix) atomicAdd(&s_hist[(k >> shift) & 0xFFu], 1u);
            }
            __syncthreads();
            if (threadIdx.x == 0) {
                uint32_t above = 0, krem = s_krem;
                int b = 255;
                for (; b > 0; --b) {
                    if (above + s_hist[b] >= krem) break;
                    above += s_hist[b];
                }
                s_prefix = (prefix << 8) | (uint32_t)b;
                s_krem = krem - above;
            }
            __syncthreads();
        }
        tau = s_prefix;
        need = s_krem;
    }
    // ordered compaction, 1024 tokens per round
    uint32_t base_keep = 0, base_eq = 0;
    for (int t0 = 0; t0 < T; t0 += 1024) {
        const int t = t0 + threadIdx.x;
        const uint32_t k = t < T ? key[t] : 0u;
        const uint32_t gt = t < T && a.k_tok > 0 && k > tau, eq = t < T && a.k_tok > 0 && k == tau;
        uint32_t tot_eq, tot_keep;
        const uint32_t rank_eq = base_eq + block_excl_scan(eq, s_warp, &tot_eq);
        const uint32_t keep = gt || (eq && rank_eq < need);
        const uint32_t posk = base_keep + block_excl_scan(keep, s_warp, &tot_keep);
        if (t < T) {
            flag[t] = (uint8_t)keep;
            if (keep) list[posk] = t;
            if ((t & (kResTile - 1)) == 0) off[t / kResTile] = (int32_t)posk;
        }
        base_eq += tot_eq;
        base_keep += tot_keep;
    }
    if (threadIdx.x == 0) {
        off[nslice] = (int32_t)base_keep;
        if ((int64_t)base_keep != a.k_tok) atomicMax(a.status, (int32_t)kFlagCountMismatch);
    }
}

// Z1K with the selected rows zeroed.  grid (row blocks, units), 256 threads, one 16-byte vector per thread and step.
__global__ void __launch_bounds__(256) token_drop_kernel(TokenArgs a) {
    const int unit = a.unit_begin + blockIdx.y;
    const int nb = a.B == 4 ? 4 : 1, l = blockIdx.z;  // staged high-frequency tensors per unit-tensor
    const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(a.z1) + ((int64_t)unit * 2 * nb + l) * a.unit_stride);
    uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(a.z1drop) + ((int64_t)unit * nb + l) * a.unit_stride);
    const uint8_t* flag = a.flag + (int64_t)unit * a.Tmax;
    const int64_t nvec = (int64_t)a.T * 16;
    for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < nvec; v += (int64_t)gridDim.x * blockDim.x) {
        uint4 x = src[v];
        if (flag[v >> 4]) x = make_uint4(0u, 0u, 0u, 0u);
        dst[v] = x;
    }
}

// out[j][:] = z1[list[j]][:] (rows of row_u4 16-byte vectors), optionally doubled (bf16 rows of the tensor-core decode
// kernel only; exact): a block of four scales its rows by 1/2 at decode time and its deviations by 1, so their stored
// rows carry the factor 2
__global__ void __launch_bounds__(256) token_gather_kernel(const uint4* z1, const int32_t* list, int64_t k_tok, uint4* out, int row_u4,
                                                           int twice) {
    for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < k_tok * row_u4; v += (int64_t)gridDim.x * blockDim.x) {
        uint4 x = z1[(int64_t)list[v / row_u4] * row_u4 + (v % row_u4)];
        if (twice) {
            __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&x);
#pragma unroll
            for (int i = 0; i < 4; ++i) h[i] = __hadd2(h[i], h[i]);
        }
        out[v] = x;
    }
}

// ---- storage types and head dimensions without the tensor-core kernel: the same score as a float32 product ----
template <typename T>
__device__ __forceinline__ float to_f32(T x);
template <>
__device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

constexpr int kSTile = 64;   // tokens per thread block
constexpr int kSRows = 16;   // probe rows staged per round
// grid (64-token tiles, units), 256 threads: thread (token j, row group rg) takes the maximum of |q_r . z[t]| over the
// rows r of its group whose probe position sees token t; the groups and the layers merge by atomicMax on the bit
// patterns of the non-negative floats.
template <typename T>
__global__ void __launch_bounds__(256) token_score_tile_kernel(TokenArgs a, int d) {
    extern __shared__ float ssm[];
    const int ld = d + 1;
    float* zs = ssm;                 // [64][d + 1]
    float* qs = zs + kSTile * ld;    // [16][d]
    const int unit = a.unit_begin + blockIdx.y;
    const int t0 = blockIdx.x * kSTile;
    const int nt = min(kSTile, a.T - t0);
    const int h = unit % a.Hkv, pair = unit / a.Hkv;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int j = (warp & 1) * 32 + lane, rg = warp >> 1;
    const int n_ops = a.B == 4 ? 4 : 1;
    const int M = (a.B == 4 ? 1 : 2) * a.G * a.W;  // probe rows per operand
    float best = 0.f;
    for (int op = 0; op < n_ops; ++op) {
        const T* z1 = reinterpret_cast<const T*>(a.z1) + ((int64_t)unit * 2 * n_ops + op) * a.unit_stride + (int64_t)t0 * d;
        for (int i = threadIdx.x; i < kSTile * d; i += blockDim.x) {
            const int t = i / d, c = i % d;
            zs[t * ld + c] = t < nt ? to_f32<T>(z1[i]) : 0.f;
        }
        __syncthreads();
        for (int rb = 0; rb < M; rb += kSRows) {
            for (int i = threadIdx.x; i < kSRows * d; i += blockDim.x) {
                const int r = rb + i / d, c = i % d;
                float v = 0.f;
                if (r < M) {
                    const int layer = a.B == 4 ? op : r / (a.G * a.W), g = (r / a.W) % a.G, qi = r % a.W;
                    const T* q = reinterpret_cast<const T*>(a.q_layers_dev[a.B * pair + layer]);
                    v = to_f32<T>(q[((int64_t)qi * a.Hq + h * a.G + g) * d + c]);
                }
                qs[i] = v;
            }
            __syncthreads();
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
            const float* zr = zs + j * ld;
            const float* qr = qs + rg * 4 * d;
            for (int c = 0; c < d; ++c) {
                const float zv = zr[c];
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[i] = fmaf(qr[i * d + c], zv, acc[i]);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int r = rb + rg * 4 + i;
                if (r < M && j < nt && t0 + j <= a.pos[r % a.W]) best = fmaxf(best, fabsf(acc[i]));
            }
            __syncthreads();
        }
    }
    // the score carries the factor of Eq. 1's inverse (c for a pair; a block of four's deviations are in layer space already)
    if (j < nt) atomicMax(a.score + (int64_t)unit * a.Tmax + t0 + j, __float_as_uint(best * (a.B == 4 ? 1.f : __uint_as_float(0x3F3504F3u))));
}

}  // namespace

cudaError_t launch_token_select(const TokenArgs& a, int dtype, int d, bool tensor_core, cudaStream_t st) {
    if (a.unit_count <= 0) return cudaSuccess;
    static PerDevice once;
    int sm_count = 0;
    const size_t tile_smem = (size_t)(kSTile * (d + 1) + kSRows * d) * sizeof(float);
    cudaError_t e0 = once.ensure([&]() {
        cudaError_t e1 = cudaFuncSetAttribute(token_score_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTSmem);
        if (e1 == cudaSuccess) e1 = cudaFuncSetAttribute(token_score_tile_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
        if (e1 == cudaSuccess) e1 = cudaFuncSetAttribute(token_score_tile_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
        return e1;
    }, &sm_count);
    if (e0 != cudaSuccess) return e0;
    cudaError_t e = cudaMemsetAsync(a.score + (int64_t)a.unit_begin * a.Tmax, 0, (size_t)a.unit_count * a.Tmax * 4, st);
    if (e != cudaSuccess) return e;
    if (!tensor_core) {
        // tokens after the last probe position are seen by nobody: score 0
        const int ntiles = std::min(a.T - 1, a.pos_host[a.W - 1]) / kSTile + 1;
        if (dtype == FDKV_BF16)
            token_score_tile_kernel<__nv_bfloat16><<<dim3(ntiles, a.unit_count), 256, tile_smem, st>>>(a, d);
        else
            token_score_tile_kernel<float><<<dim3(ntiles, a.unit_count), 256, tile_smem, st>>>(a, d);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        token_select_kernel<<<a.unit_count, 1024, 0, st>>>(a);
        count_launch(2);
        return cudaGetLastError();  // (the float32 probe kernel masks the selected rows itself: no dropped copy)
    }
    ScorePlan pl;
    pl.pos_min = a.pos_host[0];
    pl.ntiles = a.pos_host[a.W - 1] / kTM + 1;  // tokens after the last probe position are seen by nobody: score 0
    pl.mblocks = (a.G * a.W + kTN - 1) / kTN;
    const int base_items = a.unit_count * a.B * pl.mblocks;
    int nsplits = std::max(1, std::min((4 * sm_count + base_items - 1) / base_items, (pl.ntiles + 7) / 8));
    pl.tiles_per_split = (pl.ntiles + nsplits - 1) / nsplits;
    pl.nsplits = (pl.ntiles + pl.tiles_per_split - 1) / pl.tiles_per_split;
    pl.items_per_unit = a.B * pl.mblocks * pl.nsplits;
    token_score_kernel<<<a.unit_count * pl.items_per_unit, kTThreads, kTSmem, st>>>(*reinterpret_cast<const CUtensorMap*>(a.tmap_z1_128), a, pl);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    token_select_kernel<<<a.unit_count, 1024, 0, st>>>(a);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    const int blocks = (int)std::min<int64_t>(64, ((int64_t)a.T * 16 + 255) / 256);
    token_drop_kernel<<<dim3(blocks, a.unit_count, a.B == 4 ? 4 : 1), 256, 0, st>>>(a);
    count_launch(3);
    count_kernel(FDKV_KERNEL_TOKEN_SCORE);
    return cudaGetLastError();
}

cudaError_t launch_token_gather(const void* z1, const int32_t* list, int64_t k_tok, void* out, int row_bytes, int twice, cudaStream_t st) {
    if (k_tok <= 0) return cudaSuccess;
    const int row_u4 = row_bytes / 16;
    const int blocks = (int)std::min<int64_t>(256, (k_tok * row_u4 + 255) / 256);
    token_gather_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<const uint4*>(z1), list, k_tok, reinterpret_cast<uint4*>(out), row_u4, twice);
    count_launch(1);
    return cudaGetLastError();
}

}  // namespace fdkv
