// Routing probe on the 5th-generation tensor cores (bf16 storage, head_dim 128): the error term of Eq. 2.
//
// For a unit and a candidate (shared: R = Z1 of K; residual: R = Z1 of K with the kept entries zeroed) the probe
// needs sum_{rows, keys j <= pos(row)} (Q_row . R_j)^2 over the 2*G*W probe rows (2 layers x G group heads x W
// probe queries).  That is a dense [rows x 128] x [128 x T] contraction whose result is squared, masked causally
// and summed without ever leaving the SM:
//   * work item = (unit, layer of the pair, block of 128 probe rows, candidate, range of 256-token key tiles);
//     one CTA per item, 6 warps: warp 0 = TMA producer, warp 1 = MMA issuer (and TMEM owner), warps 2-5 = epilogue;
//   * A (the item's 128 Q rows) is written once into shared memory by the epilogue threads, in the
//     128-byte-swizzled K-major layout a TMA copy would give it; B tiles (256 tokens x 128 channels, same layout)
//     stream through a 3-stage TMA ring;
//   * per key tile 8 tcgen05.mma (M = 128, N = 256, K = 16, kind::f16, both operands from shared memory,
//     bf16 x bf16 -> f32) fill one of two alternating 128 x 256 f32 accumulators: all 512 columns of tensor memory.
//     The hand-over of an accumulator (commit -> epilogue -> release -> next MMA) is a round trip of about a
//     microsecond; with a single set it was paid on every tile and cost as much as the arithmetic, which is why A
//     lives in shared memory: the columns it took in tensor memory buy the second set.  (Two M tiles against
//     128-token key tiles, the same bytes per flop, measured 4 % slower.);
//   * epilogue: tcgen05.ld (32 lanes x 32 columns per instruction), square, mask keys after the row's probe
//     position, accumulate; the set is released as soon as its last columns are in registers; one float64 sum per
//     item, summed across items in a fixed order by the finalize kernel.
// Every mbarrier wait is bounded; on expiry the CTA flags the device status word, stops waiting and still frees
// its tensor memory before it retires.
#include <cuda.h>

#include <algorithm>

#include "fdkv_internal.h"
#include "mbar_wait.cuh"

namespace fdkv {

namespace {

constexpr int kBN = kProbeBoxRows;             // key tokens per tile (N of the MMA)
constexpr int kMT = 256 / kBN;                 // M tiles (128 Q rows each) per work item: 2 at N = 128, 1 at N = 256
constexpr int kBStages = kBN == 128 ? 5 : 3;
constexpr int kAccSets = 2;
constexpr int kBHalf = kBN * 128;              // one 64-channel half of a B tile: 32 KiB
constexpr int kBStageBytes = 2 * kBHalf;       // 64 KiB
constexpr int kHdr = 1024;
constexpr int kAHalf = 128 * 128;              // one 64-channel half of an A tile (128 Q rows): 16 KiB
constexpr int kABytes = kMT * 2 * kAHalf;      // the item's M tiles
constexpr int kProbeSmem = kHdr + kABytes + kBStages * kBStageBytes;  // 225 KiB in either form
constexpr int kPThreads = 6 * 32;
// Tensor memory (512 columns): two alternating sets of kMT 128 x kBN f32 accumulators (one per M tile).
constexpr int kTmemCols = 512;
constexpr int kAccSet = kMT * kBN;
static_assert(kAccSets * kAccSet <= kTmemCols && (kBN == 128 || kBN == 256), "tensor memory budget");
// header: full[8] @0, empty[8] @64, tfull[2] @128, tempty[2] @144, tmem slot @160, abort @164, reduce @192 (4 doubles)
constexpr int oFull = 0, oEmpty = 64, oTFull = 128, oTEmpty = 144, oSlot = 160, oAbort = 164, oRed = 192;

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
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);          // start address
    d |= (uint64_t)1 << 16;                            // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;                  // stride byte offset
    d |= (uint64_t)1 << 46;                            // descriptor version
    d |= (uint64_t)2 << 61;                            // 128-byte swizzle
    return d;
}
// instruction descriptor: D = f32, A = B = bf16, both K-major, M = 128, N = kBN
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);

// D[tmem] (+)= A[smem] * B[smem]^T; ACC = 0 overwrites D
template <int ACC>
__device__ __forceinline__ void umma_ss(uint32_t tmem_d, uint64_t da, uint64_t db) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
        "l"(da), "l"(db), "r"(kIdesc), "n"(ACC)
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

struct TcPlan {
    int items_per_unit;  // B layers x mblocks x 2 candidates x nsplits
    int mblocks, nsplits, ntiles, tiles_per_split;
    int pos_min, pos_max;
};

__global__ void __launch_bounds__(kPThreads, 1)
probe_tc_kernel(const __grid_constant__ CUtensorMap tmap_z1, const __grid_constant__ CUtensorMap tmap_drop, ProbeArgs a, TcPlan pl) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t sm0 = s_u32(smem);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + oAbort);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (sm0 & 1023u) {
        if (threadIdx.x == 0) atomicMax(a.status, (int32_t)kFlagCountMismatch);
        return;
    }
    // ---- decode the work item ----
    int it = blockIdx.x;
    const int unit = a.unit_begin + it / pl.items_per_unit;
    it %= pl.items_per_unit;
    const int split = it % pl.nsplits; it /= pl.nsplits;
    const int cand = it & 1; it >>= 1;
    const int mblock = it % pl.mblocks; it /= pl.mblocks;
    const int layer = it;  // layer inside the depth block: 0 .. B-1
    const int h = unit % a.Hkv, pair = unit / a.Hkv;
    const int tile0 = split * pl.tiles_per_split;
    const int tile1 = min(pl.ntiles, tile0 + pl.tiles_per_split);
    const int ntile = max(0, tile1 - tile0);
    const int rows_layer = a.G * a.W;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kBStages; ++s) { mb_init(sm0 + oFull + 8 * s, 1); mb_init(sm0 + oEmpty + 8 * s, 1); }
        for (int s = 0; s < 2; ++s) { mb_init(sm0 + oTFull + 8 * s, 1); mb_init(sm0 + oTEmpty + 8 * s, 4); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {  // tensor memory: all 512 columns
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sm0 + oSlot), "r"((uint32_t)kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(smem + oSlot);
    // ---- A operand: row r = mblock*256 + mt*128 + rl of this layer's probe block, r = g*W + qi -> Q[layer][qi][h*G+g][:],
    //      row rl of M tile mt: 16 chunks of 16 bytes, chunk c of a 64-channel half stored at chunk c ^ (rl & 7) ----
    if (warp >= 2) {
        const int rl = (warp & 3) * 32 + lane;
        const __nv_bfloat16* q = reinterpret_cast<const __nv_bfloat16*>(a.q_layers_dev[a.B * pair + layer]);
#pragma unroll 1
        for (int mt = 0; mt < kMT; ++mt) {
            const int r = mblock * (128 * kMT) + mt * 128 + rl;
            uint8_t* const arow = smem + kHdr + mt * 2 * kAHalf + rl * 128;
            const uint4* src = reinterpret_cast<const uint4*>(q + ((int64_t)(r % a.W) * a.Hq + h * a.G + r / a.W) * 128);
#pragma unroll
            for (int i = 0; i < 16; ++i)  // (padding rows are zero: they contribute nothing)
                *reinterpret_cast<uint4*>(arow + (i >> 3) * kAHalf + (((i & 7) ^ (rl & 7)) << 4)) = r < rows_layer ? src[i] : make_uint4(0u, 0u, 0u, 0u);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic stores, read by the tensor core
    }
    __syncthreads();
    const uint32_t b0 = sm0 + kHdr + kABytes;

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            const CUtensorMap* map = cand ? &tmap_drop : &tmap_z1;
            // rows of this unit's K coefficients: staged Z1 holds K and V per unit (unit-tensor 2*unit), the dropped copy K only
            // (a block of four layers stages one operand per layer: [unit-tensor][4] and [unit][4])
            const int64_t row0 = a.B == 4 ? ((cand ? (int64_t)unit : (int64_t)unit * 2) * 4 + layer) * a.Tmax
                                          : (cand ? (int64_t)unit : (int64_t)unit * 2) * a.Tmax;
            for (int i = 0; i < ntile; ++i) {
                const int s = i % kBStages;
                const uint32_t ph = (uint32_t)(i / kBStages) & 1u;
                mb_wait(sm0 + oEmpty + 8 * s, ph ^ 1u, abort_flag, a.status);
                if (*abort_flag) break;
                const uint32_t full = sm0 + oFull + 8 * s, dst = b0 + s * kBStageBytes;
                const int y = (int)(row0 + (int64_t)(tile0 + i) * kBN);
                mb_expect_tx(full, kBStageBytes);
                tma_2d(dst, map, 0, y, full);
                tma_2d(dst + kBHalf, map, 64, y, full);
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer =================
        if (lane == 0) {
            for (int i = 0; i < ntile; ++i) {
                const int s = i % kBStages, as = i % kAccSets;
                mb_wait(sm0 + oTEmpty + 8 * as, ((uint32_t)(i / kAccSets) & 1u) ^ 1u, abort_flag, a.status);
                mb_wait(sm0 + oFull + 8 * s, (uint32_t)(i / kBStages) & 1u, abort_flag, a.status);
                if (*abort_flag) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                // one descriptor per stage and for A; the k steps and the two M tiles only add compile-time constants
                const uint64_t db_stage = smem_desc(b0 + s * kBStageBytes);
                const uint64_t da_all = smem_desc(sm0 + kHdr);
                const uint32_t d0 = tmem_base + (uint32_t)(as * kAccSet);
#pragma unroll
                for (int k = 0; k < 8; ++k) {  // 8 steps of 16 channels: 32 bytes inside the swizzle atom of either operand
#pragma unroll
                    for (int mt = 0; mt < kMT; ++mt) {  // the M tiles alternate: consecutive MMAs never wait for each other's accumulator
                        const uint64_t db = db_stage + (uint64_t)(((k >> 2) * kBHalf + (k & 3) * 32) >> 4);
                        const uint64_t da = da_all + (uint64_t)((mt * 2 * kAHalf + (k >> 2) * kAHalf + (k & 3) * 32) >> 4);
                        if (k == 0) umma_ss<0>(d0 + mt * kBN, da, db);
                        else umma_ss<1>(d0 + mt * kBN, da, db);
                    }
                }
                umma_commit(sm0 + oEmpty + 8 * s);    // the B stage is free once these MMAs have read it
                umma_commit(sm0 + oTFull + 8 * as);   // the accumulators are complete
            }
        }
    } else {
        // ================= epilogue: warps 2..5 own TMEM lanes 32*(warp%4) .. +31 =================
        const int lq = warp & 3;
        const int rl = lq * 32 + lane;  // row within a 128-row M tile == TMEM lane
        int pos_row[kMT];
#pragma unroll
        for (int mt = 0; mt < kMT; ++mt) {
            const int r = mblock * (128 * kMT) + mt * 128 + rl;
            pos_row[mt] = r < rows_layer ? a.pos[r % a.W] : -1;  // padding rows never count
        }
        double total = 0.0;
        for (int i = 0; i < ntile; ++i) {
            const int as = i % kAccSets;
            const int t0 = (tile0 + i) * kBN;
            mb_wait(sm0 + oTFull + 8 * as, (uint32_t)(i / kAccSets) & 1u, abort_flag, a.status);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            float acc = 0.f;
            if (!*abort_flag) {
                const bool all_visible = t0 + kBN - 1 <= pl.pos_min;  // every key of the tile precedes every probe position
#pragma unroll
                for (int round = 0; round < kAccSet / 64; ++round) {  // 64 accumulator columns of this lane per round, two loads in flight
                    const int mt = round / (kBN / 64), c0 = (round % (kBN / 64)) * 64;
                    uint32_t r0[32], r1[32];
                    const uint32_t ta = tmem_base + ((uint32_t)(lq * 32) << 16) + (uint32_t)(as * kAccSet + mt * kBN + c0);
                    const int tc = t0 + c0;
                    tmem_ld32(ta, r0);
                    tmem_ld32(ta + 32, r1);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    if (round == kAccSet / 64 - 1) {  // the set's last columns are in registers: hand it back before the arithmetic
                        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                        __syncwarp();
                        if (lane == 0) mb_arrive(sm0 + oTEmpty + 8 * as);
                    }
                    if (all_visible && pos_row[mt] >= 0) {
                        float acc1 = 0.f;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const float u = __uint_as_float(r0[j]), v = __uint_as_float(r1[j]);
                            acc = fmaf(u, u, acc);
                            acc1 = fmaf(v, v, acc1);
                        }
                        acc += acc1;
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const float u = __uint_as_float(r0[j]), v = __uint_as_float(r1[j]);
                            if (tc + j <= pos_row[mt]) acc = fmaf(u, u, acc);
                            if (tc + 32 + j <= pos_row[mt]) acc = fmaf(v, v, acc);
                        }
                    }
                }
            } else {
                __syncwarp();
                if (lane == 0) mb_arrive(sm0 + oTEmpty + 8 * as);
            }
            total += (double)acc;
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) total += __shfl_xor_sync(0xFFFFFFFFu, total, o);
        if (lane == 0) reinterpret_cast<double*>(smem + oRed)[lq] = total;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (*abort_flag)
        for (int i = 0; i < 200; ++i) __nanosleep(1000);  // let copies and MMAs in flight finish before the memory goes away
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTmemCols) : "memory");
    }
    if (threadIdx.x == 0) {
        const double* red = reinterpret_cast<const double*>(smem + oRed);
        // part slot of this item inside its unit: (layer, mblock, split); candidate selects the column
        const int slot = (layer * pl.mblocks + mblock) * pl.nsplits + split;
        a.part[((int64_t)unit * a.nptiles_max + slot) * 2 + cand] = red[0] + red[1] + red[2] + red[3];
    }
}

}  // namespace

cudaError_t launch_probe_tc(const ProbeArgs& a, int dtype, cudaStream_t st, bool* handled, int* nparts) {
    *handled = false;
    if (dtype != FDKV_BF16 || a.d != 128 || !a.tmap_z1 || !a.tmap_drop) return cudaSuccess;
    static PerDevice once;
    int sm_count = 0;
    cudaError_t e0 = once.ensure([&]() { return cudaFuncSetAttribute(probe_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kProbeSmem); }, &sm_count);
    if (e0 != cudaSuccess) return e0;
    TcPlan pl;
    pl.pos_min = a.pos_host[0];
    pl.pos_max = a.pos_host[a.W - 1];
    pl.ntiles = pl.pos_max / kBN + 1;  // keys after the last probe position never count
    pl.mblocks = (a.G * a.W + 128 * kMT - 1) / (128 * kMT);
    const int base_items = a.unit_count * a.B * pl.mblocks * 2;
    // split the key range so that the grid fills the machine several times over, but keep >= 8 tiles per item
    int nsplits = std::max(1, std::min((4 * sm_count + base_items - 1) / base_items, (pl.ntiles + 7) / 8));
    pl.tiles_per_split = (pl.ntiles + nsplits - 1) / nsplits;
    nsplits = (pl.ntiles + pl.tiles_per_split - 1) / pl.tiles_per_split;
    pl.nsplits = nsplits;
    pl.items_per_unit = a.B * pl.mblocks * 2 * nsplits;
    const int slots = a.B * pl.mblocks * nsplits;
    if (slots > a.nptiles_max) return cudaErrorInvalidValue;  // cannot happen: the part array is sized for max_probe_parts()
    probe_tc_kernel<<<a.unit_count * pl.items_per_unit, kPThreads, kProbeSmem, st>>>(
        *reinterpret_cast<const CUtensorMap*>(a.tmap_z1), *reinterpret_cast<const CUtensorMap*>(a.tmap_drop), a, pl);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    count_launch(1);
    count_kernel(FDKV_KERNEL_PROBE_TC);
    *nparts = slots;
    *handled = true;
    return cudaSuccess;
}

}  // namespace fdkv
