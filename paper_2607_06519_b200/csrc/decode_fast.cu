// Decode attention over the packed cache for bf16 storage, head_dim 128 (the paragraph after Eq. 3: shared
// coefficients broadcast to both layers of the pair, residual coefficients added only where indexed, the full
// cache never materialised).
//
// One persistent CTA of eight warps per SM.  128-token K and V boxes of the packed cache stream through a ring of
// shared-memory stages with TMA (128-byte swizzle, mbarrier completion).  The CTA's tile sequence sits in a small
// segment table in shared memory; whichever warp finishes a tile last re-arms its stage with the tile three ahead,
// so no warp is a dedicated producer.  Each warp owns 16 tokens of a stage and a private online-softmax state:
//   S = K q^T        mma.sync m16n8k16, tokens on M (ldmatrix of the swizzled K box), the G query heads on N;
//   P = exp2(S - max) per column; for G <= 4 columns 4-7 repeat the heads and carry the bf16 rounding remainder of
//                    P, so P acts with ~16 bits; movmatrix turns the accumulator layout into the next B operand;
//   O^T += V^T P^T   mma.sync, channels on M (ldmatrix.trans of the V box).
// (Heads on M, as in a prefill kernel, would use 4 of 16 rows and twice the instructions: mma.sync runs at a quarter
// of the tcgen05 rate on this part and was the limiter in that form.)
// Residual units: the warp scatters its slice's kept Z1 entries into a private zeroed 16x128 bf16 scratch tile
// and runs the same two products on it with the layer's sign, so the correction is exact in float32.  (Adding the
// entries into the landed rows in place, rounded to bf16, was faster to write but quadrupled the output error.)
// The list ranges are loaded one tile per lane 32-64 tiles ahead and handed out by shuffle; the lists themselves
// are pulled into L2 three tiles ahead and into registers one tile ahead.
// Work is a flat list of (unit, tile) pairs cut into one contiguous range per CTA (cost-weighted), so a CTA may
// finish one unit and start the next; each (CTA, unit) segment writes one split-K partial and the CTA that takes
// the unit's last ticket combines them.
#include <cuda.h>
#include <cuda_fp16.h>

#include <algorithm>

#include "fdkv_internal.h"
#include "mbar_wait.cuh"

namespace fdkv {

namespace {

constexpr int kTT = 128;         // tokens per stage
constexpr int kStages = 3;
constexpr int kCW = kTT / 16;    // warps, 16 tokens of a stage each
constexpr int kThreads = kCW * 32;  // 256 threads: two warps per scheduler, so up to 255 registers per thread
constexpr int kHalfBytes = kTT * 128;        // one 64-channel box of 128 tokens
constexpr int kStageBytes = 4 * kHalfBytes;  // K ch 0-63, K ch 64-127, V ch 0-63, V ch 64-127
constexpr int kScratchBytes = 4096;          // per consumer warp: 16 tokens x 128 channels bf16 (or its O tile at merge)
constexpr int kHeaderBytes = 2048;
constexpr int kMaxSeg = 24;  // (unit, range) segments one CTA can walk: at most units / CTAs + 2
constexpr int kSmemBytes = kHeaderBytes + kStages * kStageBytes + kCW * kScratchBytes;
constexpr int kMaxCtas = 296;
constexpr int kMaxUnits = kFastMaxUnits;
constexpr int kPF = 8;  // residual entries prefetched per lane and list
constexpr int kPartStride = 128 + 4;  // floats per split-K part: max, sum, 2 pad, 128 accumulators (16-byte aligned)
static_assert(kTT == kRowPad, "row blocks are padded to whole stages");
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");

struct FastSched {
    uint32_t start[kMaxCtas + 1];  // unit << 20 | first 16-token slice of CTA c; start[ncta] = units << 20
    int ncta, units;
    int any_tail;  // some sequence of the batch holds generated tokens in this layer's tail (host mirror)
};
struct PartCount {
    uint8_t n[kMaxUnits];  // split-K parts per unit (at most kMaxSplits)
};
struct TailLens {
    int32_t n[kMaxUnits];  // generated tokens in this layer's tail per sequence, this call's append included (host mirror)
};
static_assert(kMaxSplits < 256 && kMaxSplits % 32 == 0, "part counts are bytes; the combine holds one part per lane and round");

// header offsets
constexpr int kOffFull = 0, kOffAbort = 128, kOffTicket = 132, kOffM = 256, kOffL = 512, kOffSeg = 1024, kOffSegInfo = 1920,
              kOffCnt = 1936;
// one (unit, tile range) segment of a CTA: arena rows of its K / V boxes and tail, first tile, prefill tiles, first
// index in the CTA's tile sequence, and the sequence / head whose tail it also streams (or -1)
struct Seg {
    int krow, vrow, tkrow, tvrow;
    int tb, rows16, npre;  // first token of the range, its tokens rounded up to 16, its 128-token tiles (the last may be partial)
    int it0, tail_u;       // first tile in the CTA's sequence; the unit whose tail follows the range, or -1
};
static_assert(kMaxSeg * sizeof(Seg) <= 896, "segment table fits its header slot");

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t movmatrix_t(uint32_t a) {  // transpose an 8 x 8 matrix of 16-bit elements held by the warp
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                        uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// the two e4m3 bytes in the low half of x -> two f16 values (exact).  (An integer form - byte permute, shift, mask, with a
// factor 2^-8 folded into the scales - was measured: 15 % slower alone, 9 % slower when sharing the work half and half.)
__device__ __forceinline__ uint32_t cvt_e4m3x2(uint32_t x) {
    uint32_t d;
    asm("{\n\t.reg .b16 t;\n\tcvt.u16.u32 t, %1;\n\tcvt.rn.f16x2.e4m3x2 %0, t;\n\t}" : "=r"(d) : "r"(x));
    return d;
}
__device__ __forceinline__ uint32_t prmt1(uint32_t a, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %1, %2;" : "=r"(d) : "r"(a), "r"(sel));
    return d;
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
    const __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void st_shared_u16(uint32_t addr, uint16_t v) {
    asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"(v) : "memory");
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void st_shared_zero16(uint32_t addr) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(addr), "r"(0u) : "memory");
}

// byte offset of (row, channel chunk of 8) inside a [rows][64 ch] box with the 128-byte swizzle
__device__ __forceinline__ uint32_t swz(int row, int chunk8) { return (uint32_t)(row * 128 + (((chunk8 & 7) ^ (row & 7)) << 4)); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(lo)) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(hi)) << 16);
}


// F8: the packed rows are e4m3 codes (one 128-byte row per token, per-channel float32 scales): the codes are converted
// to f16 in registers after ldmatrix, both products run as f16 mma with the K scales folded into q and the V scales
// applied to the output; the residual scratch tile then holds f16 values relative to the scales, in the converted
// fragments' channel order (the commit step writes the lists that way).  The generated-token tails stay bf16: when a
// segment reaches them the warp stashes the softmax state of its 8-bit tiles, runs the tails with the plain bf16 code
// on a fresh state and joins the two at the merge.
template <bool F8>
__global__ void __launch_bounds__(kThreads, 1)
decode_fast_kernel(const __grid_constant__ CUtensorMap tmap, const __grid_constant__ CUtensorMap tmap8, DecodeArgs a, FastSched sch,
                   PartCount pc, TailLens tl) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t smem0 = smem_u32(smem_raw);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem_raw + kOffAbort);
    if (smem0 & 1023u) {  // the swizzled boxes need 1024-byte alignment; report instead of computing garbage
        if (threadIdx.x == 0) atomicMax(a.status, (int32_t)kFlagCountMismatch);
        return;
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // Let the next kernel in the stream start its own prologue as soon as SMs free up (programmatic dependent
    // launch); everything this kernel reads before its own griddepcontrol.wait is static since commit.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem0 + kOffFull + 8 * s, 1);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }

    const int cta = blockIdx.x;
    const uint32_t s0 = sch.start[cta], s1 = sch.start[cta + 1];
    const int u_first = (int)(s0 >> 20), t_first = (int)(s0 & 0xFFFFFu);
    const int u_last = (int)(s1 >> 20), t_last = (int)(s1 & 0xFFFFFu);
    const uint64_t arena = reinterpret_cast<uint64_t>(a.arena_base);
    const uint32_t stage0 = smem0 + kHeaderBytes;
    const bool is_producer = threadIdx.x == 0;
    // The second layer of a pair walks every range backwards: it starts on the Z0 rows the first layer read last,
    // which are the ones most likely still in L2 (both layers of a shared / residual unit stream the same Z0).
    // (Measured: 1.4 % per step; L2 eviction hints on the TMA loads did not add to it.)
    const bool rev = (a.layer & 1) != 0;

    // ================= the CTA's tile sequence: a small segment table in shared memory =================
    // Tile `it` of the CTA (all segments, prefill tiles then tail tiles of each) always lands in stage it % kStages.
    // Whichever warp is the last to finish a tile refills its stage with tile it + kStages at once (a counter per
    // stage, no waiting producer), so copies are issued the moment a stage is free.
    Seg* const segs = reinterpret_cast<Seg*>(smem_raw + kOffSeg);
    int* const seg_info = reinterpret_cast<int*>(smem_raw + kOffSegInfo);  // [0] segments, [1] tiles in total
    int* const stage_cnt = reinterpret_cast<int*>(smem_raw + kOffCnt);
    auto issue_rows = [&](int s, int kr, int vr, bool f8_box) {  // s = the tile's stage (its index in the CTA's sequence mod kStages)
        const uint32_t full = smem0 + kOffFull + 8 * s;
        const uint32_t dst = stage0 + s * kStageBytes;
        if (F8 && f8_box) {  // one 128-token x 128-byte box per tensor, in the first half of the K and of the V slot
            mbar_expect_tx(full, 2 * kHalfBytes);
            tma_load_2d(dst, &tmap8, 0, kr, full);
            tma_load_2d(dst + 2 * kHalfBytes, &tmap8, 0, vr, full);
        } else {
            mbar_expect_tx(full, kStageBytes);
            tma_load_2d(dst, &tmap, 0, kr, full);
            tma_load_2d(dst + kHalfBytes, &tmap, 64, kr, full);
            tma_load_2d(dst + 2 * kHalfBytes, &tmap, 0, vr, full);
            tma_load_2d(dst + 3 * kHalfBytes, &tmap, 64, vr, full);
        }
    };
    auto issue_tile = [&](int it) {
        int si = 0;
        while (si + 1 < seg_info[0] && it >= segs[si + 1].it0) ++si;
        const Seg g = segs[si];
        const int j = it - g.it0;
        // ranges start on any 16-token slice and their tiles count from there; the box of the partial tile that ends a
        // range is moved back over rows the CTA has read already (masked when used), so that no copy passes the range's end
        const int tok = max(0, g.tb + min((rev ? g.npre - 1 - j : j) * kTT, g.rows16 - kTT));
        const int kr = j < g.npre ? g.krow + tok : g.tkrow + (j - g.npre) * kTT;
        const int vr = j < g.npre ? g.vrow + tok : g.tvrow + (j - g.npre) * kTT;
        issue_rows(it % kStages, kr, vr, j < g.npre);
    };
    int prologue_issued = 0;
    if (is_producer) {
        // static part (packed cache, fixed since commit): may run before the dependency wait
        int n = 0, it0 = 0;
        for (int u = u_first; u <= u_last && u < sch.units; ++u) {
            const int b = u / a.Hkv, h = u % a.Hkv;
            const UnitDesc* ud = a.desc + ((int64_t)b * a.L + a.layer) * a.Hkv + h;
            const int nsl = (ud->T + kResTile - 1) / kResTile;
            const int sb = u == u_first ? t_first : 0;
            const int se = u == u_last ? t_last : nsl;
            if (se <= sb) continue;
            if (n == kMaxSeg) { atomicMax(a.status, (int32_t)kFlagCountMismatch); break; }  // cannot happen: see the launcher
            Seg g;
            g.krow = (int)((reinterpret_cast<uint64_t>(ud->k_rows) - arena) >> (F8 ? 7 : 8));  // rows of 128 or 256 bytes
            g.vrow = (int)((reinterpret_cast<uint64_t>(ud->v_rows) - arena) >> (F8 ? 7 : 8));
            g.tkrow = g.tvrow = 0;
            g.tb = sb * kResTile;
            g.rows16 = (min(se, nsl) - sb) * kResTile;
            g.npre = (g.rows16 + kTT - 1) / kTT;
            g.it0 = it0;
            g.tail_u = se == nsl ? u : -1;  // this CTA also streams the unit's tail (length known after the wait)
            segs[n++] = g;
            it0 += g.npre;
        }
        seg_info[0] = n;
        seg_info[1] = it0;
        for (int s = 0; s < kStages; ++s) stage_cnt[s] = 0;
        if (n > 0)
            for (; prologue_issued < kStages && prologue_issued < segs[0].npre; ++prologue_issued)
                issue_tile(prologue_issued);
    }
    // per-warp scratch starts zeroed
    for (int i = threadIdx.x; i < kCW * kScratchBytes / 16; i += kThreads)
        st_shared_zero16(smem0 + kHeaderBytes + kStages * kStageBytes + i * 16);
    __syncthreads();  // barriers initialised, static table built (still inside the previous kernel's shadow)
    // everything below may depend on the kernels launched before this one (q, appended tail rows, partial slots)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (!sch.any_tail) {
        // no tails anywhere: the static table is final; a short first segment may have left stages to fill
        if (is_producer)
            for (int it = prologue_issued; it < kStages && it < seg_info[1]; ++it) issue_tile(it);
    } else {
    if (warp == 0 && a.k_new) {
        // Generated tokens of this call: the thread block that streams a unit's tail appends the unit's new K and V
        // rows itself (16 lanes x 16 bytes each) and makes them visible to the tensor copies it issues next; a layer
        // call stays one kernel, and k_new / v_new are read behind the dependency wait.
        for (int i = 0; i < seg_info[0]; ++i) {
            const int tu = segs[i].tail_u;
            if (tu < 0) continue;
            const int tb = tu / a.Hkv, th = tu % a.Hkv;
            const int n = min(tl.n[tb], a.max_tail);
            if (n <= 0) continue;
            const int64_t row = (((int64_t)a.layer * a.max_batch + tb) * a.Hkv + th) * a.tail_rows + (n - 1);
            const uint4* src = reinterpret_cast<const uint4*>(lane < 16 ? a.k_new : a.v_new) + ((int64_t)tb * a.Hkv + th) * 16 + (lane & 15);
            uint4* dst = reinterpret_cast<uint4*>(lane < 16 ? a.tail_k : a.tail_v) + row * 16 + (lane & 15);
            *dst = *src;
            if (lane == 0 && th == 0) a.tail_len[a.layer * a.max_batch + tb] = n;  // the device copy of the length (other kernels read it)
        }
        asm volatile("fence.proxy.async;" ::: "memory");
        __syncwarp();
    }
    if (is_producer) {
        // tails: rows may have been written by the kernel right before this one (or just above); lengths are the host's
        int it0 = 0;
        for (int i = 0; i < seg_info[0]; ++i) {
            Seg g = segs[i];
            g.it0 = it0;
            if (g.tail_u >= 0) {
                const int tail_b = g.tail_u / a.Hkv, tail_h = g.tail_u % a.Hkv;
                const int n = min(tl.n[tail_b], a.max_tail);
                const int64_t o = (((int64_t)a.layer * a.max_batch + tail_b) * a.Hkv + tail_h) * a.tail_rows;
                g.tkrow = (int)(((reinterpret_cast<uint64_t>(a.tail_k) - arena) >> 8) + o);
                g.tvrow = (int)(((reinterpret_cast<uint64_t>(a.tail_v) - arena) >> 8) + o);
                it0 += (n + kTT - 1) / kTT;
            }
            it0 += g.npre;
            segs[i] = g;
        }
        seg_info[1] = it0;
        for (int it = prologue_issued; it < kStages && it < it0; ++it) issue_tile(it);  // nobody computes yet: fill every stage
    }
    __syncthreads();
    }

    // ================= compute: every warp takes 16 tokens of every stage =================
    {
        const int gid = lane >> 2, tig = lane & 3;  // mma fragment coordinates: head row, column pair
        const int r0 = warp * 16;
        const uint32_t scratch = smem0 + kHeaderBytes + kStages * kStageBytes + warp * kScratchBytes;
        float* const scratch_f = reinterpret_cast<float*>(smem_raw + kHeaderBytes + kStages * kStageBytes + warp * kScratchBytes);
        float* const sm_m = reinterpret_cast<float*>(smem_raw + kOffM);
        float* const sm_l = reinterpret_cast<float*>(smem_raw + kOffL);
        const float kLog2e = 1.4426950408889634f;
        const float kLazyMax = 8.f;  // (log2 units) the running maximum is only moved when a score passes it by more than this
        const float inv_sqrt_d = 0.08838834764831845f;  // 1/sqrt(128)

        int it = 0;
        for (int u = u_first; u <= u_last && u < sch.units; ++u) {
            const int b = u / a.Hkv, h = u % a.Hkv;
            const UnitDesc ud = a.desc[((int64_t)b * a.L + a.layer) * a.Hkv + h];
            const int T = ud.T;
            const int nres = (T + kResTile - 1) / kResTile;
            const int sb = u == u_first ? t_first : 0;
            const int se = u == u_last ? t_last : nres;
            if (se <= sb) continue;
            // this CTA's tokens of the unit: [tok_b, tok_e), cut on 16-token slices; 128-token tiles count from tok_b
            const int tok_b = sb * kResTile, tok_e = min(se * kResTile, T), rows16 = (se - sb) * kResTile;
            int ntail = 0, n_tail_rows = 0;
            if (sch.any_tail && se == nres) {
                n_tail_rows = min(tl.n[b], a.max_tail);
                ntail = (n_tail_rows + kTT - 1) / kTT;
            }
            const int npre = (rows16 + kTT - 1) / kTT, nseg = npre + ntail;
            const bool coef = ud.mode != FDKV_MODE_EXACT, resid = ud.mode == FDKV_MODE_RESIDUAL;
            const uint32_t sgn = ud.sign < 0.f ? 0x80008000u : 0u;

            // q fragments: B operand columns = the G query heads of this KV head.  With G <= 4 columns 4-7 repeat
            // them: in the second product those columns carry the bf16 rounding remainder of P, so P acts in ~16 bits.
            const bool split = a.G <= 4;
            const int qcol = split ? (gid & 3) : gid;
            uint32_t qb[8][2];
            auto load_q = [&](bool f8) {
                const __nv_bfloat16* qh = reinterpret_cast<const __nv_bfloat16*>(a.q) + ((int64_t)b * a.Hq + h * a.G + qcol) * 128;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    if (F8 && f8) {
                        // a converted register holds channels 4 tig .. 4 tig + 3 of the 16-channel step: its low pair is the
                        // first k-slot pair, its high pair the second; q carries the K scales, as f16
                        const int c0 = 16 * kk + 4 * tig;
                        float qv[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) qv[i] = qcol < a.G ? __bfloat162float(qh[c0 + i]) * ud.k_scale[c0 + i] : 0.f;
                        qb[kk][0] = pack_f16(qv[0], qv[1]);
                        qb[kk][1] = pack_f16(qv[2], qv[3]);
                    } else {
                        qb[kk][0] = qcol < a.G ? *reinterpret_cast<const uint32_t*>(qh + 16 * kk + 2 * tig) : 0u;
                        qb[kk][1] = qcol < a.G ? *reinterpret_cast<const uint32_t*>(qh + 16 * kk + 8 + 2 * tig) : 0u;
                    }
                }
            };
            if constexpr (F8) {
                load_q(true);
            } else {  // (kept inline for the bf16 kernel: routing it through the lambda cost 0.5 %)
                const __nv_bfloat16* qh = reinterpret_cast<const __nv_bfloat16*>(a.q) + ((int64_t)b * a.Hq + h * a.G + qcol) * 128;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    qb[kk][0] = qcol < a.G ? *reinterpret_cast<const uint32_t*>(qh + 16 * kk + 2 * tig) : 0u;
                    qb[kk][1] = qcol < a.G ? *reinterpret_cast<const uint32_t*>(qh + 16 * kk + 8 + 2 * tig) : 0u;
                }
            }
            // O^T[channel][column]: eight 16-channel m-tiles; this thread holds columns 2 tig, 2 tig + 1
            float oacc[8][4];
#pragma unroll
            for (int j = 0; j < 8; ++j) oacc[j][0] = oacc[j][1] = oacc[j][2] = oacc[j][3] = 0.f;
            float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};  // per held column; l is this thread's share
            float m_st[2] = {-INFINITY, -INFINITY}, l_st[2] = {0.f, 0.f};     // 8-bit rows: the state stashed before the bf16 tails
            bool stashed = false;
            // split-K part slot of this segment = number of CTAs with tiles of this unit before this one
            int slot = 0;
            for (int c2 = cta - 1; c2 >= 0; --c2) {
                const uint32_t ustart = (uint32_t)u << 20, e2 = sch.start[c2 + 1], s2 = sch.start[c2];
                if (e2 <= ustart) break;                 // ends before this unit's first tile
                if (max(s2, ustart) < e2) ++slot;        // a non-empty range inside this unit
                if (s2 <= ustart) break;
            }

            // ---- residual lists (packed entries): ranges two tiles ahead, entries one tile ahead ----
            const uint32_t* k_ent = reinterpret_cast<const uint32_t*>(ud.k_idx);
            const uint32_t* v_ent = reinterpret_cast<const uint32_t*>(ud.v_idx);
            int cr[4] = {0, 0, 0, 0}, nr[4] = {0, 0, 0, 0}, fr[4] = {0, 0, 0, 0};  // {k begin, k end, v begin, v end}: this tile, next, the one after
            uint32_t pke[kPF], pve[kPF];
            // token-granular residual: one ascending token list (k_idx) with per-slice counts (k_off) for K and V,
            // and the selected tokens' Z1 rows packed densely (k_val / v_val, 256 bytes each)
            const bool tokmode = resid && ud.res_kind == 1;
            const uint4* t_krows = reinterpret_cast<const uint4*>(ud.k_val);
            const uint4* t_vrows = reinterpret_cast<const uint4*>(ud.v_val);
            int ptk[2] = {0, 0}, ptv[2] = {0, 0};
            // List ranges of this warp's slice, one tile per lane: lane l of a batch holds tile rb + l of the segment
            // ({begin, end} of the K and of the V list), loaded 32 to 64 tiles before use and handed out by shuffle.
            int rb = 0, rk[2] = {0, 0}, rv[2] = {0, 0}, rk_n[2] = {0, 0}, rv_n[2] = {0, 0};
            auto load_batch = [&](int jb, int (&k)[2], int (&v)[2]) {
                const int jj = jb + lane;
                k[0] = k[1] = v[0] = v[1] = 0;
                if (resid && jj < npre) {
                    // the tile's slices not yet read: [first, se); the box may start before them (see issue_tile)
                    const int first = sb + (rev ? npre - 1 - jj : jj) * (kTT / kResTile);
                    const int o = max(0, min(first, se - kTT / kResTile)) + warp;
                    const int o0 = min(max(o, first), se), o1 = min(max(o + 1, first), se);
                    k[0] = ud.k_off[o0]; k[1] = ud.k_off[o1];
                    if (tokmode) { v[0] = k[0]; v[1] = k[1]; }
                    else { v[0] = ud.v_off[o0]; v[1] = ud.v_off[o1]; }
                }
            };
            auto get_ranges = [&](int j, int (&r)[4]) {  // rb <= j < rb + 64
                const bool nx = j - rb >= 32;
                const int src = (j - rb) & 31;
                r[0] = __shfl_sync(0xFFFFFFFFu, nx ? rk_n[0] : rk[0], src);
                r[1] = __shfl_sync(0xFFFFFFFFu, nx ? rk_n[1] : rk[1], src);
                r[2] = __shfl_sync(0xFFFFFFFFu, nx ? rv_n[0] : rv[0], src);
                r[3] = __shfl_sync(0xFFFFFFFFu, nx ? rv_n[1] : rv[1], src);
            };
            // pull a tile's list slices (or selected token rows) into L2 a few tiles ahead: lanes 0-15 the K side,
            // lanes 16-31 the V side, one 128-byte line each
            auto l2_prefetch = [&](const int (&r)[4]) {
                const int hl = lane & 15;
                const void* ptr = nullptr;
                if (tokmode) {
                    const int j = r[0] + (hl >> 1);
                    if (j < r[1]) ptr = reinterpret_cast<const char*>(lane < 16 ? t_krows : t_vrows) + (int64_t)j * 256 + (hl & 1) * 128;
                } else {
                    const int e0 = lane < 16 ? r[0] : r[2], e1 = lane < 16 ? r[1] : r[3];
                    const int e = (e0 & ~31) + 32 * hl;
                    if (e < e1) ptr = (lane < 16 ? k_ent : v_ent) + e;
                }
                if (ptr) asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr));
            };
            auto prefetch = [&](const uint32_t* ent, int e0, int e1, uint32_t (&pe)[kPF]) {
#pragma unroll
                for (int i = 0; i < kPF; ++i) {
                    const int e = e0 + lane + 32 * i;
                    if (e < e1) pe[i] = ent[e];
                }
            };
            // scatter one list slice into the scratch tile: each entry carries its own shared-memory offset
            auto scatter = [&](const uint32_t* ent, int e0, int e1, const uint32_t (&pe)[kPF]) {
#pragma unroll
                for (int i = 0; i < kPF; ++i) {
                    const int e = e0 + lane + 32 * i;
                    if (e < e1) st_shared_u16(scratch + ((pe[i] >> 16) << 1), (uint16_t)(pe[i] & 0xFFFFu));
                }
                for (int e = e0 + 32 * kPF + lane; e < e1; e += 32) {  // dense slices: direct loads
                    const uint32_t w = ent[e];
                    st_shared_u16(scratch + ((w >> 16) << 1), (uint16_t)(w & 0xFFFFu));
                }
            };
            // token rows: two tokens per round (half a warp each, 16 bytes per lane), two rounds in registers
            auto prefetch_tok = [&](const uint4* rows, int e0, int e1, uint32_t (&pe)[kPF], int (&pt)[2]) {
#pragma unroll
                for (int r = 0; r < 2; ++r) {
                    const int j = e0 + 2 * r + (lane >> 4);
                    if (j < e1) {
                        const uint4 v = rows[(int64_t)j * 16 + (lane & 15)];
                        pe[4 * r] = v.x; pe[4 * r + 1] = v.y; pe[4 * r + 2] = v.z; pe[4 * r + 3] = v.w;
                        pt[r] = k_ent[j];  // the token list sits where the packed layout keeps the K entries
                    }
                }
            };
            auto scatter_tok = [&](const uint4* rows, int e0, int e1, const uint32_t (&pe)[kPF], const int (&pt)[2]) {
                const int chunk = lane & 15;
#pragma unroll
                for (int r = 0; r < 2; ++r) {
                    const int j = e0 + 2 * r + (lane >> 4);
                    if (j < e1) {
                        const int row = pt[r] & 15;
                        st_shared_v4(scratch + (chunk >> 3) * 2048 + swz(row, chunk), pe[4 * r], pe[4 * r + 1], pe[4 * r + 2], pe[4 * r + 3]);
                    }
                }
                for (int j = e0 + 4 + (lane >> 4); j < e1; j += 2) {  // more than four selected tokens in the slice
                    const int row = (int)k_ent[j] & 15;
                    const uint4 v = rows[(int64_t)j * 16 + chunk];
                    st_shared_v4(scratch + (chunk >> 3) * 2048 + swz(row, chunk), v.x, v.y, v.z, v.w);
                }
            };
            auto zero_scratch = [&]() {
#pragma unroll
                for (int i = 0; i < kScratchBytes / 16 / 32; ++i) st_shared_zero16(scratch + (lane + 32 * i) * 16);
            };
            if (resid) {
                load_batch(0, rk, rv);
                load_batch(32, rk_n, rv_n);
                get_ranges(0, cr);
                get_ranges(1, nr);
                get_ranges(2, fr);
                l2_prefetch(nr);
                l2_prefetch(fr);
                if (tokmode) {
                    prefetch_tok(t_krows, cr[0], cr[1], pke, ptk);
                    prefetch_tok(t_vrows, cr[2], cr[3], pve, ptv);
                } else {
                    prefetch(k_ent, cr[0], cr[1], pke);
                    prefetch(v_ent, cr[2], cr[3], pve);
                }
            }

            // A warp is done reading stage s (tile j of this segment): the last of the eight refills it.  Three tiles ahead
            // is usually still a packed tile of this segment, whose rows follow from registers; only across a segment
            // boundary (or into the tails) the segment table is walked.  The refill sits on the critical path of the ring.
            const int unit_kr = (int)((reinterpret_cast<uint64_t>(ud.k_rows) - arena) >> (F8 ? 7 : 8));
            const int unit_vr = (int)((reinterpret_cast<uint64_t>(ud.v_rows) - arena) >> (F8 ? 7 : 8));
            auto release_here = [&](int s, int j) {
                __syncwarp();
                if (lane == 0) {
                    // (atomicInc wraps the counter back to zero at the eighth arrival; tile j + kStages reuses stage s)
                    const unsigned old = atomicInc(reinterpret_cast<unsigned*>(stage_cnt) + s, kCW - 1);
                    if (old == kCW - 1) {
                        const int jn = j + kStages;
                        if (jn < npre) {
                            const int tok = max(0, tok_b + min((rev ? npre - 1 - jn : jn) * kTT, rows16 - kTT));
                            issue_rows(s, unit_kr + tok, unit_vr + tok, true);
                        } else if (it + jn < seg_info[1]) {
                            issue_tile(it + jn);
                        }
                    }
                }
            };
            // O[head][channel] into the warp's float scratch: column g plus (G <= 4) its remainder column g + 4, held by the
            // lane two over.  Rows gid / gid + 8 of an m-tile are channels gid and gid + 8, or (8-bit tiles) 2 gid and
            // 2 gid + 1, whose code sums are still to be multiplied by the channel's V scale.
            auto store_o = [&](bool f8_layout, bool accumulate, float f0, float f1) {
#pragma unroll
                for (int jm = 0; jm < 8; ++jm) {
                    float v[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        v[i] = oacc[jm][i];
                        if (split) v[i] += __shfl_xor_sync(0xFFFFFFFFu, v[i], 2);
                    }
                    if (!split || tig < 2) {
                        const int ch_a = f8_layout ? 16 * jm + 2 * gid : 16 * jm + gid, ch_b = f8_layout ? ch_a + 1 : ch_a + 8;
                        const float sa = f8_layout ? ud.v_scale[ch_a] : 1.f, sb = f8_layout ? ud.v_scale[ch_b] : 1.f;
                        float* p0 = scratch_f + 2 * tig * 128;
                        float* p1 = p0 + 128;
                        if (accumulate) {
                            p0[ch_a] += v[0] * sa * f0; p1[ch_a] += v[1] * sa * f1; p0[ch_b] += v[2] * sb * f0; p1[ch_b] += v[3] * sb * f1;
                        } else {
                            p0[ch_a] = v[0] * sa; p1[ch_a] = v[1] * sa; p0[ch_b] = v[2] * sb; p1[ch_b] = v[3] * sb;
                        }
                    }
                }
            };
            // (the tile body lives in decode_fast_tile.inc so that it can be instantiated per tile kind without a lambda:
            // as a generic lambda it cost the bf16 kernel 6 %)
#define FDKV_TAIL_TILE false
            for (int j = 0; j < (F8 ? npre : nseg); ++j)
#include "decode_fast_tile.inc"
#undef FDKV_TAIL_TILE
            if constexpr (F8) {
#define FDKV_TAIL_TILE true
                for (int j = npre; j < nseg; ++j)
#include "decode_fast_tile.inc"
#undef FDKV_TAIL_TILE
            }
            it += nseg;

            // ---- merge the eight warps' states into this segment's split-K partial ----
            {
                float lq[2] = {l_run[0], l_run[1]};
#pragma unroll
                for (int o = 4; o < 32; o <<= 1) {
                    lq[0] += __shfl_xor_sync(0xFFFFFFFFu, lq[0], o);
                    lq[1] += __shfl_xor_sync(0xFFFFFFFFu, lq[1], o);
                }
                if (F8 && stashed) {
                    // join the stashed state of the 8-bit tiles (already in the scratch) with the tails' state
                    float f_st[2], f_tl[2];
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const float M = fmaxf(m_st[e], m_run[e]);
                        f_st[e] = m_st[e] == -INFINITY ? 0.f : ex2(m_st[e] - M);
                        f_tl[e] = m_run[e] == -INFINITY ? 0.f : ex2(m_run[e] - M);
                        lq[e] = l_st[e] * f_st[e] + lq[e] * f_tl[e];
                        m_run[e] = M;
                    }
                    if (!split || tig < 2) {  // the positions this lane wrote at the stash
#pragma unroll
                        for (int jm = 0; jm < 8; ++jm) {
                            float* p0 = scratch_f + 2 * tig * 128 + 16 * jm + 2 * gid;
                            p0[0] *= f_st[0]; p0[1] *= f_st[0]; p0[128] *= f_st[1]; p0[129] *= f_st[1];
                        }
                    }
                    __syncwarp();
                    store_o(false, true, f_tl[0], f_tl[1]);
                } else {
                    if constexpr (F8) {
                        store_o(true, false, 1.f, 1.f);
                    } else {
#pragma unroll
                        for (int jm = 0; jm < 8; ++jm) {
                            float v[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                v[i] = oacc[jm][i];
                                if (split) v[i] += __shfl_xor_sync(0xFFFFFFFFu, v[i], 2);
                            }
                            if (!split || tig < 2) {
                                const int ch = 16 * jm + gid, col = 2 * tig;
                                scratch_f[col * 128 + ch] = v[0];
                                scratch_f[(col + 1) * 128 + ch] = v[1];
                                scratch_f[col * 128 + ch + 8] = v[2];
                                scratch_f[(col + 1) * 128 + ch + 8] = v[3];
                            }
                        }
                    }
                }
                if (gid == 0) {
#pragma unroll
                    for (int e = 0; e < 2; ++e) { sm_m[warp * 8 + 2 * tig + e] = m_run[e]; sm_l[warp * 8 + 2 * tig + e] = lq[e]; }
                }
                __syncthreads();
                for (int i = threadIdx.x; i < a.G * 128; i += kThreads) {
                    const int g = i >> 7, ch = i & 127;
                    float M = -INFINITY;
#pragma unroll
                    for (int w = 0; w < kCW; ++w) M = fmaxf(M, sm_m[w * 8 + g]);
                    float L = 0.f, A = 0.f;
                    if (M != -INFINITY) {
#pragma unroll
                        for (int w = 0; w < kCW; ++w) {
                            const float f = ex2(sm_m[w * 8 + g] - M);
                            L = fmaf(sm_l[w * 8 + g], f, L);
                            const float* ow = reinterpret_cast<const float*>(smem_raw + kHeaderBytes + kStages * kStageBytes + w * kScratchBytes);
                            A = fmaf(ow[g * 128 + ch], f, A);
                        }
                    }
                    float* part = a.partials + (((int64_t)b * a.Hq + h * a.G + g) * kMaxSplits + slot) * kPartStride;
                    if (ch == 0) { part[0] = M * 0.6931471805599453f; part[1] = L; }  // the combine step works in natural-log units
                    part[4 + ch] = A;
                }
                // ---- split-K combine by whichever CTA finishes this unit last (atomic ticket, nobody waits) ----
                // The block barrier orders every thread's part stores before thread 0's fence, which is cumulative: the
                // ticket increment publishes the whole part at device scope; the last CTA's reads go to L2 (ld.cg).
                __syncthreads();
                int* const s_ticket = reinterpret_cast<int*>(smem_raw + kOffTicket);
                if (threadIdx.x == 0) {
                    int t;  // one release+acquire read-modify-write instead of fence, atomic, fence
                    asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(t) : "l"(a.counters + u) : "memory");
                    *s_ticket = t;
                }
                __syncthreads();
                const int nparts = pc.n[u];
                if (*s_ticket == nparts - 1) {
                    // Warp w takes head w % G and every (8/G)-th part of it, 4 channels per lane; the scratch area
                    // holds the per-warp sums, the header the per-warp denominators.
                    float* const red = reinterpret_cast<float*>(smem_raw + kHeaderBytes + kStages * kStageBytes);  // [8][128]
                    {
                        const int g = warp % a.G, pgi = warp / a.G, npg = kCW / a.G;
                        const float* pp = a.partials + ((int64_t)b * a.Hq + h * a.G + g) * kMaxSplits * kPartStride;
                        float mreg[kMaxSplits / 32], lreg[kMaxSplits / 32];
                        float mx = -INFINITY;
#pragma unroll
                        for (int i = 0; i < kMaxSplits / 32; ++i) {
                            const int sp = lane + 32 * i;
                            mreg[i] = sp < nparts ? __ldcg(pp + sp * kPartStride) : -INFINITY;
                            lreg[i] = sp < nparts ? __ldcg(pp + sp * kPartStride + 1) : 0.f;
                        }
#pragma unroll
                        for (int i = 0; i < kMaxSplits / 32; ++i) mx = fmaxf(mx, mreg[i]);
#pragma unroll
                        for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
                        float ls = 0.f;
#pragma unroll
                        for (int i = 0; i < kMaxSplits / 32; ++i) {
                            mreg[i] = mreg[i] == -INFINITY ? 0.f : __expf(mreg[i] - mx);  // now the part's weight
                            ls = fmaf(lreg[i], mreg[i], ls);
                        }
#pragma unroll
                        for (int o = 16; o; o >>= 1) ls += __shfl_xor_sync(0xFFFFFFFFu, ls, o);
                        // part weights to shared memory (one row per warp, after the eight 128-float sums), then the
                        // accumulator rows in batches of eight independent loads
                        float* const wts = red + kCW * 128 + warp * kMaxSplits;
#pragma unroll
                        for (int i = 0; i < kMaxSplits / 32; ++i) wts[lane + 32 * i] = mreg[i];
                        __syncwarp();
                        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                        for (int base = pgi; base < nparts; base += 8 * npg) {
                            float4 v[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const int sp = base + j * npg;
                                if (sp < nparts) v[j] = __ldcg(reinterpret_cast<const float4*>(pp + sp * kPartStride + 4) + lane);
                            }
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const int sp = base + j * npg;
                                if (sp < nparts) {
                                    const float f = wts[sp];
                                    acc.x = fmaf(v[j].x, f, acc.x); acc.y = fmaf(v[j].y, f, acc.y);
                                    acc.z = fmaf(v[j].z, f, acc.z); acc.w = fmaf(v[j].w, f, acc.w);
                                }
                            }
                        }
                        reinterpret_cast<float4*>(red + warp * 128)[lane] = acc;
                        if (lane == 0) sm_l[warp] = ls;
                    }
                    __syncthreads();
                    for (int i = threadIdx.x; i < a.G * 128; i += kThreads) {
                        const int g = i >> 7, ch = i & 127;
                        float A = 0.f;
                        for (int w = g; w < kCW; w += a.G) A += red[w * 128 + ch];
                        const float L = sm_l[g];
                        const float r = L > 0.f ? A / L : 0.f;
                        const int64_t o = ((int64_t)b * a.Hq + h * a.G + g) * 128 + ch;
                        if (a.out_dtype == FDKV_BF16)
                            reinterpret_cast<__nv_bfloat16*>(a.out)[o] = __float2bfloat16_rn(r);
                        else
                            reinterpret_cast<float*>(a.out)[o] = r;
                    }
                    if (threadIdx.x == 0) a.counters[u] = 0;  // ready for the next launch
                    __syncthreads();
                }
                zero_scratch();
                __syncthreads();
            }
        }
    }
    // after a timed-out wait: give copies that may still be in flight time to land before the CTA retires
    if (*abort_flag)
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
}

}  // namespace

bool make_rows_tensor_map(void* base, size_t bytes, int box_rows, void* tmap_out) {
    typedef CUresult (*encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess) {
        cudaGetLastError();
        return false;
    }
    const cuuint64_t rows = bytes / 256;
    if (rows == 0 || rows > 0x7FFFFFFFull || box_rows < 1 || box_rows > 256) return false;
    const cuuint64_t gdim[2] = {128, rows};
    const cuuint64_t gstride[1] = {256};
    const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};  // 64 channels x box_rows tokens
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = reinterpret_cast<encode_fn>(fn)(reinterpret_cast<CUtensorMap*>(tmap_out), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base,
                                                 gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// The same region viewed as rows of 128 bytes (8-bit row streams): one 128-byte x box_rows box per copy, 128-byte swizzle.
bool make_rows_tensor_map_u8(void* base, size_t bytes, int box_rows, void* tmap_out) {
    typedef CUresult (*encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess) {
        cudaGetLastError();
        return false;
    }
    const cuuint64_t rows = bytes / 128;
    if (rows == 0 || rows > 0x7FFFFFFFull || box_rows < 1 || box_rows > 256) return false;
    const cuuint64_t gdim[2] = {128, rows};
    const cuuint64_t gstride[1] = {128};
    const cuuint32_t box[2] = {128, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = reinterpret_cast<encode_fn>(fn)(reinterpret_cast<CUtensorMap*>(tmap_out), CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, base, gdim,
                                                 gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool make_arena_tensor_map(void* arena, size_t arena_bytes, void* tmap_out) {
    return make_rows_tensor_map(arena, arena_bytes, kTT, tmap_out);
}

// Host side of a launch: the cost-weighted cut of the batch's (unit, 16-token slice) list into one range per CTA and the
// split-K part count of every unit.  Uses only the host views in `a` (lengths, modes, shape); no device access.
static cudaError_t plan_decode_schedule(const DecodeArgs& a, int units, int sm_count, FastSched& sch, PartCount& cs) {
    // ---- cost-weighted schedule: whole CTAs per unit when there are enough CTAs, else a flat cut of the (unit, tile) list ----
    std::vector<int64_t> wp(units + 1, 0);
    // ranges are cut on 16-token slices (the granularity of the residual lists), so that the CTAs of a unit differ by
    // at most one slice; each range is streamed as 128-token tiles from its first slice, the last one partial
    std::vector<int> nt(units), ns(units), es(units), wt(units);  // 128-token tiles, 16-token slices, slices + tail, cost per tile
    int64_t total_tiles = 0;
    for (int u = 0; u < units; ++u) {
        const int T = a.host_T[u / a.Hkv];
        nt[u] = (T + kTT - 1) / kTT;
        ns[u] = (T + kResTile - 1) / kResTile;
        if (ns[u] >= (1 << 20)) return cudaErrorInvalidValue;  // cannot happen: T * 128 < 2^31
        total_tiles += nt[u];
    }
    // cost per tile: bytes in units of 512 B (the K and V boxes, plus the lists' share for residual units), residual
    // tiles scaled by the measured ratio of their compute time to a plain tile's (rc)
    // With whole CTAs per unit (latency-bound regime) a residual tile of the entry form costs a fixed part (the scratch
    // tile and the second products) plus a part per list entry: measured 2.0 plain tiles at 1024 entries per tile and
    // tensor (keep 1/16), 1.65 at 512 (keep 1/32); with 8-bit rows (a dearer plain tile) about 1.7 at either density.
    const double res_a = a.rows_f8 ? 1.55 : 1.25;
    const double res_b = a.rows_f8 ? 0.15 : 0.87;
    auto weigh = [&](double rc) {
        for (int u = 0; u < units; ++u) {
            const int T = a.host_T[u / a.Hkv];
            const int64_t k = (int64_t)T * 128 * a.keep_num / a.keep_den;
            wt[u] = 2 * kTT * 256 / 512;
            if (a.host_modes[u] == FDKV_MODE_RESIDUAL) {
                const int64_t res_bytes = a.tok_rule ? 2 * ((int64_t)T * a.keep_num / a.keep_den) * 260 : 2 * k * 4;  // rows + index, or packed entries
                if (rc == 0.0) wt[u] = (int)(wt[u] * (res_a + res_b * (double)k / nt[u] / 1024.0));
                else wt[u] = (int)((wt[u] + (res_bytes / nt[u] + 511) / 512) * rc);
                wt[u] = std::max(1, wt[u]);
            }
            // the CTA that ends a unit also streams its tail of generated tokens (whole plain tiles): counted as slices
            // of the unit's kind behind the unit's own, so that this CTA gets correspondingly fewer of those
            const int tail = a.host_tail ? std::min(a.host_tail[u / a.Hkv], a.max_tail) : 0;
            // Measured: the CTA that ends a unit runs behind its siblings at equal shares (with tails it also reads their
            // lengths behind the dependency wait); charging it eight plain tiles' worth of slices (in eighths of a tile
            // below) is the optimum of a sweep at 32k, with and without tails (+1.6 % / +6 %), and neutral at 128k.
            constexpr int kEndExtra = 64;  // (eighths of a plain tile)
            es[u] = ns[u] + ((tail + kTT - 1) / kTT * (kTT / kResTile) + kEndExtra) * (2 * kTT * 256 / 512) / std::max(1, wt[u]);
            wp[u + 1] = wp[u] + (int64_t)es[u] * wt[u];  // (in eighths of the tile cost)
        }
    };
    // (measured best: 1.7 when every unit gets whole CTAs, 1.5 in the flat cut of a batch)
    weigh(a.tok_rule ? 1.7 : 0.0);
    const int ncta = (int)std::min<int64_t>(std::min(std::min(sm_count, kMaxCtas), kMaxSplits), total_tiles);
    sch.ncta = ncta;
    sch.any_tail = a.any_tail;
    sch.units = units;
    bool whole = units <= ncta;
    std::vector<int> nc(units, 1);
    if (whole) {
        // Whole CTAs per unit (no CTA pays a second merge + ticket): shares proportional to the unit's cost, at least
        // one each, the remainder to the units with the largest cost per CTA; never more CTAs than tiles.
        int given = units;
        for (int u = 0; u < units; ++u) {
            const int extra = std::min<int64_t>((int64_t)nt[u] - 1, (int64_t)((double)(ncta - units) * (double)(wp[u + 1] - wp[u]) / (double)wp[units]));
            nc[u] += std::max(0, extra);
            given += std::max(0, extra);
        }
        while (given < ncta) {
            int best = -1;
            double best_load = 0.0;
            for (int u = 0; u < units; ++u) {
                const double load = (double)(wp[u + 1] - wp[u]) / nc[u];
                if (nc[u] < nt[u] && load > best_load) { best_load = load; best = u; }
            }
            if (best < 0) break;
            ++nc[best];
            ++given;
        }
        if (given != ncta) whole = false;
        // with few CTAs per unit the integer shares are too uneven (2 vs 3 CTAs is +50 %): cut the flat list instead
        double worst = 0.0;
        for (int u = 0; u < units; ++u) worst = std::max(worst, (double)(wp[u + 1] - wp[u]) / nc[u]);
        if (worst > 1.06 * (double)wp[units] / ncta) whole = false;
    }
    if (whole) {
        int c = 0;
        for (int u = 0; u < units; ++u)
            for (int j = 0; j < nc[u]; ++j) sch.start[c++] = ((uint32_t)u << 20) | (uint32_t)std::min<int64_t>(ns[u] - 1, (int64_t)es[u] * j / nc[u]);
        sch.start[ncta] = (uint32_t)units << 20;
    } else {
        weigh(1.5);
        int u = 0;
        for (int c = 0; c < ncta; ++c) {
            const int64_t target = wp[units] * c / ncta;
            while (u + 1 < units && wp[u + 1] <= target) ++u;
            const int slice = (int)std::min<int64_t>(ns[u], (target - wp[u]) / wt[u]);
            sch.start[c] = ((uint32_t)u << 20) | (uint32_t)slice;
        }
        sch.start[ncta] = (uint32_t)units << 20;
        // A CTA's segment table holds kMaxSeg units: where the cost cut gives one CTA a longer run of very short units
        // (a batch of one long and many one-token sequences), move whole units to its neighbours: first towards the
        // front, then towards the back.  Ranges stay ordered; a CTA may end up without work.
        auto nseg = [&](uint32_t s0, uint32_t s1) {
            const int ua = (int)(s0 >> 20), ta = (int)(s0 & 0xFFFFFu), ub = (int)(s1 >> 20), tb = (int)(s1 & 0xFFFFFu);
            int n = 0;
            for (int u2 = ua; u2 <= ub && u2 < units; ++u2)
                if ((u2 == ub ? tb : ns[u2]) > (u2 == ua ? ta : 0)) ++n;
            return n;
        };
        for (int c = ncta - 1; c >= 1; --c)
            while (nseg(sch.start[c], sch.start[c + 1]) > kMaxSeg) sch.start[c] = ((sch.start[c] >> 20) + 1) << 20;
        for (int c = 0; c + 1 < ncta; ++c)
            while (nseg(sch.start[c], sch.start[c + 1]) > kMaxSeg)
                sch.start[c + 1] = (sch.start[c + 1] & 0xFFFFFu) ? (sch.start[c + 1] >> 20) << 20 : ((sch.start[c + 1] >> 20) - 1) << 20;
    }
    // parts per unit = CTAs whose range contains at least one of its tiles
    for (int u = 0; u < kMaxUnits; ++u) cs.n[u] = 0;
    for (int c = 0; c < ncta; ++c) {
        const int ua = (int)(sch.start[c] >> 20), ta = (int)(sch.start[c] & 0xFFFFFu);
        const int ub = (int)(sch.start[c + 1] >> 20), tb = (int)(sch.start[c + 1] & 0xFFFFFu);
        int nseg_cta = 0;
        for (int u = ua; u <= ub && u < units; ++u) {
            const int b0 = u == ua ? ta : 0, b1 = u == ub ? tb : ns[u];
            if (b1 > b0) ++nseg_cta;
            if (b1 > b0 && cs.n[u] < 255) cs.n[u]++;
        }
        if (nseg_cta > kMaxSeg) return cudaErrorInvalidValue;  // only when units > kMaxSeg * CTAs (see the pass above)
    }
    for (int u = 0; u < units; ++u)
        if (cs.n[u] > kMaxSplits) return cudaErrorInvalidValue;  // cannot happen: ncta <= kMaxSplits
    return cudaSuccess;
}

// The plan alone, for a given number of CTAs (fdkv_plan_decode: host only, no device is touched).
cudaError_t plan_decode_host(const DecodeArgs& a, int n_ctas, uint32_t* start_out, int32_t* ncta_out, int32_t* parts_out) {
    const int units = a.batch * a.Hkv;
    if (units < 1 || units > kMaxUnits || n_ctas < 1) return cudaErrorInvalidValue;
    FastSched sch;
    PartCount cs;
    const cudaError_t e = plan_decode_schedule(a, units, n_ctas, sch, cs);
    if (e != cudaSuccess) return e;
    for (int c = 0; c <= sch.ncta; ++c) start_out[c] = sch.start[c];
    for (int u = 0; u < units; ++u) parts_out[u] = cs.n[u];
    *ncta_out = sch.ncta;
    return cudaSuccess;
}

cudaError_t launch_decode_fast(const DecodeArgs& a, cudaStream_t st, bool* handled) {
    *handled = false;
    const int units = a.batch * a.Hkv;
    if (!a.tmap || !a.packed_lists || a.d != 128 || units > kMaxUnits || units < 1) return cudaSuccess;
    if (a.rows_f8 && !a.tmap_u8) return cudaSuccess;
    static PerDevice once;
    int sm_count = 0;
    cudaError_t e0 = once.ensure([&]() {
        cudaError_t e = cudaFuncSetAttribute(decode_fast_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        return cudaFuncSetAttribute(decode_fast_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    }, &sm_count);
    if (e0 != cudaSuccess) return e0;
    FastSched sch;
    PartCount cs;
    {
        const cudaError_t pe = plan_decode_schedule(a, units, sm_count, sch, cs);
        if (pe != cudaSuccess) return pe;
    }
    const int ncta = sch.ncta;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ncta);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const CUtensorMap& m16 = *reinterpret_cast<const CUtensorMap*>(a.tmap);
    const CUtensorMap& m8 = *reinterpret_cast<const CUtensorMap*>(a.rows_f8 ? a.tmap_u8 : a.tmap);
    TailLens tl;
    for (int b = 0; b < a.batch; ++b) tl.n[b] = a.host_tail ? a.host_tail[b] : 0;
    cudaError_t e = a.rows_f8 ? cudaLaunchKernelEx(&cfg, decode_fast_kernel<true>, m16, m8, a, sch, cs, tl)
                              : cudaLaunchKernelEx(&cfg, decode_fast_kernel<false>, m16, m8, a, sch, cs, tl);
    if (e != cudaSuccess) return e;
    count_launch(1);
    count_kernel(FDKV_KERNEL_DECODE_FAST);
    *handled = true;
    return cudaGetLastError();
}

}  // namespace fdkv
