// Index-ordered compaction of the sparse residual (Eq. 3, entry form), as one pass over the keys (Z1 in the storage
// type, or the float32 energies of four-layer blocks).
//
// Persistent thread blocks take 32 KiB chunks of the unit-tensors in ticket order (a global counter, so every chunk
// with a lower ticket has been started by a block that is resident: the look-back below cannot wait on work that
// has no SM).  Six blocks share an SM: while one waits for its copy or at a barrier, the others compute, which
// measured faster than three blocks that each prefetch their next chunk into a second buffer.  Tickets run over
// the unit-tensors first (ticket t = chunk t / n of unit-tensor t % n): the blocks that are resident at one time
// then work on different unit-tensors, and a look-back finds a finished record a few chunks back instead of
// walking through hundreds of chunks that are all in flight.  A chunk is copied into shared memory by one bulk TMA
// copy (mbarrier transaction count).  Per chunk:
//   A  every thread compares its 16-byte vectors with the threshold (bf16: on 16-bit pairs inside 32-bit registers) and
//      writes one keep byte and one tie byte per eight elements into two bit maps; K tensors also get their copy with
//      the kept coefficients zeroed (the second operand of the probe);
//   B  one prefix sum over the word counts of both maps; the chunk's counts (keys above / equal to the threshold) are
//      published, and the counts of all earlier chunks of the unit-tensor are summed by a decoupled look-back over
//      the published records;
//   C  ties are kept in index order while fewer than `need` precede them: with the counts before the chunk and the
//      prefix inside it every word knows which of its ties are kept and where its entries go in the list;
//   D  every 16-token tile gets its offset in the list;
//   E  entry-parallel write: thread r of the chunk's list finds its word by binary search in the prefix, its bit by
//      a population-count descent, and stores index, value and packed entry -- consecutive threads, consecutive
//      list positions, whatever the distribution of the kept entries over tokens and channels.
// A bf16 key is the 15 magnitude bits, so `key > tau` for both halves of a word is one masked add: with
// a = w & 0x7FFF7FFF, bit 15 (31) of a + (0x7FFF - tau16) * 0x10001 is set exactly when the low (high) half exceeds
// tau16, and with 0x8000 - tau16 when it reaches it (no carry crosses the halves: every half sum stays below 2^16).
#include <algorithm>

#include "fdkv_internal.h"
#include "mbar_wait.cuh"

namespace fdkv {

namespace {

constexpr int kChunkBytes = 32768;              // a chunk: 16 384 bf16 or 8 192 float32 keys
constexpr int kMaxChunkWords = kChunkBytes / 2 / 32;  // words of a chunk's bit map (bf16)
constexpr int kFusedThreads = 256;
constexpr uint32_t kSpinCap = 1u << 22;         // polls of a look-back before it gives up

// shared memory (bytes)
constexpr int oBuf = 0;                               // the chunk
constexpr int oKeep = kChunkBytes;                    // keep map
constexpr int oTie = oKeep + kMaxChunkWords * 4;      // tie map; from step C on the list position of every word's first entry
constexpr int oPre = oTie;                            // (a thread holds its tie words in registers before it writes their positions)
constexpr int oWarp = oPre + (kMaxChunkWords + 8) * 4;  // per-warp sums
constexpr int oMisc = oWarp + 128;                    // ticket, (unused), before_gt, before_eq, abort flag
constexpr int oBar = oMisc + 64;                      // the copy's mbarrier
constexpr int kFusedSmem = oBar + 16;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint32_t pair_mask8(uint32_t g0, uint32_t g1, uint32_t g2, uint32_t g3) {
    // bit 15 / 31 of word j -> bit 2j / 16 + 2j, then the upper set folded down by 15: elements 0..7 in order
    uint32_t t = (g0 >> 15) & 0x00010001u;
    t |= (g1 >> 13) & 0x00040004u;
    t |= (g2 >> 11) & 0x00100010u;
    t |= (g3 >> 9) & 0x00400040u;
    return (t | (t >> 15)) & 0xFFu;
}

// position of the k-th (from zero) set bit of x; x has more than k set bits
__device__ __forceinline__ int kth_set_bit(uint32_t x, uint32_t k) {
    int pos = 0;
#pragma unroll
    for (int width = 16; width >= 1; width >>= 1) {
        const uint32_t c = __popc(x & ((1u << width) - 1u));
        if (k >= c) {
            k -= c;
            pos += width;
            x >>= width;
        }
    }
    return pos;
}

// Exclusive prefix over the block's threads of `mine` (the count of the thread's words of a bit map).  Returns the
// thread's exclusive prefix and the total; `warp_sums` is a scratch array of one entry per warp.
__device__ __forceinline__ uint32_t block_prefix(uint32_t mine, uint32_t* warp_sums, uint32_t& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t incl = mine;
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, s);
        if (lane >= s) incl += t;
    }
    __syncthreads();  // (the scratch array may still be read from the previous use)
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    uint32_t before = 0, all = 0;
#pragma unroll
    for (int w = 0; w < kFusedThreads / 32; ++w) {
        const uint32_t s = warp_sums[w];
        if (w < warp) before += s;
        all += s;
    }
    total = all;
    return before + incl - mine;
}

template <typename T>
__global__ void __launch_bounds__(kFusedThreads) select_fused_kernel(SelectArgs a, int chunks_per_ut, int nchunks, uint32_t* ticket,
                                                                     unsigned long long* records) {
    constexpr bool BF = sizeof(T) == 2;
    constexpr int kChunkElems = kChunkBytes / (int)sizeof(T);
    constexpr int kChunkWords = kChunkElems / 32;
    constexpr int kWordsPerThread = kChunkWords / kFusedThreads;  // 2 (bf16) or 1 (float32) consecutive words of a bit map
    extern __shared__ __align__(128) uint8_t smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t* const keep_map = reinterpret_cast<uint32_t*>(smem + oKeep);
    uint32_t* const tie_map = reinterpret_cast<uint32_t*>(smem + oTie);
    uint32_t* const pre = reinterpret_cast<uint32_t*>(smem + oPre);
    uint32_t* const warp_sums = reinterpret_cast<uint32_t*>(smem + oWarp);
    volatile uint32_t* const misc = reinterpret_cast<volatile uint32_t*>(smem + oMisc);
    volatile uint32_t* const abort_flag = misc + 4;
    const uint32_t bar0 = smem_u32(smem + oBar);

    // one thread takes a ticket and starts the copy of that chunk
    auto fetch = [&]() {
        const uint32_t t = atomicAdd(ticket, 1u);
        misc[0] = t;
        if (t < (uint32_t)nchunks) {
            const int ut = a.ut_begin + (int)(t % (uint32_t)a.ut_count), ck = (int)(t / (uint32_t)a.ut_count);
            const int64_t e0 = (int64_t)ck * kChunkElems;
            const uint32_t bytes = (uint32_t)min((int64_t)kChunkElems, (int64_t)a.T * a.d - e0) * (uint32_t)sizeof(T);
            const T* src = reinterpret_cast<const T*>(a.z1) + (int64_t)ut * a.unit_stride + e0;
            const uint32_t bar = bar0, dst = smem_u32(smem + oBuf);
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                         "l"(src), "r"(bytes), "r"(bar)
                         : "memory");
        }
    };
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar0));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        *abort_flag = 0;
        fetch();
    }
    __syncthreads();

    for (uint32_t it = 0;; ++it) {
        const uint32_t tk = misc[0];
        if (tk >= (uint32_t)nchunks) break;
        const int ut = a.ut_begin + (int)(tk % (uint32_t)a.ut_count), ck = (int)(tk / (uint32_t)a.ut_count);
        const uint32_t tau = a.sel[ut].tau, need = a.sel[ut].need;
        const int64_t e0 = (int64_t)ck * kChunkElems;
        const int n_e = (int)min((int64_t)kChunkElems, (int64_t)a.T * a.d - e0);  // a multiple of 8
        const uint8_t* const buf = smem + oBuf;
        // (only bf16 storage has the copy without the kept entries: it is the tensor-core probe's operand)
        __nv_bfloat16* const drop = (BF && a.z1drop && !(ut & 1))
                                        ? reinterpret_cast<__nv_bfloat16*>(a.z1drop) + (int64_t)(ut >> 1) * a.unit_stride + e0
                                        : nullptr;
        // a threshold above every key (nothing kept) has no 16-bit form: both addends zero leave bit 15 of every half clear
        const bool none = tau == 0xFFFFFFFFu;
        const uint32_t add_gt = none ? 0u : (0x7FFFu - (tau >> 16)) * 0x00010001u;
        const uint32_t add_ge = none ? 0u : (0x8000u - (tau >> 16)) * 0x00010001u;

        mbar_wait_bounded(bar0, it & 1u, abort_flag, a.status);

        // ---- A: keep and tie bytes, the dropped-coefficient copy ----
#pragma unroll 4
        for (int q = 0; q < kChunkElems / 8 / kFusedThreads; ++q) {
            const int vi = q * kFusedThreads + tid;  // eight elements = one byte of the maps
            uint32_t m8 = 0, e8 = 0;
            if (vi * 8 < n_e) {
                if constexpr (BF) {
                    const uint4 v = *reinterpret_cast<const uint4*>(buf + vi * 16);
                    const uint32_t a0 = v.x & 0x7FFF7FFFu, a1 = v.y & 0x7FFF7FFFu, a2 = v.z & 0x7FFF7FFFu, a3 = v.w & 0x7FFF7FFFu;
                    const uint32_t g0 = a0 + add_gt, g1 = a1 + add_gt, g2 = a2 + add_gt, g3 = a3 + add_gt;
                    const uint32_t x0 = g0 ^ (a0 + add_ge), x1 = g1 ^ (a1 + add_ge), x2 = g2 ^ (a2 + add_ge), x3 = g3 ^ (a3 + add_ge);
                    m8 = pair_mask8(g0, g1, g2, g3);
                    if (((x0 | x1 | x2 | x3) & 0x80008000u) && !none) e8 = pair_mask8(x0, x1, x2, x3);
                    if (drop) {
                        // kept halves cleared: bit 15 / 31 of the compare sums widened to half masks (kept ties follow in C)
                        auto cleared = [](uint32_t wv, uint32_t g) { return wv & ~(((g >> 15) & 0x00010001u) * 0xFFFFu); };
                        *reinterpret_cast<uint4*>(drop + vi * 8) = make_uint4(cleared(v.x, g0), cleared(v.y, g1), cleared(v.z, g2), cleared(v.w, g3));
                    }
                } else {
                    // float32 keys: the 31 magnitude bits (a threshold above every key compares false everywhere)
                    const uint4 lo = *reinterpret_cast<const uint4*>(buf + vi * 32), hi = *reinterpret_cast<const uint4*>(buf + vi * 32 + 16);
                    const uint32_t k8[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const uint32_t key = k8[i] & 0x7FFFFFFFu;
                        m8 |= (uint32_t)(key > tau) << i;
                        e8 |= (uint32_t)(key == tau) << i;
                    }
                }
            }
            reinterpret_cast<uint8_t*>(keep_map)[vi] = (uint8_t)m8;
            reinterpret_cast<uint8_t*>(tie_map)[vi] = (uint8_t)e8;
        }
        __syncthreads();
        // ---- B: word counts of both maps and their prefix over the chunk, one scan: keys above the threshold in the
        // low half of a word, keys equal to it in the high half (a chunk holds 2^14 elements) ----
        uint32_t kw[kWordsPerThread], tw[kWordsPerThread], mine = 0;
#pragma unroll
        for (int h = 0; h < kWordsPerThread; ++h) {
            kw[h] = keep_map[kWordsPerThread * tid + h];
            tw[h] = tie_map[kWordsPerThread * tid + h];
            mine += __popc(kw[h]) | (__popc(tw[h]) << 16);
        }
        uint32_t total;
        const uint32_t excl = block_prefix(mine, warp_sums, total);
        const uint32_t c_gt = total & 0xFFFFu, c_eq = total >> 16;
        // the chunk's record, and the sums over the unit-tensor's earlier chunks
        if (warp == 0) {
            // a record: state in the top two bits (1 = this chunk's counts, 2 = counts of this and all earlier chunks),
            // keys above the threshold in bits 31..61, keys equal to it in bits 0..30
            const unsigned long long own = ((unsigned long long)c_gt << 31) | c_eq;
            unsigned long long* const rec = records + (int64_t)(ut - a.ut_begin) * chunks_per_ut;
            unsigned long long before = 0;
            if (ck > 0) {
                if (lane == 0) atomicExch(rec + ck, own | (1ull << 62));
                int j = ck - 1;
                uint32_t spins = 0;
                while (j >= 0) {
                    const int at = j - lane;
                    unsigned long long r = at >= 0 ? *reinterpret_cast<volatile unsigned long long*>(rec + at) : (2ull << 62);
                    const uint32_t missing = __ballot_sync(0xFFFFFFFFu, (r >> 62) == 0ull);
                    if (missing) {
                        if (++spins > kSpinCap || *abort_flag) {  // bounded: give up, say so, finish with what there is
                            *abort_flag = 1;
                            if (lane == 0) atomicMax(a.status, (int32_t)kFlagTimeout);
                            break;
                        }
                        __nanosleep(20);
                        continue;
                    }
                    const uint32_t full = __ballot_sync(0xFFFFFFFFu, (r >> 62) == 2ull);  // lanes that end the walk
                    const int stop = full ? __ffs((int)full) - 1 : 32;
                    unsigned long long part = (lane <= stop && at >= 0) ? (r & ((1ull << 62) - 1ull)) : 0ull;
#pragma unroll
                    for (int s = 16; s; s >>= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, s);
                    before += part;
                    if (full) break;
                    j -= 32;
                }
            }
            if (lane == 0) {
                atomicExch(rec + ck, (before + own) | (2ull << 62));
                misc[2] = (uint32_t)(before >> 31);
                misc[3] = (uint32_t)(before & 0x7FFFFFFFull);
            }
        }
        __syncthreads();
        const uint32_t before_gt = misc[2], before_eq = misc[3];
        const uint32_t ties_before = min(before_eq, need);
        const uint32_t base = before_gt + ties_before;  // list position of the chunk's first kept entry
        const uint32_t n_keep = c_gt + min(before_eq + c_eq, need) - ties_before;
        // ---- C: ties are kept in index order while fewer than `need` precede them; every word's list position ----
        {
            uint32_t r_gt = excl & 0xFFFFu, r_eq = before_eq + (excl >> 16);  // keys above / ties before the thread's words
#pragma unroll
            for (int h = 0; h < kWordsPerThread; ++h) {
                const int w = kWordsPerThread * tid + h;
                pre[w] = r_gt + min(r_eq, need) - ties_before;
                const uint32_t c = __popc(tw[h]);
                if (c && r_eq < need) {
                    uint32_t sel = tw[h];
                    if (need - r_eq < c) sel = tw[h] & ((2u << kth_set_bit(tw[h], need - r_eq - 1)) - 1u);  // the lowest need - r_eq ties
                    keep_map[w] = kw[h] | sel;
                    if (drop)
                        for (uint32_t kk = sel; kk; kk &= kk - 1) drop[w * 32 + __ffs((int)kk) - 1] = __ushort_as_bfloat16((unsigned short)0);
                }
                r_gt += __popc(kw[h]);
                r_eq += c;
            }
        }
        __syncthreads();
        // ---- D: tile offsets ----
        const int tile_words = kResTile * a.d / 32;                    // bit-map words of a 16-token tile
        const int tiles_here = (n_e + kResTile * a.d - 1) / (kResTile * a.d);
        const int tile0 = (int)(e0 / (kResTile * a.d));
        int32_t* const off = a.tile_off + (int64_t)ut * (a.ntiles_max + 1);
        if (tid < tiles_here) off[tile0 + tid] = (int32_t)(base + pre[tid * tile_words]);
        if (tid == 0 && ck == chunks_per_ut - 1) {
            off[tile0 + tiles_here] = (int32_t)(base + n_keep);
            if ((int64_t)(base + n_keep) != a.k && !*abort_flag) atomicMax(a.status, (int32_t)kFlagCountMismatch);
        }
        // ---- E: entry-parallel write ----
        int32_t* const idx = a.idx + (int64_t)ut * a.kcap + base;
        T* const val = reinterpret_cast<T*>(a.val) + (int64_t)ut * a.kcap + base;
        uint32_t* const pk = (BF && a.packed) ? a.packed + (int64_t)ut * a.kcap + base : nullptr;
        for (uint32_t r = tid; r < n_keep; r += kFusedThreads) {
            // the last word whose prefix does not exceed r holds entry r (empty words share their successor's prefix)
            int w = 0;
#pragma unroll
            for (int s = kChunkWords / 2; s; s >>= 1)
                if (pre[w + s] <= r) w += s;
            const int flat = w * 32 + kth_set_bit(keep_map[w], r - pre[w]);
            const T v = reinterpret_cast<const T*>(buf)[flat];
            idx[r] = (int32_t)(e0 + flat);
            val[r] = v;
            if constexpr (BF) {
                if (pk) {
                    // (byte offset / 2) inside a 16-token x 128-channel tile of two 64-channel halves with 128-byte rows whose
                    // 16-byte chunks are XOR-swizzled with the row
                    const int row = (flat >> 7) & 15, ch = flat & 127;
                    const uint32_t o = (uint32_t)((ch >> 6) * 2048 + row * 128 + ((((ch >> 3) & 7) ^ (row & 7)) << 4) + (ch & 7) * 2);
                    pk[r] = (uint32_t)__bfloat16_as_ushort(v) | ((o >> 1) << 16);
                }
            }
        }
        __syncthreads();  // the buffer and the maps are free again: the next ticket and its copy
        if (tid == 0) fetch();
        __syncthreads();
    }
}

}  // namespace

cudaError_t launch_select_fused(const SelectArgs& a, int dtype, cudaStream_t st) {
    static PerDevice once;
    int sms = 0;
    cudaError_t e = once.ensure([&]() {
        cudaError_t e1 = cudaFuncSetAttribute(select_fused_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFusedSmem);
        if (e1 != cudaSuccess) return e1;
        return cudaFuncSetAttribute(select_fused_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFusedSmem);
    }, &sms);
    if (e != cudaSuccess) return e;
    const int64_t n = (int64_t)a.T * a.d;
    const int chunk_elems = kChunkBytes / (dtype == FDKV_BF16 ? 2 : 4);
    const int chunks_per_ut = (int)((n + chunk_elems - 1) / chunk_elems);
    const int64_t nchunks = (int64_t)chunks_per_ut * a.ut_count;
    if (nchunks <= 0) return cudaSuccess;
    // the look-back records (one 64-bit word per chunk; a chunk holds at least four 16-token tiles, the array one word
    // per tile) and the ticket counter start at zero
    unsigned long long* records = a.lb_records + (int64_t)a.ut_begin * a.ntiles_max;
    uint32_t* ticket = a.lb_ticket;
    if ((e = cudaMemsetAsync(records, 0, (size_t)nchunks * 8, st)) != cudaSuccess) return e;
    if ((e = cudaMemsetAsync(ticket, 0, 4, st)) != cudaSuccess) return e;
    const int grid = (int)std::min<int64_t>(nchunks, (int64_t)sms * 6);  // six blocks of 37 KiB per SM
    if (dtype == FDKV_BF16)
        select_fused_kernel<__nv_bfloat16><<<grid, kFusedThreads, kFusedSmem, st>>>(a, chunks_per_ut, (int)nchunks, ticket, records);
    else
        select_fused_kernel<float><<<grid, kFusedThreads, kFusedSmem, st>>>(a, chunks_per_ut, (int)nchunks, ticket, records);
    count_launch(1);
    return cudaGetLastError();
}

}  // namespace fdkv
