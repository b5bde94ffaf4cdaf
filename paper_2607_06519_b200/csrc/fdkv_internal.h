// Internal declarations shared by the translation units of libfdkv (not part of the public ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstddef>
#include <cstdint>
#include <mutex>
#include <vector>

#include "../../include/fdkv.h"

namespace fdkv {

constexpr int kResTile = 16;         // tokens per residual-offset tile: off[j] = first list entry of tokens >= 16 j
constexpr int kHistBins = 32768;     // one bin per 15-bit magnitude prefix (a whole bf16 key)
constexpr int kMaxSplits = 160;      // split-K partial slots per (sequence, query head)
constexpr int kMaxW = 128;           // probe queries
constexpr int kListPad = 32;         // slack entries after each residual list (aligned over-reads stay in bounds)
constexpr int kMaxGroup = 8;
constexpr int kProbeBoxRows = 256;   // key tokens per tile of the tensor-core probe (rows of its TMA boxes)
constexpr int kFastMaxUnits = 1024;   // (sequences x KV heads) one launch of the bf16 / head_dim 128 decode kernel plans for
constexpr int kProbeTile = 64;       // tokens per probe CTA (generic kernel)
constexpr int kRowPad = 128;         // packed row blocks and tails are padded (zero rows) to this many tokens

enum DeviceFlag : int32_t { kFlagOk = 0, kFlagTimeout = 1, kFlagCountMismatch = 2, kFlagTailFull = 3 };

// What decode reads for one (sequence, layer, KV head).
struct UnitDesc {
    const void* k_rows;  // [T][d]: Z0 of K (shared / residual) or the layer's original K rows (exact)
    const void* v_rows;
    // residual mode only.  Portable layout: ascending flat indices t*d + ch and the stored values.  Packed layout
    // (bf16, head_dim 128): k_idx holds one 32-bit word per entry, value bits in the low half and the entry's
    // position inside its 16-token slice (a ready-made shared-memory offset / 2) in the high half; k_val is null.
    const int32_t* k_idx;
    const void* k_val;
    const int32_t* k_off;  // [ceil(T/16) + 1] first entry of each 16-token tile
    const int32_t* v_idx;
    const void* v_val;
    const int32_t* v_off;
    int32_t mode;
    int32_t T;
    float sign;  // multiplier of the residual values relative to the rows: +1 / -1 for the two layers of a pair,
                 // 2 for a layer of a four-layer block (rows scaled by 1/2, deviations by 1)
    int32_t res_kind;  // residual layout: 0 packed entries (k_idx / v_idx), 1 token rows (k_idx = token list, k_val / v_val = rows, k_off = per-slice counts)
    float scale;       // what the stored rows are multiplied by: 1/sqrt 2 (pair coefficients), 1/2 (block of four), 1 (exact)
    int32_t rows_f8;   // 1: k_rows / v_rows hold e4m3 codes (128 bytes per token) with per-channel scales below
    const float* k_scale;  // [d] float32, rows_f8 only
    const float* v_scale;
};

struct SelState {
    uint32_t prefix;  // magnitude-key prefix fixed so far (left-aligned in 31 bits once complete)
    uint32_t k_rem;   // entries still to take at or below the prefix
    uint32_t tau;     // final threshold key (31-bit magnitude pattern; bf16 keys are shifted left by 16)
    uint32_t need;    // entries with key == tau to keep (lowest flat indices first)
};

struct Shape {
    int L, P, Hq, Hkv, G, d;
    int max_batch, Tmax, max_tail;
    int dtype, esize;
    int keep_num, keep_den;
    int64_t kmax;      // floor(Tmax*d*num/den)
    int64_t kcap;      // list capacity incl. slack
    int ntiles_max;    // ceil(Tmax/16)
    int nptiles_max;   // ceil(Tmax/kProbeTile)
    int NU, NT;        // units and unit-tensors (K and V) of one sequence
    int tail_rows;     // max_tail rounded up to kRowPad
    int tok_rule;      // 1: token-granular residual chosen by the probe
    int B;             // layers per depth block: 2 or 4
    int max_fold;      // generated tokens that may be folded into the compressed form per sequence
    int rows_f8;       // committed row streams are e4m3 codes with per-channel scales
    int64_t kfold_max; // floor(max_fold*d*num/den): list room reserved for them
    int NB;            // staged high-frequency tensors per unit-tensor: 1 (Z1 of a pair) or 4 (the layers' deviations)
    int64_t ktok_max, ktok_cap;  // floor(Tmax*num/den) and the list capacity incl. slack
};

struct WsLayout {
    size_t tok_score, tok_flag, tok_list, tok_off;
    size_t energy, eval;  // four-layer blocks: per-position high-frequency energy (float32) and the kept energies
    size_t status, z0, z1, z1drop, hist, sel, lb_records, lb_ticket, tile_off, idx, val, packed, probe_part, probe_pos, scores, modes,
        partials, counters, io_q, io_k, io_v, io_out, jobs, total;  // io_*: host-I/O staging, [L] layers each
};
struct ArenaLayout {
    size_t tail_len, desc, tail_k, tail_v, bump, worst_total;
};

struct SeqState {
    bool committed = false;
    int T = 0;
    std::vector<int32_t> modes;  // [NU], -1 unknown
    size_t bytes_by_mode[3] = {0, 0, 0};
    std::vector<int32_t> tail_len;  // host mirror per layer
    int fold_used = 0;              // tokens folded so far
    int64_t k_entries = 0;          // entries per residual list (prompt + folded chunks)
};

}  // namespace fdkv

struct fdkv_ctx {
    fdkv_config cfg;
    fdkv::Shape s;
    fdkv::WsLayout ws;
    fdkv::ArenaLayout ar;
    char* arena;
    size_t arena_bytes;
    char* work;
    size_t work_bytes;
    size_t bump;  // next free arena offset
    int staged_seq = -1;
    int staged_T = 0;
    std::vector<uint8_t> pair_compressed, pair_probed;
    std::vector<const void*> k_layers, v_layers;
    int64_t stride_t = 0, stride_h = 0;
    bool modes_overridden = false;
    std::vector<fdkv::SeqState> seqs;
    std::vector<fdkv::UnitDesc> desc_host;  // [max_batch][L][Hkv]
    alignas(64) unsigned char tmap[128];    // CUtensorMap of the arena (bf16, head_dim 128 only)
    bool has_tmap = false;
    alignas(64) unsigned char tmap_z1[128], tmap_drop[128];  // probe operands (bf16, head_dim 128 only)
    bool has_probe_tmaps = false;
    alignas(64) unsigned char tmap_z1_128[128];  // staged Z1 with 128-token boxes (token-score kernel)
    bool tok_tc = false;                         // token rule served by the tensor-core kernels (bf16, head_dim 128)
    std::vector<uint8_t> pair_scored;            // token rule: the probe has chosen this pair's token sets
    bool packed_lists = false;              // decode runs the bf16 / head_dim 128 kernel on packed residual entries
    alignas(64) unsigned char tmap_u8[128]; // CUtensorMap of the arena as 128-byte rows (8-bit row streams)
};

namespace fdkv {

// ---- launchers implemented in compress.cu / probe.cu / decode.cu; each returns cudaGetLastError() ----
constexpr int kSplitPairs = 32;  // layer pairs one launch of the split kernel covers
struct CompressArgs {
    // the four [T][Hkv][d] strided tensors (K and V of layers 2p, 2p+1) of each pair of the launch
    const void *k0[kSplitPairs], *k1[kSplitPairs], *v0[kSplitPairs], *v1[kSplitPairs];
    int n_pairs;
    int64_t stride_t, stride_h;
    int T, d, Hkv;
    int tensors;  // 2: K and V of every head (unit-tensor = head*2 + is_v); 1: K only (unit-tensor = head)
    int ut_base;  // first unit-tensor of the first pair in the stage; pair j adds j*Hkv*tensors
    int64_t unit_stride;  // elements between staged unit-tensors (Tmax*d)
    void *z0, *z1;
    uint32_t* hist;
};
cudaError_t launch_split_hist(const CompressArgs& a, int dtype, cudaStream_t st);

struct SelectArgs {
    int ut_begin, ut_count;
    int T, d;
    int64_t k;
    int64_t unit_stride, kcap;
    int ntiles_max;
    const void* z1;
    uint32_t* hist;
    SelState* sel;
    unsigned long long* lb_records;  // look-back records of the ordered select: one 64-bit word per (unit-tensor, chunk), ntiles_max per unit-tensor
    uint32_t* lb_ticket;             // its ticket counter (one word)
    int32_t* tile_off;
    int32_t* idx;
    void* val;
    void* z1drop;      // optional [unit][Tmax*d]: Z1 of K with the kept entries zeroed (tensor-core probe), or null
    uint32_t* packed;  // optional packed entries for the bf16 / head_dim 128 decode kernel (null otherwise)
    int32_t* status;
};
cudaError_t launch_select_and_compact(const SelectArgs& a, int dtype, cudaStream_t st);
// count, offsets and ordered write as one pass over the keys (select_fused.cu); a.sel holds the thresholds
cudaError_t launch_select_fused(const SelectArgs& a, int dtype, cudaStream_t st);

// ---- four-layer blocks (block4.cu) ----
struct Split4Args {
    const void* k[4];  // the block's four [T][Hkv][d] strided K tensors, layer order
    const void* v[4];
    int64_t stride_t, stride_h;
    int T, d, Hkv;
    int ut_base;          // first unit-tensor of the block (unit-tensor = head*2 + is_v)
    int64_t unit_stride;  // elements between staged tensors (Tmax*d)
    void* z0;             // [NT][unit_stride]
    void* dev;            // [NT][4][unit_stride]: deviation of each layer from the block mean
    float* energy;        // [NT][unit_stride]
    void* drop;           // optional [NU][4][unit_stride]: second copy of the K deviations (the gather zeroes its kept positions)
    uint32_t* hist;
};
cudaError_t launch_split4_hist(const Split4Args& a, int dtype, cudaStream_t st);
struct Gather4Args {
    int ut_begin, ut_count;
    int64_t k, kcap, unit_stride;
    const void* dev;     // [NT][4][unit_stride]
    const int32_t* idx;  // [NT][kcap] ascending kept positions
    void* val;           // [NT][4][kcap] the four layers' values at the kept positions
    uint32_t* packed;    // optional [NT][4][kcap] packed entries (value doubled: the rows are scaled by 1/2), or null
    void* drop;          // optional [NU][4][unit_stride]: the K deviations (copied there beforehand); kept positions get zeroed
};
cudaError_t launch_gather4(const Gather4Args& a, int dtype, cudaStream_t st);

struct ProbeArgs {
    int B;  // layers per block: 2 (one Z1 operand, both layers' queries) or 4 (one deviation operand per layer)
    int unit_begin, unit_count;  // units of the pair range (unit = pair*Hkv + h)
    int T, d, Hq, Hkv, G, W;
    int64_t unit_stride, kcap;
    int ntiles_max, nptiles_max;
    const void* z1;  // staged Z1 (unit-tensor ut = unit*2 for K)
    const int32_t* idx;
    const int32_t* tile_off;
    const uint8_t* tok_flag;          // token rule, float32 probe kernel: [NU][Tmax] flags of the selected tokens (else null)
    const void* const* q_layers_dev;  // device array [L] of pointers
    const int32_t* pos;
    double* part;    // [NU][nptiles_max][2]
    double* scores;  // [NU][2]
    int32_t* modes;  // [NU]
    double lambda, omega[3];
    int32_t* modes_out;  // user buffers for the pair range, may be null
    float* scores_out;
    // tensor-core path (bf16, head_dim 128): tensor maps over the staged Z1 and the dropped copy, viewed as
    // [rows][128] bf16 with 128-token x 64-channel boxes; null when unavailable
    const void *tmap_z1, *tmap_drop;
    int Tmax;
    const int32_t* pos_host;
    int32_t* status;
};
cudaError_t launch_probe(const ProbeArgs& a, int dtype, cudaStream_t st);

struct DecodeArgs {
    const UnitDesc* desc;  // [batch][.. layer ..] : desc + (b*L + layer)*Hkv + h
    int L, layer, batch, Hq, Hkv, G, d, max_tail, max_batch;
    int Tmax_batch;  // largest T among the batch (host side, sizes the grid)
    const void *q, *k_new, *v_new;
    void* out;
    int out_dtype;
    void *tail_k, *tail_v;  // [L][max_batch][Hkv][tail_rows][d], tail_rows = max_tail rounded up to kRowPad
    int tail_rows;
    // host-side views used only to plan the launch (valid during the call)
    const int32_t* host_T;      // [batch]
    const int32_t* host_modes;  // [batch][Hkv] modes of this layer's pair
    const int32_t* host_tail;   // [batch] generated tokens in this layer's tail per sequence (after this call's append), or null
    int any_tail;               // some sequence of the batch has generated tokens in this layer's tail (after this call's append)
    const void* tmap;           // CUtensorMap over the arena as rows of 256 bytes, or null
    const void* tmap_u8;        // the same arena as rows of 128 bytes (8-bit row streams), or null
    int rows_f8;
    const void* arena_base;
    int keep_num, keep_den;
    int packed_lists;
    int tok_rule;
    int32_t* tail_len;      // [L][max_batch]
    float* partials;        // [batch][Hq][kMaxSplits][d+4]: max, sum, 2 pad, d accumulators
    int32_t* counters;      // [max_batch][Hkv] split-K arrival tickets, zero between launches
    int32_t* status;
};
cudaError_t launch_decode(const DecodeArgs& a, int dtype, cudaStream_t st);
// Encodes a 2-D tensor map over the arena viewed as [rows][128] bf16 (256-byte rows), 64x64 boxes, 128-byte swizzle.
bool make_arena_tensor_map(void* arena, size_t arena_bytes, void* tmap_out);
// Same view ([rows][128] bf16, 64-channel x box_rows boxes, 128-byte swizzle) over any 256-byte aligned region.
bool make_rows_tensor_map(void* base, size_t bytes, int box_rows, void* tmap_out);
// ---- 8-bit row streams (rows_fp8.cu) ----
// One stored tensor: codes[t][c] = e4m3(src[t*stride_t + c] / scale[c]), scale[c] = max_t |src| / 448 (1 if zero); src bf16,
// d = 128; scale points at a 1 KiB slot whose second half holds the channel maxima while the job runs.
struct QuantJob {
    const void* src;
    int64_t stride_t;
    int32_t T, pad_;
    uint8_t* codes;
    float* scale;
};
// One residual list of a unit whose rows are 8-bit: value -> f16(value / scale[channel]), position permuted inside its
// 16-channel group to the order the kernel's converted fragments use (K and V differ).
// (rows = 1: dst == src are n densely packed 128-channel bf16 rows of the token rule, converted in place.)
struct RepackJob {
    uint32_t* dst;
    const uint32_t* src;
    int64_t n;
    const float* scale;
    int32_t is_v, rows;
};
// One copy of the commit step: dst[0, bytes) = consecutive rows of row_bytes taken every src_pitch bytes from src
// (row_bytes == src_pitch: a plain copy).  Pointers 16-byte aligned, row_bytes and src_pitch multiples of 16, bytes a
// multiple of 4.  All copies of a commit run as one launch over a job table.
struct CopyJob {
    const char* src;
    char* dst;
    int64_t bytes;
    int64_t src_pitch;
    int32_t row_bytes, pad_;
};
cudaError_t plan_decode_host(const DecodeArgs& a, int n_ctas, uint32_t* start_out, int32_t* ncta_out, int32_t* parts_out);
cudaError_t launch_copy_jobs(const CopyJob* jobs_dev, int njobs, int64_t bytes_max, cudaStream_t st);
cudaError_t launch_quantise_jobs(const QuantJob* jobs_dev, int njobs, int T_max, cudaStream_t st);
cudaError_t launch_repack_jobs(const RepackJob* jobs_dev, int njobs, int64_t n_max, cudaStream_t st);
bool make_rows_tensor_map_u8(void* base, size_t bytes, int box_rows, void* tmap_out);

// dst[i] = src[i] + add, i < n (list offsets and indices of a folded chunk)
cudaError_t launch_offset_copy(int32_t* dst, const int32_t* src, int n, int add, cudaStream_t st);
cudaError_t launch_strided_copy(const void* src, int64_t stride_t, void* dst, int T, int d, int esize, cudaStream_t st);

// ---- token-granular residual (token_rule.cu) ----
struct TokenArgs {
    int B;  // layers per depth block: 2 (one Z1 operand, both layers' queries) or 4 (one deviation operand per layer)
    int unit_begin, unit_count;
    int T, Tmax, Hq, Hkv, G, W, ntiles_max;
    int64_t k_tok, ktok_cap, unit_stride;
    const void* z1;                    // staged Z1 (K of unit u at unit-tensor 2u)
    void* z1drop;                      // [unit][Tmax*128] Z1 of K with the selected rows zeroed
    const void* const* q_layers_dev;
    const int32_t* pos;
    const int32_t* pos_host;
    uint32_t* score;                   // [unit][Tmax] float bits (non-negative)
    uint8_t* flag;                     // [unit][Tmax]
    int32_t* list;                     // [unit][ktok_cap]
    int32_t* off;                      // [unit][ntiles_max + 1]
    const void* tmap_z1_128;
    int32_t* status;
};
// tensor_core: bf16 / head_dim 128 contexts (tcgen05 score kernel + the dropped-row copy); otherwise the float32 score kernel
cudaError_t launch_token_select(const TokenArgs& a, int dtype, int d, bool tensor_core, cudaStream_t st);
cudaError_t launch_token_gather(const void* z1, const int32_t* list, int64_t k_tok, void* out, int row_bytes, int twice, cudaStream_t st);

// Function attributes (the opt-in to large dynamic shared memory) and the SM count belong to a device, not to the
// process: every launcher keeps one of these and runs its set-up the first time it meets the current device.
struct PerDevice {
    static constexpr int kMaxDevices = 64;
    std::mutex mu;
    bool done[kMaxDevices] = {};
    int sms[kMaxDevices] = {};
    // init() -> cudaError_t runs once per device (under the lock); *sm_count (optional) receives the device's SM count.
    template <typename F>
    cudaError_t ensure(F&& init, int* sm_count = nullptr) {
        int dev = -1;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
        std::lock_guard<std::mutex> lock(mu);
        if (!done[dev]) {
            e = cudaDeviceGetAttribute(&sms[dev], cudaDevAttrMultiProcessorCount, dev);
            if (e == cudaSuccess) e = init();
            if (e != cudaSuccess) return e;
            done[dev] = true;
        }
        if (sm_count) *sm_count = sms[dev];
        return cudaSuccess;
    }
};
// The bookkeeping of PerDevice::ensure without a device (host-side test hook): how many of the `n` device ids in `devs`
// would run their set-up, in order, on a fresh table.
int per_device_first_visits(const int* devs, int n);

void count_launch(int n);
void count_kernel(int id);  // id: fdkv_kernel_id
// Remembers a failed CUDA runtime call for fdkv_last_cuda_error() and returns FDKV_ERR_CUDA.
fdkv_status record_cuda_error(cudaError_t e);

}  // namespace fdkv
