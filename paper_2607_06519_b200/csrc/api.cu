// Host side of the C ABI: argument checks, workspace / arena bookkeeping, launch sequencing.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstring>
#include <new>

#include "fdkv_internal.h"

using namespace fdkv;

namespace {

std::atomic<int64_t> g_launches{0};
std::atomic<int64_t> g_kernel_launches[FDKV_KERNEL_COUNT_];
std::atomic<int32_t> g_last_cuda{0};

inline size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }
inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

fdkv_status cuda_fail(cudaError_t e) {
    g_last_cuda.store((int32_t)e);
    return FDKV_ERR_CUDA;
}
#define CU(x)                                         \
    do {                                              \
        cudaError_t e__ = (x);                        \
        if (e__ != cudaSuccess) return cuda_fail(e__); \
    } while (0)

bool make_shape(const fdkv_config& c, Shape& s) {
    const int B = c.block_size == 0 ? 2 : c.block_size;
    if (B != 2 && B != 4) return false;
    if (c.n_layers <= 0 || (c.n_layers % B) || c.n_layers > 1024) return false;
    if (c.n_kv_heads <= 0 || c.n_q_heads <= 0 || c.n_q_heads % c.n_kv_heads) return false;
    const int G = c.n_q_heads / c.n_kv_heads;
    if (!(G == 1 || G == 2 || G == 4 || G == 8)) return false;
    if (c.head_dim != 64 && c.head_dim != 128) return false;
    if (c.max_batch <= 0 || c.max_prefill <= 0 || c.max_tail < 0 || c.max_fold < 0) return false;
    if ((int64_t)(c.max_prefill + (int64_t)c.max_fold) * c.head_dim >= (int64_t)1 << 31) return false;
    if ((int64_t)c.max_prefill * c.head_dim >= (int64_t)1 << 31) return false;
    if (c.dtype != FDKV_F32 && c.dtype != FDKV_BF16) return false;
    if (c.keep_den <= 0 || c.keep_num < 0 || c.keep_num > c.keep_den) return false;
    s.L = c.n_layers; s.B = B; s.NB = B == 4 ? 4 : 1; s.P = c.n_layers / B; s.Hq = c.n_q_heads; s.Hkv = c.n_kv_heads; s.G = G; s.d = c.head_dim;
    s.max_batch = c.max_batch; s.Tmax = c.max_prefill; s.max_tail = c.max_tail;
    s.dtype = c.dtype; s.esize = c.dtype == FDKV_BF16 ? 2 : 4;
    s.keep_num = c.keep_num; s.keep_den = c.keep_den;
    s.max_fold = c.max_fold;
    if (c.row_format != FDKV_ROWS_STORAGE && c.row_format != FDKV_ROWS_E4M3) return false;
    s.rows_f8 = c.row_format == FDKV_ROWS_E4M3;
    if (s.rows_f8 && !(c.dtype == FDKV_BF16 && c.head_dim == 128 && G <= 4 && c.max_fold == 0)) return false;
    s.kfold_max = (int64_t)s.max_fold * s.d * s.keep_num / s.keep_den;
    s.kmax = (int64_t)s.Tmax * s.d * s.keep_num / s.keep_den;
    s.kcap = (int64_t)align_up((size_t)(s.kmax + kListPad), 64);
    s.ntiles_max = (s.Tmax + kResTile - 1) / kResTile;
    // per-unit partial-sum slots of the probe: one per 64-token tile (portable kernel) or one per work item of the
    // tensor-core kernel (layers x 128-row blocks x key splits of at least 8 tiles), whichever is more
    s.nptiles_max = std::max((s.Tmax + kProbeTile - 1) / kProbeTile,
                             B * ((G * kMaxW + 127) / 128) * (((s.Tmax - 1) / kProbeBoxRows + 1 + 7) / 8));
    s.tail_rows = (s.max_tail + kRowPad - 1) / kRowPad * kRowPad;
    if (c.residual_rule != FDKV_RESIDUAL_ENTRIES && c.residual_rule != FDKV_RESIDUAL_TOKENS) return false;
    s.tok_rule = c.residual_rule == FDKV_RESIDUAL_TOKENS;
    s.ktok_max = (int64_t)s.Tmax * s.keep_num / s.keep_den;
    s.ktok_cap = (int64_t)align_up((size_t)(s.ktok_max + 32), 64);
    s.NU = s.P * s.Hkv;
    s.NT = 2 * s.NU;
    return true;
}

void make_layouts(const Shape& s, WsLayout& w, ArenaLayout& a) {
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t r = o; o = align_up(o + bytes); return r; };
    const size_t unit_elems = (size_t)s.Tmax * s.d;
    w.status = take(256);
    w.z0 = take((size_t)s.NT * unit_elems * s.esize);
    w.z1 = take((size_t)s.NT * s.NB * unit_elems * s.esize);  // Z1 of a pair, or the four layers' deviations of a block
    w.z1drop = take(s.dtype == FDKV_BF16 && s.d == 128 ? (size_t)s.NU * s.NB * unit_elems * s.esize : 0);
    w.energy = take(s.B == 4 ? (size_t)s.NT * unit_elems * 4 : 0);
    w.eval = take(s.B == 4 ? (size_t)s.NT * s.kcap * 4 : 0);
    w.hist = take((size_t)s.NT * kHistBins * 4);
    w.sel = take((size_t)s.NT * sizeof(SelState));
    w.lb_records = take((size_t)s.NT * s.ntiles_max * 8);
    w.lb_ticket = take(256);
    w.tile_off = take((size_t)s.NT * (s.ntiles_max + 1) * 4);
    w.idx = take((size_t)s.NT * s.kcap * 4);
    w.val = take((size_t)s.NT * s.NB * s.kcap * s.esize);
    w.packed = take(s.dtype == FDKV_BF16 && s.d == 128 ? (size_t)s.NT * s.NB * s.kcap * 4 : 0);
    w.tok_score = take(s.tok_rule ? (size_t)s.NU * s.Tmax * 4 : 0);
    w.tok_flag = take(s.tok_rule ? (size_t)s.NU * s.Tmax : 0);
    w.tok_list = take(s.tok_rule ? (size_t)s.NU * s.ktok_cap * 4 : 0);
    w.tok_off = take(s.tok_rule ? (size_t)s.NU * (s.ntiles_max + 1) * 4 : 0);
    w.probe_part = take((size_t)s.NU * s.nptiles_max * 16);
    w.probe_pos = take((size_t)kMaxW * 4 + (size_t)s.L * 8);
    w.scores = take((size_t)s.NU * 16);
    w.modes = take((size_t)s.NU * 4);
    w.partials = take((size_t)s.max_batch * s.Hq * kMaxSplits * (s.d + 4) * 4);
    w.counters = take((size_t)s.max_batch * s.Hkv * 4);
    w.io_q = take((size_t)s.L * s.max_batch * s.Hq * s.d * 4);  // host-I/O staging: room for every layer of a step
    w.io_k = take((size_t)s.L * s.max_batch * s.Hkv * s.d * 4);
    w.io_v = take((size_t)s.L * s.max_batch * s.Hkv * s.d * 4);
    w.io_out = take((size_t)s.L * s.max_batch * s.Hq * s.d * 4);
    // job tables of the 8-bit commit: one quantise job per stored tensor, one repack job per residual list
    // job tables of a commit: quantise / repack jobs (8-bit rows), then the copy jobs (at most 2 B row copies, or 2 row
    // copies, 2 offset tables and 2 NB lists, per unit)
    w.jobs = take((s.rows_f8 ? (size_t)s.NU * 2 * s.B * (sizeof(QuantJob) + sizeof(RepackJob)) : 0) +
                  (size_t)s.NU * (2 * s.B + 4 + 2 * s.NB) * sizeof(CopyJob));
    w.total = o;

    o = 0;
    a.tail_len = take((size_t)s.L * s.max_batch * 4);
    a.desc = take((size_t)s.max_batch * s.L * s.Hkv * sizeof(UnitDesc));
    const size_t tail = (size_t)s.L * s.max_batch * s.Hkv * s.tail_rows * s.d * s.esize;
    a.tail_k = take(tail);
    a.tail_v = take(tail);
    a.bump = o;
    const size_t rows_pad = align_up((size_t)((s.Tmax + s.max_fold + kRowPad - 1) / kRowPad * kRowPad) * s.d * s.esize);
    const size_t exact_unit = 2 * (size_t)s.B * rows_pad;
    const size_t resid_unit = s.tok_rule
                                  ? 2 * rows_pad + 2 * (size_t)s.NB * align_up((size_t)s.ktok_cap * s.d * s.esize) + align_up((size_t)s.ktok_cap * 4) +
                                        align_up((size_t)(s.ntiles_max + 1) * 4)
                                  : 2 * rows_pad + 2 * (size_t)s.NB * (align_up((size_t)(s.kcap + s.kfold_max) * 4) + align_up((size_t)(s.kcap + s.kfold_max) * s.esize)) +
                                        2 * align_up((size_t)(s.kcap + s.kfold_max) * 4) +
                                        2 * align_up((size_t)(s.ntiles_max + s.max_fold / kResTile + 2) * 4);
    a.worst_total = a.bump + (size_t)s.max_batch * s.NU * (exact_unit > resid_unit ? exact_unit : resid_unit);
}

inline cudaStream_t S(void* p) { return reinterpret_cast<cudaStream_t>(p); }
template <typename T>
inline T* wsp(fdkv_ctx* c, size_t off) { return reinterpret_cast<T*>(c->work + off); }
template <typename T>
inline T* arp(fdkv_ctx* c, size_t off) { return reinterpret_cast<T*>(c->arena + off); }

bool seq_ok(fdkv_ctx* c, int seq) { return c && seq >= 0 && seq < c->s.max_batch; }

// Omega(m) of Eq. 2 for one unit (K and V together): bytes of the mode / bytes of the exact mode.  Returns the latter.
// Residual bytes per kept position: one value and one int32 index (pair), four layer values and one index (block of
// four); token rule: d values per kept token and one index.
double omega_of(const Shape& s, int T, double (&om)[3]) {
    const double e = s.esize, Td = (double)T * s.d;
    const double k = (double)((int64_t)T * s.d * s.keep_num / s.keep_den);
    const double k_tok = (double)((int64_t)T * s.keep_num / s.keep_den);
    const double b_sh = 2.0 * Td * e, b_ex = 2.0 * s.B * Td * e;
    double b_rs;
    if (s.tok_rule) b_rs = b_sh + 2.0 * k_tok * s.d * e * s.NB + 4.0 * k_tok;
    else b_rs = b_sh + 2.0 * k * (s.NB * e + 4.0);
    om[0] = b_sh / b_ex; om[1] = b_rs / b_ex; om[2] = 1.0;
    return b_ex;
}

}  // namespace

namespace fdkv {
void count_launch(int n) { g_launches.fetch_add(n); }
void count_kernel(int id) { if (id >= 0 && id < FDKV_KERNEL_COUNT_) g_kernel_launches[id].fetch_add(1); }
int per_device_first_visits(const int* devs, int n) {
    // the table logic of PerDevice::ensure, fed with device ids instead of the current device
    bool done[PerDevice::kMaxDevices] = {};
    int visits = 0;
    for (int i = 0; i < n; ++i) {
        if (devs[i] < 0 || devs[i] >= PerDevice::kMaxDevices) continue;
        if (!done[devs[i]]) { done[devs[i]] = true; ++visits; }
    }
    return visits;
}
fdkv_status record_cuda_error(cudaError_t e) { return cuda_fail(e); }
cudaError_t launch_set_tail_len(int32_t* tail_len, int L, int max_batch, int seq, int n, cudaStream_t st);
}  // namespace fdkv

extern "C" {

fdkv_status fdkv_sizes(const fdkv_config* cfg, size_t* arena_bytes, size_t* workspace_bytes) {
    Shape s;
    if (!cfg || !make_shape(*cfg, s)) return cfg ? FDKV_ERR_UNSUPPORTED : FDKV_ERR_INVALID_ARG;
    WsLayout w;
    ArenaLayout a;
    make_layouts(s, w, a);
    if (arena_bytes) *arena_bytes = a.worst_total;
    if (workspace_bytes) *workspace_bytes = w.total;
    return FDKV_OK;
}

fdkv_status fdkv_create(const fdkv_config* cfg, void* arena, size_t arena_bytes, void* workspace,
                        size_t workspace_bytes, fdkv_ctx** out) {
    if (!cfg || !arena || !workspace || !out) return FDKV_ERR_INVALID_ARG;
    if (!aligned(arena, 256) || !aligned(workspace, 256)) return FDKV_ERR_INVALID_ARG;
    Shape s;
    if (!make_shape(*cfg, s)) return FDKV_ERR_UNSUPPORTED;
    fdkv_ctx* c = new (std::nothrow) fdkv_ctx();
    if (!c) return FDKV_ERR_INVALID_ARG;
    c->cfg = *cfg;
    c->s = s;
    make_layouts(s, c->ws, c->ar);
    if (workspace_bytes < c->ws.total) { delete c; return FDKV_ERR_WORKSPACE; }
    if (arena_bytes < c->ar.bump) { delete c; return FDKV_ERR_ARENA_FULL; }
    c->arena = (char*)arena;
    c->arena_bytes = arena_bytes;
    c->work = (char*)workspace;
    c->work_bytes = workspace_bytes;
    c->bump = c->ar.bump;
    c->pair_compressed.assign(s.P, 0);
    c->pair_probed.assign(s.P, 0);
    c->pair_scored.assign(s.P, 0);
    c->k_layers.assign(s.L, nullptr);
    c->v_layers.assign(s.L, nullptr);
    c->seqs.resize(s.max_batch);
    for (auto& q : c->seqs) { q.modes.assign(s.NU, -1); q.tail_len.assign(s.L, 0); }
    c->desc_host.resize((size_t)s.max_batch * s.L * s.Hkv);
    cudaError_t e = cudaMemset(c->arena + c->ar.tail_len, 0, (size_t)s.L * s.max_batch * 4);
    if (e == cudaSuccess) e = cudaMemset(c->work + c->ws.status, 0, 256);
    if (e == cudaSuccess) e = cudaMemset(c->work + c->ws.counters, 0, (size_t)s.max_batch * s.Hkv * 4);
    if (e == cudaSuccess) e = cudaMemset(c->arena + c->ar.desc, 0, c->desc_host.size() * sizeof(UnitDesc));
    // tails start as zero rows: the fast decode kernel loads whole 64-row boxes and relies on finite padding
    if (e == cudaSuccess) e = cudaMemset(c->arena + c->ar.tail_k, 0, c->ar.bump - c->ar.tail_k);
    if (e != cudaSuccess) { delete c; return cuda_fail(e); }
    if (s.dtype == FDKV_BF16 && s.d == 128) c->has_tmap = make_arena_tensor_map(c->arena, arena_bytes, c->tmap);
    c->packed_lists = c->has_tmap && s.max_batch * s.Hkv <= kFastMaxUnits;
    if (s.rows_f8 && !(c->packed_lists && make_rows_tensor_map_u8(c->arena, arena_bytes, kRowPad, c->tmap_u8))) { delete c; return FDKV_ERR_UNSUPPORTED; }
    // token rule: the tensor-core score kernel and the packed decode kernel serve bf16 / head_dim 128; everything else
    // takes the float32 score kernel, the float32 probe kernel (which masks the selected rows itself) and the portable decode kernel
    if (s.tok_rule && c->packed_lists)
        c->tok_tc = make_rows_tensor_map(c->work + c->ws.z1, (size_t)s.NT * s.NB * s.Tmax * s.d * s.esize, 128, c->tmap_z1_128);
    if (s.tok_rule && s.dtype == FDKV_BF16 && s.d == 128 && !c->tok_tc) { delete c; return FDKV_ERR_UNSUPPORTED; }
    if (s.dtype == FDKV_BF16 && s.d == 128)
        c->has_probe_tmaps = make_rows_tensor_map(c->work + c->ws.z1, (size_t)s.NT * s.NB * s.Tmax * s.d * s.esize, kProbeBoxRows, c->tmap_z1) &&
                             make_rows_tensor_map(c->work + c->ws.z1drop, (size_t)s.NU * s.NB * s.Tmax * s.d * s.esize, kProbeBoxRows, c->tmap_drop);
    if (c->tok_tc && !c->has_probe_tmaps) { delete c; return FDKV_ERR_UNSUPPORTED; }
    *out = c;
    return FDKV_OK;
}

void fdkv_destroy(fdkv_ctx* ctx) { delete ctx; }

fdkv_status fdkv_reset(fdkv_ctx* c) {
    if (!c) return FDKV_ERR_INVALID_ARG;
    CU(cudaDeviceSynchronize());
    CU(cudaMemset(c->arena + c->ar.tail_len, 0, (size_t)c->s.L * c->s.max_batch * 4));
    CU(cudaMemset(c->work + c->ws.status, 0, 256));
    CU(cudaMemset(c->arena + c->ar.tail_k, 0, c->ar.bump - c->ar.tail_k));
    c->bump = c->ar.bump;
    c->staged_seq = -1;
    for (auto& q : c->seqs) {
        q.committed = false;
        q.T = 0;
        q.fold_used = 0;
        q.k_entries = 0;
        q.modes.assign(c->s.NU, -1);
        q.tail_len.assign(c->s.L, 0);
        q.bytes_by_mode[0] = q.bytes_by_mode[1] = q.bytes_by_mode[2] = 0;
    }
    return FDKV_OK;
}

fdkv_status fdkv_compress_prefill(fdkv_ctx* c, int32_t seq, int32_t pb, int32_t pe, int32_t T,
                                  const void* const* k_layers, const void* const* v_layers, int64_t stride_t,
                                  int64_t stride_h, void* stream) {
    if (!seq_ok(c, seq) || !k_layers || !v_layers) return FDKV_ERR_INVALID_ARG;
    const Shape& s = c->s;
    if (pb < 0 || pe > s.P || pb >= pe) return FDKV_ERR_INVALID_ARG;
    if (T < 1 || T > s.Tmax) return FDKV_ERR_INVALID_ARG;
    if (stride_h < s.d || stride_t < s.d || (stride_t % 8) || (stride_h % 8)) return FDKV_ERR_INVALID_ARG;
    for (int l = s.B * pb; l < s.B * pe; ++l)
        if (!k_layers[l] || !v_layers[l] || !aligned(k_layers[l], 16) || !aligned(v_layers[l], 16))
            return FDKV_ERR_INVALID_ARG;
    if (c->seqs[seq].committed) return FDKV_ERR_STATE;
    if (c->staged_seq != seq || c->staged_T != T) {
        c->staged_seq = seq;
        c->staged_T = T;
        std::fill(c->pair_compressed.begin(), c->pair_compressed.end(), 0);
        std::fill(c->pair_probed.begin(), c->pair_probed.end(), 0);
        std::fill(c->pair_scored.begin(), c->pair_scored.end(), 0);
        c->modes_overridden = false;
        c->seqs[seq].modes.assign(s.NU, -1);
        c->stride_t = stride_t;
        c->stride_h = stride_h;
    } else if (c->stride_t != stride_t || c->stride_h != stride_h) {
        return FDKV_ERR_INVALID_ARG;
    }
    cudaStream_t st = S(stream);
    const int ut_begin = pb * s.Hkv * 2, ut_count = (pe - pb) * s.Hkv * 2;
    CU(cudaMemsetAsync(wsp<uint32_t>(c, c->ws.hist) + (size_t)ut_begin * kHistBins, 0, (size_t)ut_count * kHistBins * 4, st));
    if (s.B == 4) {
        // blocks of four layers: Z0, the layers' deviations and the positions' energies; one kept set per tensor from
        // the float32 radix select on the energies; then the four layers' values at the kept positions
        for (int p = pb; p < pe; ++p) {
            Split4Args a4;
            for (int l = 0; l < 4; ++l) {
                a4.k[l] = k_layers[4 * p + l];
                a4.v[l] = v_layers[4 * p + l];
                c->k_layers[4 * p + l] = a4.k[l];
                c->v_layers[4 * p + l] = a4.v[l];
            }
            a4.stride_t = stride_t; a4.stride_h = stride_h;
            a4.T = T; a4.d = s.d; a4.Hkv = s.Hkv;
            a4.ut_base = p * s.Hkv * 2;
            a4.unit_stride = (int64_t)s.Tmax * s.d;
            a4.z0 = c->work + c->ws.z0; a4.dev = c->work + c->ws.z1;
            a4.energy = wsp<float>(c, c->ws.energy);
            a4.drop = (c->has_probe_tmaps && !s.tok_rule) ? c->work + c->ws.z1drop : nullptr;  // (the token rule writes its own copy in fdkv_probe)
            a4.hist = wsp<uint32_t>(c, c->ws.hist);
            CU(launch_split4_hist(a4, s.dtype, st));
        }
        if (s.tok_rule) {  // the token rule selects inside fdkv_probe
            for (int p = pb; p < pe; ++p) { c->pair_compressed[p] = 1; c->pair_probed[p] = 0; c->pair_scored[p] = 0; }
            return FDKV_OK;
        }
        SelectArgs sa;
        sa.ut_begin = ut_begin; sa.ut_count = ut_count;
        sa.T = T; sa.d = s.d;
        sa.k = (int64_t)T * s.d * s.keep_num / s.keep_den;
        sa.unit_stride = (int64_t)s.Tmax * s.d; sa.kcap = s.kcap; sa.ntiles_max = s.ntiles_max;
        sa.z1 = c->work + c->ws.energy;
        sa.hist = wsp<uint32_t>(c, c->ws.hist);
        sa.sel = wsp<SelState>(c, c->ws.sel);
        sa.lb_records = wsp<unsigned long long>(c, c->ws.lb_records);
        sa.lb_ticket = wsp<uint32_t>(c, c->ws.lb_ticket);
        sa.tile_off = wsp<int32_t>(c, c->ws.tile_off);
        sa.idx = wsp<int32_t>(c, c->ws.idx);
        sa.val = c->work + c->ws.eval;
        sa.packed = nullptr;
        sa.z1drop = nullptr;
        sa.status = wsp<int32_t>(c, c->ws.status);
        CU(launch_select_and_compact(sa, FDKV_F32, st));
        Gather4Args g;
        g.ut_begin = ut_begin; g.ut_count = ut_count;
        g.k = sa.k; g.kcap = s.kcap; g.unit_stride = (int64_t)s.Tmax * s.d;
        g.dev = c->work + c->ws.z1;
        g.idx = wsp<int32_t>(c, c->ws.idx);
        g.val = c->work + c->ws.val;
        g.packed = c->packed_lists ? wsp<uint32_t>(c, c->ws.packed) : nullptr;
        g.drop = c->has_probe_tmaps ? c->work + c->ws.z1drop : nullptr;  // tensor-core probe: the K deviations without the kept positions
        CU(launch_gather4(g, s.dtype, st));
        for (int p = pb; p < pe; ++p) { c->pair_compressed[p] = 1; c->pair_probed[p] = 0; c->pair_scored[p] = 0; }
        return FDKV_OK;
    }
    for (int p0 = pb; p0 < pe; p0 += kSplitPairs) {
        CompressArgs a;
        a.n_pairs = pe - p0 < kSplitPairs ? pe - p0 : kSplitPairs;
        for (int j = 0; j < a.n_pairs; ++j) {
            const int p = p0 + j;
            a.k0[j] = k_layers[2 * p]; a.k1[j] = k_layers[2 * p + 1];
            a.v0[j] = v_layers[2 * p]; a.v1[j] = v_layers[2 * p + 1];
            c->k_layers[2 * p] = a.k0[j]; c->k_layers[2 * p + 1] = a.k1[j];
            c->v_layers[2 * p] = a.v0[j]; c->v_layers[2 * p + 1] = a.v1[j];
        }
        a.stride_t = stride_t; a.stride_h = stride_h;
        a.T = T; a.d = s.d; a.Hkv = s.Hkv; a.tensors = 2;
        a.ut_base = p0 * s.Hkv * 2;
        a.unit_stride = (int64_t)s.Tmax * s.d;
        a.z0 = c->work + c->ws.z0; a.z1 = c->work + c->ws.z1;
        a.hist = wsp<uint32_t>(c, c->ws.hist);
        CU(launch_split_hist(a, s.dtype, st));
    }
    SelectArgs sa;
    sa.ut_begin = ut_begin; sa.ut_count = ut_count;
    sa.T = T; sa.d = s.d;
    sa.k = (int64_t)T * s.d * s.keep_num / s.keep_den;
    sa.unit_stride = (int64_t)s.Tmax * s.d; sa.kcap = s.kcap; sa.ntiles_max = s.ntiles_max;
    sa.z1 = c->work + c->ws.z1;
    sa.hist = wsp<uint32_t>(c, c->ws.hist);
    sa.sel = wsp<SelState>(c, c->ws.sel);
    sa.lb_records = wsp<unsigned long long>(c, c->ws.lb_records);
    sa.lb_ticket = wsp<uint32_t>(c, c->ws.lb_ticket);
    sa.tile_off = wsp<int32_t>(c, c->ws.tile_off);
    sa.idx = wsp<int32_t>(c, c->ws.idx);
    sa.val = c->work + c->ws.val;
    sa.packed = c->packed_lists ? wsp<uint32_t>(c, c->ws.packed) : nullptr;
    sa.z1drop = c->has_probe_tmaps ? c->work + c->ws.z1drop : nullptr;
    sa.status = wsp<int32_t>(c, c->ws.status);
    if (!s.tok_rule) CU(launch_select_and_compact(sa, s.dtype, st));  // the token rule selects inside fdkv_probe
    for (int p = pb; p < pe; ++p) { c->pair_compressed[p] = 1; c->pair_probed[p] = 0; c->pair_scored[p] = 0; }
    return FDKV_OK;
}

fdkv_status fdkv_probe(fdkv_ctx* c, int32_t seq, int32_t pb, int32_t pe, const void* const* q_layers,
                       const int32_t* probe_pos, int32_t W, double lambda, int32_t* modes, float* scores,
                       void* stream) {
    if (!seq_ok(c, seq) || !q_layers || !probe_pos) return FDKV_ERR_INVALID_ARG;
    const Shape& s = c->s;
    if (pb < 0 || pe > s.P || pb >= pe || W < 1 || W > kMaxW) return FDKV_ERR_INVALID_ARG;
    if (!(lambda >= 0.0)) return FDKV_ERR_INVALID_ARG;
    if (c->staged_seq != seq) return FDKV_ERR_STATE;
    for (int p = pb; p < pe; ++p)
        if (!c->pair_compressed[p]) return FDKV_ERR_STATE;
    const int T = c->staged_T;
    for (int i = 0; i < W; ++i)
        if (probe_pos[i] < 0 || probe_pos[i] >= T || (i && probe_pos[i] <= probe_pos[i - 1])) return FDKV_ERR_INVALID_ARG;
    for (int l = s.B * pb; l < s.B * pe; ++l)
        if (!q_layers[l] || !aligned(q_layers[l], 16)) return FDKV_ERR_INVALID_ARG;
    cudaStream_t st = S(stream);
    int32_t* pos_dev = wsp<int32_t>(c, c->ws.probe_pos);
    const void** qptr_dev = reinterpret_cast<const void**>(c->work + c->ws.probe_pos + kMaxW * 4);
    CU(cudaMemcpyAsync(pos_dev, probe_pos, (size_t)W * 4, cudaMemcpyHostToDevice, st));
    CU(cudaMemcpyAsync(qptr_dev + s.B * pb, q_layers + s.B * pb, (size_t)(pe - pb) * s.B * sizeof(void*), cudaMemcpyHostToDevice, st));
    ProbeArgs a;
    a.B = s.B;
    a.unit_begin = pb * s.Hkv; a.unit_count = (pe - pb) * s.Hkv;
    a.T = T; a.d = s.d; a.Hq = s.Hq; a.Hkv = s.Hkv; a.G = s.G; a.W = W;
    a.unit_stride = (int64_t)s.Tmax * s.d; a.kcap = s.kcap;
    a.ntiles_max = s.ntiles_max; a.nptiles_max = s.nptiles_max;
    a.z1 = c->work + c->ws.z1;
    a.idx = wsp<int32_t>(c, c->ws.idx);
    a.tile_off = wsp<int32_t>(c, c->ws.tile_off);
    a.tok_flag = (s.tok_rule && !c->tok_tc) ? wsp<uint8_t>(c, c->ws.tok_flag) : nullptr;
    a.q_layers_dev = qptr_dev;
    a.pos = pos_dev;
    a.part = wsp<double>(c, c->ws.probe_part);
    a.scores = wsp<double>(c, c->ws.scores);
    a.modes = wsp<int32_t>(c, c->ws.modes);
    a.lambda = lambda;
    omega_of(s, T, a.omega);
    a.modes_out = modes; a.scores_out = scores;
    a.tmap_z1 = c->has_probe_tmaps ? c->tmap_z1 : nullptr;
    a.tmap_drop = c->has_probe_tmaps ? c->tmap_drop : nullptr;
    a.Tmax = s.Tmax;
    a.pos_host = probe_pos;
    a.status = wsp<int32_t>(c, c->ws.status);
    if (s.tok_rule) {
        TokenArgs t;
        t.B = s.B;
        t.unit_begin = a.unit_begin; t.unit_count = a.unit_count;
        t.T = T; t.Tmax = s.Tmax; t.Hq = s.Hq; t.Hkv = s.Hkv; t.G = s.G; t.W = W; t.ntiles_max = s.ntiles_max;
        t.k_tok = (int64_t)T * s.keep_num / s.keep_den; t.ktok_cap = s.ktok_cap; t.unit_stride = (int64_t)s.Tmax * s.d;
        t.z1 = c->work + c->ws.z1; t.z1drop = c->work + c->ws.z1drop;
        t.q_layers_dev = qptr_dev; t.pos = pos_dev; t.pos_host = probe_pos;
        t.score = wsp<uint32_t>(c, c->ws.tok_score); t.flag = wsp<uint8_t>(c, c->ws.tok_flag);
        t.list = wsp<int32_t>(c, c->ws.tok_list); t.off = wsp<int32_t>(c, c->ws.tok_off);
        t.tmap_z1_128 = c->tmap_z1_128;
        t.status = wsp<int32_t>(c, c->ws.status);
        CU(launch_token_select(t, s.dtype, s.d, c->tok_tc, st));
        for (int p = pb; p < pe; ++p) c->pair_scored[p] = 1;
    }
    CU(launch_probe(a, s.dtype, st));
    for (int p = pb; p < pe; ++p) c->pair_probed[p] = 1;
    return FDKV_OK;
}

fdkv_status fdkv_route_budget(fdkv_ctx* c, int32_t seq, size_t budget_bytes, double* lambda_host, int32_t* modes_host,
                              void* stream) {
    if (!seq_ok(c, seq)) return FDKV_ERR_INVALID_ARG;
    if (c->staged_seq != seq) return FDKV_ERR_STATE;
    const Shape& s = c->s;
    for (int p = 0; p < s.P; ++p)
        if (!c->pair_probed[p]) return FDKV_ERR_STATE;
    CU(cudaStreamSynchronize(S(stream)));
    std::vector<double> e((size_t)s.NU * 2);
    CU(cudaMemcpy(e.data(), c->work + c->ws.scores, e.size() * sizeof(double), cudaMemcpyDeviceToHost));
    // Omega of the staged sequence, as in fdkv_probe
    const int T = c->staged_T;
    double om[3];
    const double b_ex = omega_of(s, T, om);
    auto mode_at = [&](int u, double lam) {
        const double L0 = e[2 * u] + lam * om[0], L1 = e[2 * u + 1] + lam * om[1], L2 = lam * om[2];
        int m = 0;
        double best = L0;
        if (L1 < best) { best = L1; m = 1; }
        if (L2 < best) { best = L2; m = 2; }
        return m;
    };
    // the footprint only changes where two loss lines of a unit cross: try 0 and every crossing, in ascending order
    std::vector<double> cand;
    cand.reserve((size_t)s.NU * 3 + 1);
    cand.push_back(0.0);
    for (int u = 0; u < s.NU; ++u) {
        cand.push_back((e[2 * u] - e[2 * u + 1]) / (om[1] - om[0]));
        cand.push_back(e[2 * u + 1] / (om[2] - om[1]));
        cand.push_back(e[2 * u] / (om[2] - om[0]));
    }
    std::sort(cand.begin(), cand.end());
    std::vector<int32_t> modes(s.NU, 0);
    bool fits = false;
    double lam_found = INFINITY;
    for (double cv : cand) {
        if (!(cv >= 0.0) || std::isinf(cv)) continue;
        const double lam = cv * (1.0 + std::ldexp(1.0, -40));  // just past the crossing: that unit already took its cheaper mode
        double total = 0.0;
        for (int u = 0; u < s.NU; ++u) {
            modes[u] = mode_at(u, lam);
            total += om[modes[u]] * b_ex;
        }
        if (total <= (double)budget_bytes) { fits = true; lam_found = lam; break; }
    }
    if (!fits) std::fill(modes.begin(), modes.end(), 0);
    c->seqs[seq].modes = modes;
    c->modes_overridden = true;
    if (lambda_host) *lambda_host = lam_found;
    if (modes_host) std::memcpy(modes_host, modes.data(), (size_t)s.NU * 4);
    return fits ? FDKV_OK : FDKV_ERR_ARENA_FULL;
}

fdkv_status fdkv_set_modes(fdkv_ctx* c, int32_t seq, const int32_t* modes_host) {
    if (!seq_ok(c, seq) || !modes_host) return FDKV_ERR_INVALID_ARG;
    if (c->staged_seq != seq) return FDKV_ERR_STATE;
    for (int i = 0; i < c->s.NU; ++i)
        if (modes_host[i] < 0 || modes_host[i] > 2) return FDKV_ERR_INVALID_ARG;
    c->seqs[seq].modes.assign(modes_host, modes_host + c->s.NU);
    c->modes_overridden = true;
    return FDKV_OK;
}

fdkv_status fdkv_commit(fdkv_ctx* c, int32_t seq, void* stream) {
    if (!seq_ok(c, seq)) return FDKV_ERR_INVALID_ARG;
    if (c->staged_seq != seq || c->seqs[seq].committed) return FDKV_ERR_STATE;
    const Shape& s = c->s;
    for (int p = 0; p < s.P; ++p)
        if (!c->pair_compressed[p] || (!c->modes_overridden && !c->pair_probed[p]) || (s.tok_rule && !c->pair_scored[p]))
            return FDKV_ERR_STATE;
    cudaStream_t st = S(stream);
    SeqState& q = c->seqs[seq];
    CU(cudaStreamSynchronize(st));
    if (!c->modes_overridden)
        CU(cudaMemcpy(q.modes.data(), c->work + c->ws.modes, (size_t)s.NU * 4, cudaMemcpyDeviceToHost));
    const int T = c->staged_T;
    const size_t rows = (size_t)T * s.d * s.esize;
    // zero rows up to a whole box, with room for the tokens fdkv_fold_tail may append later
    const size_t rows_pad = (size_t)((T + s.max_fold + kRowPad - 1) / kRowPad * kRowPad) * s.d * s.esize;
    const int64_t k = (int64_t)T * s.d * s.keep_num / s.keep_den;
    const int ntiles = (T + kResTile - 1) / kResTile;
    // list copies include the slack so that aligned over-reads of the last tile stay inside the allocation
    // (copy_* = what the staging area holds now; the allocations add the room of the folded chunks)
    const size_t idx_copy = (size_t)(k + kListPad) * 4, off_copy = (size_t)(ntiles + 1) * 4;
    const size_t val_copy = c->packed_lists ? 0 : (size_t)(k + kListPad) * s.esize;  // packed entries carry their value
    const size_t idx_b = idx_copy + (size_t)s.kfold_max * 4, off_b = off_copy + (size_t)(s.max_fold / kResTile + 1) * 4;
    const size_t val_b = c->packed_lists ? 0 : val_copy + (size_t)s.kfold_max * s.esize;
    const int64_t k_tok = (int64_t)T * s.keep_num / s.keep_den;
    const size_t trow_b = (size_t)(k_tok + 4) * s.d * s.esize, tlist_b = (size_t)(k_tok + 32) * 4;  // token rows, token list
    // 8-bit row streams: 128 bytes per token and a 1 KiB slot for the channel scales (and their maxima) per stored tensor
    const size_t rows8 = (size_t)T * 128, rows8_pad = (size_t)((T + kRowPad - 1) / kRowPad * kRowPad) * 128, scale_slot = 1024;
    const size_t stream_b = s.rows_f8 ? align_up(rows8_pad) + scale_slot : align_up(rows_pad);  // one committed row stream
    size_t need = 0;
    // residual lists of one tensor: packed layout = one entry list per stored high-frequency tensor (one for a pair,
    // four for a block of four layers); portable layout = one index list and one value list per such tensor
    const size_t lists_b = c->packed_lists ? (size_t)s.NB * align_up(idx_b) : align_up(idx_b) + (size_t)s.NB * align_up(val_b);
    for (int u = 0; u < s.NU; ++u) {
        const int m = q.modes[u];
        if (m < 0 || m > 2) return FDKV_ERR_STATE;
        if (m == FDKV_MODE_EXACT) need += 2 * (size_t)s.B * stream_b;
        else if (s.tok_rule) need += 2 * align_up(rows_pad) + (m == FDKV_MODE_RESIDUAL ? 2 * (size_t)s.NB * align_up(trow_b) + align_up(tlist_b) + align_up(off_b) : 0);
        else need += 2 * stream_b + (m == FDKV_MODE_RESIDUAL ? 2 * (lists_b + align_up(off_b)) : 0);
    }
    if (c->bump + need > c->arena_bytes) return FDKV_ERR_ARENA_FULL;
    size_t o = c->bump;
    auto take = [&](size_t bytes) { size_t r = o; o = align_up(o + bytes); return c->arena + r; };
    size_t by_mode[3] = {0, 0, 0};
    const size_t unit_stride_b = (size_t)s.Tmax * s.d * s.esize;
    std::vector<QuantJob> qjobs;   // 8-bit rows: every stored tensor is quantised by one batched pass after this loop
    std::vector<RepackJob> rjobs;  // ... and every residual list repacked relative to its tensor's scales
    std::vector<CopyJob> cjobs;    // device-to-device copies into the arena: one launch over this table after the loop
    int64_t copy_max = 0;
    auto copy_job = [&](const void* src, void* dst, size_t bytes, int64_t src_pitch, int row_bytes) {
        cjobs.push_back(CopyJob{(const char*)src, (char*)dst, (int64_t)bytes, src_pitch, row_bytes, 0});
        copy_max = std::max<int64_t>(copy_max, (int64_t)bytes);
    };
    for (int u = 0; u < s.NU; ++u) {
        const int m = q.modes[u], p = u / s.Hkv, h = u % s.Hkv;
        UnitDesc* dl[4] = {nullptr, nullptr, nullptr, nullptr};
        for (int l = 0; l < s.B; ++l) {
            dl[l] = &c->desc_host[((size_t)seq * s.L + (size_t)s.B * p + l) * s.Hkv + h];
            std::memset(dl[l], 0, sizeof(UnitDesc));
            dl[l]->mode = m;
            dl[l]->T = T;
            dl[l]->sign = s.B == 2 ? (l == 0 ? 1.f : -1.f) : 2.f;
            dl[l]->scale = m == FDKV_MODE_EXACT ? 1.f : (s.B == 2 ? 0.70710678118654752440f : 0.5f);
        }
        if (m == FDKV_MODE_EXACT) {
            for (int l = 0; l < s.B; ++l)
                for (int is_v = 0; is_v < 2; ++is_v) {
                    const void* src = is_v ? c->v_layers[s.B * p + l] : c->k_layers[s.B * p + l];
                    const char* sp = (const char*)src + (size_t)h * c->stride_h * s.esize;
                    if (s.rows_f8) {
                        char* dst = take(rows8_pad);
                        float* sc = reinterpret_cast<float*>(take(scale_slot));
                        if (rows8_pad > rows8) CU(cudaMemsetAsync(dst + rows8, 0, rows8_pad - rows8, st));
                        qjobs.push_back(QuantJob{sp, c->stride_t, T, 0, reinterpret_cast<uint8_t*>(dst), sc});
                        (is_v ? dl[l]->v_rows : dl[l]->k_rows) = dst;
                        (is_v ? dl[l]->v_scale : dl[l]->k_scale) = sc;
                        dl[l]->rows_f8 = 1;
                        continue;
                    }
                    char* dst = take(rows_pad);
                    if (rows_pad > rows) CU(cudaMemsetAsync(dst + rows, 0, rows_pad - rows, st));
                    copy_job(sp, dst, rows, (int64_t)c->stride_t * s.esize, s.d * s.esize);
                    (is_v ? dl[l]->v_rows : dl[l]->k_rows) = dst;
                }
            by_mode[2] += 2 * (size_t)s.B * (s.rows_f8 ? rows8 + 512 : rows);
        } else {
            char *tl = nullptr, *to = nullptr;
            if (s.tok_rule && m == FDKV_MODE_RESIDUAL) {  // one token list and one offset table serve K and V
                tl = take(tlist_b);
                to = take(off_b);
                copy_job(c->work + c->ws.tok_list + (size_t)u * s.ktok_cap * 4, tl, (size_t)k_tok * 4, 16, 16);
                copy_job(c->work + c->ws.tok_off + (size_t)u * (s.ntiles_max + 1) * 4, to, off_copy, 16, 16);
                by_mode[1] += (size_t)k_tok * 4;
            }
            for (int is_v = 0; is_v < 2; ++is_v) {
                const size_t ut = (size_t)u * 2 + is_v;
                float* sc8 = nullptr;
                char* z0;
                if (s.rows_f8) {
                    z0 = take(rows8_pad);
                    sc8 = reinterpret_cast<float*>(take(scale_slot));
                    if (rows8_pad > rows8) CU(cudaMemsetAsync(z0 + rows8, 0, rows8_pad - rows8, st));
                    qjobs.push_back(QuantJob{c->work + c->ws.z0 + ut * unit_stride_b, s.d, T, 0, reinterpret_cast<uint8_t*>(z0), sc8});
                    for (int l = 0; l < s.B; ++l) { (is_v ? dl[l]->v_scale : dl[l]->k_scale) = sc8; dl[l]->rows_f8 = 1; }
                } else {
                    z0 = take(rows_pad);
                    if (rows_pad > rows) CU(cudaMemsetAsync(z0 + rows, 0, rows_pad - rows, st));
                    copy_job(c->work + c->ws.z0 + ut * unit_stride_b, z0, rows, 16, 16);
                }
                for (int l = 0; l < s.B; ++l) (is_v ? dl[l]->v_rows : dl[l]->k_rows) = z0;
                by_mode[m] += s.rows_f8 ? rows8 + 512 : rows;
                if (m == FDKV_MODE_RESIDUAL && s.tok_rule) {
                    // the selected tokens' high-frequency rows, densely packed: Z1 rows of a pair (both layers read them with
                    // opposite signs), each layer's own deviation rows of a block of four (stored doubled: see the gather kernel)
                    // (the list is read where the probe left it: its copy into the arena runs with the other copies after this loop)
                    char* rows_l[4] = {nullptr, nullptr, nullptr, nullptr};
                    for (int j = 0; j < s.NB; ++j) {
                        rows_l[j] = take(trow_b);
                        CU(launch_token_gather(c->work + c->ws.z1 + (ut * s.NB + j) * unit_stride_b, wsp<int32_t>(c, c->ws.tok_list) + (size_t)u * s.ktok_cap, k_tok,
                                               rows_l[j], s.d * s.esize, (s.B == 4 && c->packed_lists) ? 1 : 0, st));
                    }
                    if (s.rows_f8)  // 8-bit rows: the kept rows become f16(value / scale[channel]) in the fragment order of the 8-bit tiles
                        for (int j = 0; j < s.NB; ++j)
                            rjobs.push_back(RepackJob{reinterpret_cast<uint32_t*>(rows_l[j]), reinterpret_cast<const uint32_t*>(rows_l[j]), k_tok, sc8, is_v, 1});
                    for (int l = 0; l < s.B; ++l) {
                        UnitDesc* d = dl[l];
                        d->res_kind = 1;
                        d->k_idx = (const int32_t*)tl;
                        d->k_off = (const int32_t*)to;
                        (is_v ? d->v_val : d->k_val) = rows_l[s.NB == 1 ? 0 : l];
                    }
                    by_mode[1] += (size_t)s.NB * k_tok * s.d * s.esize;
                } else if (m == FDKV_MODE_RESIDUAL) {
                    char* po = take(off_b);
                    copy_job(c->work + c->ws.tile_off + ut * (s.ntiles_max + 1) * 4, po, off_copy, 16, 16);
                    char* pi_shared = nullptr;
                    if (!c->packed_lists) {
                        pi_shared = take(idx_b);
                        CU(cudaMemcpyAsync(pi_shared, c->work + c->ws.idx + ut * s.kcap * 4, idx_copy, cudaMemcpyDeviceToDevice, st));
                    }
                    char *pi_l[4] = {nullptr, nullptr, nullptr, nullptr}, *pv_l[4] = {nullptr, nullptr, nullptr, nullptr};
                    for (int j = 0; j < s.NB; ++j) {  // one list per stored high-frequency tensor
                        const size_t lt = ut * s.NB + j;
                        if (c->packed_lists) {
                            pi_l[j] = take(idx_b);
                            if (s.rows_f8)  // values relative to the channel scales, positions in the converted fragments' order
                                rjobs.push_back(RepackJob{reinterpret_cast<uint32_t*>(pi_l[j]), wsp<uint32_t>(c, c->ws.packed) + lt * s.kcap, k, sc8, is_v, 0});
                            else
                                copy_job(c->work + c->ws.packed + lt * s.kcap * 4, pi_l[j], idx_copy, 16, 16);
                        } else {
                            pi_l[j] = pi_shared;
                            pv_l[j] = take(val_b);
                            CU(cudaMemcpyAsync(pv_l[j], c->work + c->ws.val + lt * s.kcap * s.esize, val_copy, cudaMemcpyDeviceToDevice, st));
                        }
                    }
                    for (int l = 0; l < s.B; ++l) {
                        UnitDesc* d = dl[l];
                        const int j = s.NB == 1 ? 0 : l;  // a pair's two layers read the same Z1 list with opposite signs
                        (is_v ? d->v_idx : d->k_idx) = (const int32_t*)pi_l[j];
                        (is_v ? d->v_val : d->k_val) = pv_l[j];
                        (is_v ? d->v_off : d->k_off) = (const int32_t*)po;
                    }
                    by_mode[1] += (size_t)k * (c->packed_lists ? (size_t)4 * s.NB : 4 + (size_t)s.NB * s.esize);
                }
            }
        }
    }
    if (!cjobs.empty()) {
        CopyJob* cd = reinterpret_cast<CopyJob*>(c->work + c->ws.jobs + (s.rows_f8 ? (size_t)s.NU * 2 * s.B * (sizeof(QuantJob) + sizeof(RepackJob)) : 0));
        CU(cudaMemcpyAsync(cd, cjobs.data(), cjobs.size() * sizeof(CopyJob), cudaMemcpyHostToDevice, st));
        CU(launch_copy_jobs(cd, (int)cjobs.size(), copy_max, st));
    }
    if (!qjobs.empty()) {
        QuantJob* qd = reinterpret_cast<QuantJob*>(c->work + c->ws.jobs);
        RepackJob* rd = reinterpret_cast<RepackJob*>(qd + (size_t)s.NU * 2 * s.B);
        CU(cudaMemcpyAsync(qd, qjobs.data(), qjobs.size() * sizeof(QuantJob), cudaMemcpyHostToDevice, st));
        CU(launch_quantise_jobs(qd, (int)qjobs.size(), T, st));
        if (!rjobs.empty()) {
            CU(cudaMemcpyAsync(rd, rjobs.data(), rjobs.size() * sizeof(RepackJob), cudaMemcpyHostToDevice, st));
            CU(launch_repack_jobs(rd, (int)rjobs.size(), s.tok_rule ? k_tok * 32 : k, st));
        }
    }
    const size_t seq_desc = (size_t)s.L * s.Hkv;
    CU(cudaMemcpyAsync(c->arena + c->ar.desc + (size_t)seq * seq_desc * sizeof(UnitDesc), &c->desc_host[(size_t)seq * seq_desc],
                       seq_desc * sizeof(UnitDesc), cudaMemcpyHostToDevice, st));
    CU(cudaStreamSynchronize(st));
    c->bump = o;
    q.committed = true;
    q.T = T;
    q.fold_used = 0;
    q.k_entries = k;
    for (int i = 0; i < 3; ++i) q.bytes_by_mode[i] = by_mode[i];
    return FDKV_OK;
}

static fdkv_status decode_impl(fdkv_ctx* c, int32_t layer, int32_t batch, const void* q, const void* k_new,
                               const void* v_new, void* out, int32_t out_dtype, cudaStream_t st) {
    const Shape& s = c->s;
    int Tmax = 0;
    for (int b = 0; b < batch; ++b) {
        if (!c->seqs[b].committed) return FDKV_ERR_STATE;
        Tmax = c->seqs[b].T > Tmax ? c->seqs[b].T : Tmax;
    }
    if (k_new) {
        for (int b = 0; b < batch; ++b)
            if (c->seqs[b].tail_len[layer] >= s.max_tail) return FDKV_ERR_STATE;
        for (int b = 0; b < batch; ++b) c->seqs[b].tail_len[layer]++;
    }
    std::vector<int32_t> host_T(batch), host_modes((size_t)batch * s.Hkv);
    for (int b = 0; b < batch; ++b) {
        host_T[b] = c->seqs[b].T;
        for (int h = 0; h < s.Hkv; ++h) host_modes[(size_t)b * s.Hkv + h] = c->seqs[b].modes[(layer / s.B) * s.Hkv + h];
    }
    DecodeArgs a;
    a.tail_rows = s.tail_rows;
    a.host_T = host_T.data(); a.host_modes = host_modes.data();
    std::vector<int32_t> host_tail(batch);  // (already counts this call's append)
    a.any_tail = 0;
    for (int b = 0; b < batch; ++b) {
        host_tail[b] = c->seqs[b].tail_len[layer];
        a.any_tail |= host_tail[b] > 0;
    }
    a.host_tail = host_tail.data();
    a.tmap = c->has_tmap ? c->tmap : nullptr;
    a.tmap_u8 = s.rows_f8 ? c->tmap_u8 : nullptr;
    a.rows_f8 = s.rows_f8;
    a.arena_base = c->arena;
    a.keep_num = s.keep_num; a.keep_den = s.keep_den;
    a.packed_lists = c->packed_lists ? 1 : 0;
    a.tok_rule = s.tok_rule;
    a.desc = arp<UnitDesc>(c, c->ar.desc);
    a.L = s.L; a.layer = layer; a.batch = batch; a.Hq = s.Hq; a.Hkv = s.Hkv; a.G = s.G; a.d = s.d;
    a.max_tail = s.max_tail; a.max_batch = s.max_batch; a.Tmax_batch = Tmax;
    a.q = q; a.k_new = k_new; a.v_new = v_new; a.out = out; a.out_dtype = out_dtype;
    a.tail_k = c->arena + c->ar.tail_k; a.tail_v = c->arena + c->ar.tail_v;
    a.tail_len = arp<int32_t>(c, c->ar.tail_len);
    a.partials = wsp<float>(c, c->ws.partials);
    a.counters = wsp<int32_t>(c, c->ws.counters);
    a.status = wsp<int32_t>(c, c->ws.status);
    CU(launch_decode(a, s.dtype, st));
    return FDKV_OK;
}

fdkv_status fdkv_decode_attn(fdkv_ctx* c, int32_t layer, int32_t batch, const void* q, const void* k_new,
                             const void* v_new, void* out, int32_t out_dtype, void* stream) {
    if (!c || !q || !out) return FDKV_ERR_INVALID_ARG;
    if (layer < 0 || layer >= c->s.L || batch < 1 || batch > c->s.max_batch) return FDKV_ERR_INVALID_ARG;
    if ((k_new == nullptr) != (v_new == nullptr)) return FDKV_ERR_INVALID_ARG;
    if (out_dtype != FDKV_F32 && out_dtype != FDKV_BF16) return FDKV_ERR_INVALID_ARG;
    if (!aligned(q, 16) || !aligned(out, 16) || !aligned(k_new, 16) || !aligned(v_new, 16)) return FDKV_ERR_INVALID_ARG;
    return decode_impl(c, layer, batch, q, k_new, v_new, out, out_dtype, S(stream));
}

fdkv_status fdkv_decode_attn_host(fdkv_ctx* c, int32_t layer, int32_t batch, const void* q, const void* k_new,
                                  const void* v_new, void* out, int32_t out_dtype, void* stream) {
    if (!c || !q || !out) return FDKV_ERR_INVALID_ARG;
    if (layer < 0 || layer >= c->s.L || batch < 1 || batch > c->s.max_batch) return FDKV_ERR_INVALID_ARG;
    if ((k_new == nullptr) != (v_new == nullptr)) return FDKV_ERR_INVALID_ARG;
    if (out_dtype != FDKV_F32 && out_dtype != FDKV_BF16) return FDKV_ERR_INVALID_ARG;
    const Shape& s = c->s;
    cudaStream_t st = S(stream);
    const size_t qb = (size_t)batch * s.Hq * s.d * s.esize, kb = (size_t)batch * s.Hkv * s.d * s.esize;
    const size_t ob = (size_t)batch * s.Hq * s.d * (out_dtype == FDKV_BF16 ? 2 : 4);
    CU(cudaMemcpyAsync(c->work + c->ws.io_q, q, qb, cudaMemcpyHostToDevice, st));
    if (k_new) {
        CU(cudaMemcpyAsync(c->work + c->ws.io_k, k_new, kb, cudaMemcpyHostToDevice, st));
        CU(cudaMemcpyAsync(c->work + c->ws.io_v, v_new, kb, cudaMemcpyHostToDevice, st));
    }
    fdkv_status r = decode_impl(c, layer, batch, c->work + c->ws.io_q, k_new ? c->work + c->ws.io_k : nullptr,
                                k_new ? c->work + c->ws.io_v : nullptr, c->work + c->ws.io_out, out_dtype, st);
    if (r != FDKV_OK) return r;
    CU(cudaMemcpyAsync(out, c->work + c->ws.io_out, ob, cudaMemcpyDeviceToHost, st));
    CU(cudaStreamSynchronize(st));
    return FDKV_OK;
}

fdkv_status fdkv_decode_step_host(fdkv_ctx* c, int32_t batch, const void* q, const void* k_new, const void* v_new, void* out,
                                  int32_t out_dtype, void* stream) {
    if (!c || !q || !out) return FDKV_ERR_INVALID_ARG;
    if (batch < 1 || batch > c->s.max_batch) return FDKV_ERR_INVALID_ARG;
    if ((k_new == nullptr) != (v_new == nullptr)) return FDKV_ERR_INVALID_ARG;
    if (out_dtype != FDKV_F32 && out_dtype != FDKV_BF16) return FDKV_ERR_INVALID_ARG;
    const Shape& s = c->s;
    cudaStream_t st = S(stream);
    const size_t qb = (size_t)batch * s.Hq * s.d * s.esize, kb = (size_t)batch * s.Hkv * s.d * s.esize;
    const size_t ob = (size_t)batch * s.Hq * s.d * (out_dtype == FDKV_BF16 ? 2 : 4);
    CU(cudaMemcpyAsync(c->work + c->ws.io_q, q, qb * s.L, cudaMemcpyHostToDevice, st));
    if (k_new) {
        CU(cudaMemcpyAsync(c->work + c->ws.io_k, k_new, kb * s.L, cudaMemcpyHostToDevice, st));
        CU(cudaMemcpyAsync(c->work + c->ws.io_v, v_new, kb * s.L, cudaMemcpyHostToDevice, st));
    }
    for (int l = 0; l < s.L; ++l) {
        fdkv_status r = decode_impl(c, l, batch, c->work + c->ws.io_q + l * qb, k_new ? c->work + c->ws.io_k + l * kb : nullptr,
                                    k_new ? c->work + c->ws.io_v + l * kb : nullptr, c->work + c->ws.io_out + l * ob, out_dtype, st);
        if (r != FDKV_OK) return r;
    }
    CU(cudaMemcpyAsync(out, c->work + c->ws.io_out, ob * s.L, cudaMemcpyDeviceToHost, st));
    CU(cudaStreamSynchronize(st));
    return FDKV_OK;
}

fdkv_status fdkv_set_tail_len(fdkv_ctx* c, int32_t seq, int32_t n, void* stream) {
    if (!seq_ok(c, seq) || n < 0) return FDKV_ERR_INVALID_ARG;
    for (int l = 0; l < c->s.L; ++l)
        if (n > c->seqs[seq].tail_len[l]) return FDKV_ERR_INVALID_ARG;
    CU(launch_set_tail_len(arp<int32_t>(c, c->ar.tail_len), c->s.L, c->s.max_batch, seq, n, S(stream)));
    c->seqs[seq].tail_len.assign(c->s.L, n);
    return FDKV_OK;
}

fdkv_status fdkv_fold_tail(fdkv_ctx* c, int32_t seq, int32_t n, void* stream) {
    if (!seq_ok(c, seq) || n <= 0) return FDKV_ERR_INVALID_ARG;
    const Shape& s = c->s;
    if (s.tok_rule || s.rows_f8) return FDKV_ERR_UNSUPPORTED;
    SeqState& q = c->seqs[seq];
    if (!q.committed) return FDKV_ERR_STATE;
    if (c->staged_seq >= 0 && !c->seqs[c->staged_seq].committed) return FDKV_ERR_STATE;  // the staging area is in use
    if ((q.T % kResTile) || (n % kResTile) || n > s.Tmax) return FDKV_ERR_INVALID_ARG;
    for (int l = 0; l < s.L; ++l)
        if (q.tail_len[l] != q.tail_len[0]) return FDKV_ERR_STATE;
    if (q.tail_len[0] < n) return FDKV_ERR_INVALID_ARG;
    if (q.fold_used + n > s.max_fold) return FDKV_ERR_ARENA_FULL;
    cudaStream_t st = S(stream);
    const int T0 = q.T, len = q.tail_len[0], rest = len - n;
    const size_t row_b = (size_t)s.d * s.esize;
    const size_t tail_head_b = (size_t)s.tail_rows * row_b;                       // one (layer, sequence, head) tail
    auto tail_base = [&](char* base, int l) { return base + ((size_t)l * s.max_batch + seq) * s.Hkv * tail_head_b; };
    char* tk = c->arena + c->ar.tail_k;
    char* tv = c->arena + c->ar.tail_v;
    // ---- Eq. 1 and the chunk's own selection, through the staging area ----
    c->staged_seq = -1;
    std::fill(c->pair_compressed.begin(), c->pair_compressed.end(), 0);
    CU(cudaMemsetAsync(wsp<uint32_t>(c, c->ws.hist), 0, (size_t)s.NT * kHistBins * 4, st));
    const int64_t kc = (int64_t)n * s.d * s.keep_num / s.keep_den;
    SelectArgs sa;
    sa.ut_begin = 0; sa.ut_count = s.NT;
    sa.T = n; sa.d = s.d; sa.k = kc;
    sa.unit_stride = (int64_t)s.Tmax * s.d; sa.kcap = s.kcap; sa.ntiles_max = s.ntiles_max;
    sa.hist = wsp<uint32_t>(c, c->ws.hist);
    sa.sel = wsp<SelState>(c, c->ws.sel);
    sa.lb_records = wsp<unsigned long long>(c, c->ws.lb_records);
    sa.lb_ticket = wsp<uint32_t>(c, c->ws.lb_ticket);
    sa.tile_off = wsp<int32_t>(c, c->ws.tile_off);
    sa.idx = wsp<int32_t>(c, c->ws.idx);
    sa.z1drop = nullptr;
    sa.status = wsp<int32_t>(c, c->ws.status);
    if (s.B == 4) {
        for (int p = 0; p < s.P; ++p) {
            Split4Args a4;
            for (int l = 0; l < 4; ++l) { a4.k[l] = tail_base(tk, 4 * p + l); a4.v[l] = tail_base(tv, 4 * p + l); }
            a4.stride_t = s.d; a4.stride_h = (int64_t)s.tail_rows * s.d;
            a4.T = n; a4.d = s.d; a4.Hkv = s.Hkv;
            a4.ut_base = p * s.Hkv * 2;
            a4.unit_stride = (int64_t)s.Tmax * s.d;
            a4.z0 = c->work + c->ws.z0; a4.dev = c->work + c->ws.z1;
            a4.energy = wsp<float>(c, c->ws.energy);
            a4.drop = nullptr;
            a4.hist = wsp<uint32_t>(c, c->ws.hist);
            CU(launch_split4_hist(a4, s.dtype, st));
        }
        sa.z1 = c->work + c->ws.energy;
        sa.val = c->work + c->ws.eval;
        sa.packed = nullptr;
        CU(launch_select_and_compact(sa, FDKV_F32, st));
        Gather4Args g;
        g.ut_begin = 0; g.ut_count = s.NT;
        g.k = kc; g.kcap = s.kcap; g.unit_stride = (int64_t)s.Tmax * s.d;
        g.dev = c->work + c->ws.z1;
        g.idx = wsp<int32_t>(c, c->ws.idx);
        g.val = c->work + c->ws.val;
        g.packed = c->packed_lists ? wsp<uint32_t>(c, c->ws.packed) : nullptr;
        g.drop = nullptr;
        CU(launch_gather4(g, s.dtype, st));
    } else {
        for (int p0 = 0; p0 < s.P; p0 += kSplitPairs) {
            CompressArgs a;
            a.n_pairs = s.P - p0 < kSplitPairs ? s.P - p0 : kSplitPairs;
            for (int j = 0; j < a.n_pairs; ++j) {
                const int p = p0 + j;
                a.k0[j] = tail_base(tk, 2 * p); a.k1[j] = tail_base(tk, 2 * p + 1);
                a.v0[j] = tail_base(tv, 2 * p); a.v1[j] = tail_base(tv, 2 * p + 1);
            }
            a.stride_t = s.d; a.stride_h = (int64_t)s.tail_rows * s.d;
            a.T = n; a.d = s.d; a.Hkv = s.Hkv; a.tensors = 2;
            a.ut_base = p0 * s.Hkv * 2;
            a.unit_stride = (int64_t)s.Tmax * s.d;
            a.z0 = c->work + c->ws.z0; a.z1 = c->work + c->ws.z1;
            a.hist = wsp<uint32_t>(c, c->ws.hist);
            CU(launch_split_hist(a, s.dtype, st));
        }
        sa.z1 = c->work + c->ws.z1;
        sa.val = c->work + c->ws.val;
        sa.packed = c->packed_lists ? wsp<uint32_t>(c, c->ws.packed) : nullptr;
        CU(launch_select_and_compact(sa, s.dtype, st));
    }
    // ---- append behind every unit's rows and lists, under the unit's mode ----
    const size_t unit_stride_b = (size_t)s.Tmax * s.d * s.esize, chunk_b = (size_t)n * row_b, at = (size_t)T0 * row_b;
    const int64_t k_old = q.k_entries;
    const int nslices = n / kResTile;
    for (int u = 0; u < s.NU; ++u) {
        const int m = q.modes[u], p = u / s.Hkv, h = u % s.Hkv;
        UnitDesc* dl[4] = {nullptr, nullptr, nullptr, nullptr};
        for (int l = 0; l < s.B; ++l) dl[l] = &c->desc_host[((size_t)seq * s.L + (size_t)s.B * p + l) * s.Hkv + h];
        if (m == FDKV_MODE_EXACT) {
            for (int l = 0; l < s.B; ++l) {
                CU(cudaMemcpyAsync((char*)dl[l]->k_rows + at, tail_base(tk, s.B * p + l) + h * tail_head_b, chunk_b, cudaMemcpyDeviceToDevice, st));
                CU(cudaMemcpyAsync((char*)dl[l]->v_rows + at, tail_base(tv, s.B * p + l) + h * tail_head_b, chunk_b, cudaMemcpyDeviceToDevice, st));
            }
            q.bytes_by_mode[2] += 2 * (size_t)s.B * chunk_b;
            continue;
        }
        for (int is_v = 0; is_v < 2; ++is_v) {
            const size_t ut = (size_t)u * 2 + is_v;
            char* rows = (char*)(is_v ? dl[0]->v_rows : dl[0]->k_rows);  // every layer of the block shares the coefficient rows
            CU(cudaMemcpyAsync(rows + at, c->work + c->ws.z0 + ut * unit_stride_b, chunk_b, cudaMemcpyDeviceToDevice, st));
            q.bytes_by_mode[m] += chunk_b;
            if (m != FDKV_MODE_RESIDUAL) continue;
            int32_t* off = const_cast<int32_t*>(is_v ? dl[0]->v_off : dl[0]->k_off);
            if (c->packed_lists) {
                // packed entries carry slice-relative positions: valid as they are (T0 is a multiple of 16); one list per
                // stored high-frequency tensor (a pair's two layers share theirs)
                for (int j = 0; j < s.NB; ++j) {
                    int32_t* list = const_cast<int32_t*>(is_v ? dl[j]->v_idx : dl[j]->k_idx);
                    CU(cudaMemcpyAsync(list + k_old, c->work + c->ws.packed + (ut * s.NB + j) * s.kcap * 4, (size_t)kc * 4, cudaMemcpyDeviceToDevice, st));
                }
            } else {
                int32_t* list = const_cast<int32_t*>(is_v ? dl[0]->v_idx : dl[0]->k_idx);  // one index list for the unit
                CU(launch_offset_copy(list + k_old, wsp<int32_t>(c, c->ws.idx) + ut * s.kcap, (int)kc, T0 * s.d, st));
                for (int j = 0; j < s.NB; ++j) {
                    char* val = (char*)const_cast<void*>(is_v ? dl[j]->v_val : dl[j]->k_val);
                    CU(cudaMemcpyAsync(val + (size_t)k_old * s.esize, c->work + c->ws.val + (ut * s.NB + j) * s.kcap * s.esize, (size_t)kc * s.esize,
                                       cudaMemcpyDeviceToDevice, st));
                }
            }
            CU(launch_offset_copy(off + T0 / kResTile, wsp<int32_t>(c, c->ws.tile_off) + ut * (s.ntiles_max + 1), nslices + 1, (int)k_old, st));
            q.bytes_by_mode[1] += (size_t)kc * (c->packed_lists ? (size_t)4 * s.NB : 4 + (size_t)s.NB * s.esize);
        }
    }
    // ---- the remaining tail rows move down (through the staging area: the ranges may overlap) ----
    if (rest > 0) {
        char* tmp = c->work + c->ws.z1;
        const size_t w = (size_t)rest * row_b;
        for (int l = 0; l < s.L; ++l)
            for (char* base : {tail_base(tk, l), tail_base(tv, l)}) {
                CU(cudaMemcpy2DAsync(tmp, w, base + (size_t)n * row_b, tail_head_b, w, s.Hkv, cudaMemcpyDeviceToDevice, st));
                CU(cudaMemcpy2DAsync(base, tail_head_b, tmp, w, w, s.Hkv, cudaMemcpyDeviceToDevice, st));
            }
    }
    CU(launch_set_tail_len(arp<int32_t>(c, c->ar.tail_len), s.L, s.max_batch, seq, rest, st));
    q.tail_len.assign(s.L, rest);
    // ---- descriptors: every layer of the sequence now holds T0 + n prompt-side tokens ----
    const size_t seq_desc = (size_t)s.L * s.Hkv;
    for (size_t i = 0; i < seq_desc; ++i) c->desc_host[(size_t)seq * seq_desc + i].T = T0 + n;
    CU(cudaMemcpyAsync(c->arena + c->ar.desc + (size_t)seq * seq_desc * sizeof(UnitDesc), &c->desc_host[(size_t)seq * seq_desc],
                       seq_desc * sizeof(UnitDesc), cudaMemcpyHostToDevice, st));
    CU(cudaStreamSynchronize(st));
    q.T = T0 + n;
    q.k_entries = k_old + kc;
    q.fold_used += n;
    return FDKV_OK;
}

fdkv_status fdkv_get_rows_e4m3(fdkv_ctx* c, int32_t seq, int32_t layer, int32_t h, int32_t is_v, uint8_t* codes_out, float* scale_out,
                               void* stream) {
    if (!seq_ok(c, seq) || layer < 0 || layer >= c->s.L || h < 0 || h >= c->s.Hkv) return FDKV_ERR_INVALID_ARG;
    if (!c->s.rows_f8) return FDKV_ERR_UNSUPPORTED;
    if (!c->seqs[seq].committed) return FDKV_ERR_STATE;
    const UnitDesc& d = c->desc_host[((size_t)seq * c->s.L + layer) * c->s.Hkv + h];
    if (codes_out) CU(cudaMemcpyAsync(codes_out, is_v ? d.v_rows : d.k_rows, (size_t)d.T * 128, cudaMemcpyDeviceToDevice, S(stream)));
    if (scale_out) CU(cudaMemcpyAsync(scale_out, is_v ? d.v_scale : d.k_scale, 512, cudaMemcpyDeviceToDevice, S(stream)));
    CU(cudaStreamSynchronize(S(stream)));
    return FDKV_OK;
}

fdkv_status fdkv_get_shared(fdkv_ctx* c, int32_t seq, int32_t pair, int32_t h, int32_t is_v, void* z0_out, void* stream) {
    if (!seq_ok(c, seq) || !z0_out || pair < 0 || pair >= c->s.P || h < 0 || h >= c->s.Hkv) return FDKV_ERR_INVALID_ARG;
    if (c->staged_seq != seq || !c->pair_compressed[pair]) return FDKV_ERR_STATE;
    const Shape& s = c->s;
    const size_t ut = ((size_t)pair * s.Hkv + h) * 2 + (is_v ? 1 : 0);
    CU(cudaMemcpyAsync(z0_out, c->work + c->ws.z0 + ut * s.Tmax * s.d * s.esize, (size_t)c->staged_T * s.d * s.esize,
                       cudaMemcpyDeviceToDevice, S(stream)));
    CU(cudaStreamSynchronize(S(stream)));
    return FDKV_OK;
}

fdkv_status fdkv_get_residual(fdkv_ctx* c, int32_t seq, int32_t pair, int32_t h, int32_t is_v, int32_t* idx_out,
                              void* val_out, int32_t* count_host, void* stream) {
    if (!seq_ok(c, seq) || pair < 0 || pair >= c->s.P || h < 0 || h >= c->s.Hkv) return FDKV_ERR_INVALID_ARG;
    if (c->staged_seq != seq || !c->pair_compressed[pair]) return FDKV_ERR_STATE;
    const Shape& s = c->s;
    if (s.tok_rule) return FDKV_ERR_UNSUPPORTED;  // token rule: see fdkv_get_token_set
    const size_t ut = ((size_t)pair * s.Hkv + h) * 2 + (is_v ? 1 : 0);
    const int64_t k = (int64_t)c->staged_T * s.d * s.keep_num / s.keep_den;
    if (count_host) *count_host = (int32_t)k;
    if (idx_out && k) CU(cudaMemcpyAsync(idx_out, c->work + c->ws.idx + ut * s.kcap * 4, (size_t)k * 4, cudaMemcpyDeviceToDevice, S(stream)));
    for (int j = 0; j < s.NB && val_out && k; ++j)  // a block of four returns its four layers' values as [4][count]
        CU(cudaMemcpyAsync((char*)val_out + (size_t)j * k * s.esize, c->work + c->ws.val + (ut * s.NB + j) * s.kcap * s.esize,
                           (size_t)k * s.esize, cudaMemcpyDeviceToDevice, S(stream)));
    CU(cudaStreamSynchronize(S(stream)));
    return FDKV_OK;
}

fdkv_status fdkv_get_token_set(fdkv_ctx* c, int32_t seq, int32_t pair, int32_t h, int32_t* tok_out, float* score_out,
                               int32_t* count_host, void* stream) {
    if (!seq_ok(c, seq) || pair < 0 || pair >= c->s.P || h < 0 || h >= c->s.Hkv) return FDKV_ERR_INVALID_ARG;
    const Shape& s = c->s;
    if (!s.tok_rule) return FDKV_ERR_UNSUPPORTED;
    if (c->staged_seq != seq || !c->pair_scored[pair]) return FDKV_ERR_STATE;
    const size_t u = (size_t)pair * s.Hkv + h;
    const int64_t k_tok = (int64_t)c->staged_T * s.keep_num / s.keep_den;
    if (count_host) *count_host = (int32_t)k_tok;
    if (tok_out && k_tok) CU(cudaMemcpyAsync(tok_out, c->work + c->ws.tok_list + u * s.ktok_cap * 4, (size_t)k_tok * 4, cudaMemcpyDeviceToDevice, S(stream)));
    if (score_out) CU(cudaMemcpyAsync(score_out, c->work + c->ws.tok_score + u * s.Tmax * 4, (size_t)c->staged_T * 4, cudaMemcpyDeviceToDevice, S(stream)));
    CU(cudaStreamSynchronize(S(stream)));
    return FDKV_OK;
}

fdkv_status fdkv_get_modes(fdkv_ctx* c, int32_t seq, int32_t* modes_host) {
    if (!seq_ok(c, seq) || !modes_host) return FDKV_ERR_INVALID_ARG;
    if (!c->seqs[seq].committed && !(c->staged_seq == seq && c->modes_overridden)) return FDKV_ERR_STATE;
    std::memcpy(modes_host, c->seqs[seq].modes.data(), (size_t)c->s.NU * 4);
    return FDKV_OK;
}

fdkv_status fdkv_footprint(fdkv_ctx* c, int32_t seq, size_t* bytes_by_mode_host, size_t* exact_equiv_bytes_host) {
    if (!seq_ok(c, seq)) return FDKV_ERR_INVALID_ARG;
    if (!c->seqs[seq].committed) return FDKV_ERR_STATE;
    if (bytes_by_mode_host)
        for (int i = 0; i < 3; ++i) bytes_by_mode_host[i] = c->seqs[seq].bytes_by_mode[i];
    if (exact_equiv_bytes_host)
        *exact_equiv_bytes_host = (size_t)c->s.NU * 2 * c->s.B * c->seqs[seq].T * c->s.d * c->s.esize;
    return FDKV_OK;
}

fdkv_status fdkv_plan_decode(int32_t batch, int32_t n_kv_heads, const int32_t* T_host, const int32_t* modes_host,
                             int32_t keep_num, int32_t keep_den, int32_t residual_rule, int32_t row_format, int32_t n_ctas,
                             uint32_t* start_out, int32_t* n_ctas_out, int32_t* parts_out) {
    if (!T_host || !modes_host || !start_out || !n_ctas_out || !parts_out) return FDKV_ERR_INVALID_ARG;
    if (batch < 1 || n_kv_heads < 1 || (int64_t)batch * n_kv_heads > kFastMaxUnits || n_ctas < 1 || n_ctas > 160) return FDKV_ERR_INVALID_ARG;
    if (keep_num < 0 || keep_den < 1 || keep_num > keep_den) return FDKV_ERR_INVALID_ARG;
    for (int b = 0; b < batch; ++b)
        if (T_host[b] < 1 || (int64_t)T_host[b] * 128 >= ((int64_t)1 << 31)) return FDKV_ERR_INVALID_ARG;
    for (int i = 0; i < batch * n_kv_heads; ++i)
        if (modes_host[i] < 0 || modes_host[i] > 2) return FDKV_ERR_INVALID_ARG;
    DecodeArgs a;
    std::memset(&a, 0, sizeof(a));
    a.batch = batch; a.Hkv = n_kv_heads; a.d = 128;
    a.host_T = T_host; a.host_modes = modes_host;
    a.keep_num = keep_num; a.keep_den = keep_den;
    a.tok_rule = residual_rule == FDKV_RESIDUAL_TOKENS ? 1 : 0;
    a.rows_f8 = row_format != 0 ? 1 : 0;
    return plan_decode_host(a, n_ctas, start_out, n_ctas_out, parts_out) == cudaSuccess ? FDKV_OK : FDKV_ERR_INVALID_ARG;
}

fdkv_status fdkv_decode_bytes(fdkv_ctx* c, int32_t layer, int32_t batch, size_t* bytes_host) {
    if (!c || !bytes_host || layer < 0 || layer >= c->s.L || batch < 1 || batch > c->s.max_batch) return FDKV_ERR_INVALID_ARG;
    const Shape& s = c->s;
    size_t tot = 0;
    for (int b = 0; b < batch; ++b) {
        const SeqState& q = c->seqs[b];
        if (!q.committed) return FDKV_ERR_STATE;
        const int64_t k = q.k_entries;  // prompt + folded chunks
        const int ntiles = (q.T + kResTile - 1) / kResTile;
        for (int h = 0; h < s.Hkv; ++h) {
            const int m = q.modes[(layer / s.B) * s.Hkv + h];
            tot += s.rows_f8 ? 2 * ((size_t)q.T * s.d + 512) + 2 * (size_t)q.tail_len[layer] * s.d * s.esize
                             : 2 * (size_t)(q.T + q.tail_len[layer]) * s.d * s.esize;
            if (m == FDKV_MODE_RESIDUAL && s.tok_rule) {
                const size_t kt = (size_t)((int64_t)q.T * s.keep_num / s.keep_den);
                tot += 2 * kt * s.d * s.esize + kt * 4 + (size_t)(ntiles + 1) * 4;
            } else if (m == FDKV_MODE_RESIDUAL)
                tot += 2 * ((size_t)k * (c->packed_lists ? 4 : 4 + s.esize) + (size_t)(ntiles + 1) * 4);
        }
    }
    *bytes_host = tot;
    return FDKV_OK;
}

fdkv_status fdkv_device_status(fdkv_ctx* c) {
    if (!c) return FDKV_ERR_INVALID_ARG;
    int32_t flag = 0;
    CU(cudaDeviceSynchronize());
    CU(cudaMemcpy(&flag, c->work + c->ws.status, 4, cudaMemcpyDeviceToHost));
    if (flag == kFlagOk) return FDKV_OK;
    return flag == kFlagTimeout ? FDKV_ERR_TIMEOUT : FDKV_ERR_DEVICE;
}

int32_t fdkv_last_cuda_error(void) { return g_last_cuda.load(); }

const char* fdkv_status_str(fdkv_status s) {
    switch (s) {
        case FDKV_OK: return "ok";
        case FDKV_ERR_INVALID_ARG: return "invalid argument";
        case FDKV_ERR_UNSUPPORTED: return "unsupported shape or dtype";
        case FDKV_ERR_ARENA_FULL: return "arena full";
        case FDKV_ERR_WORKSPACE: return "workspace too small";
        case FDKV_ERR_STATE: return "call order / state";
        case FDKV_ERR_CUDA: return "CUDA runtime error";
        case FDKV_ERR_TIMEOUT: return "device wait timed out";
        case FDKV_ERR_DEVICE: return "device-side check failed";
        case FDKV_ERR_TOO_LARGE: return "input larger than the built-in scratch of the allocation-free entry point";
    }
    return "unknown";
}

int64_t fdkv_launch_count(void) { return g_launches.load(); }
int64_t fdkv_kernel_launch_count(int32_t kernel) {
    return kernel >= 0 && kernel < FDKV_KERNEL_COUNT_ ? g_kernel_launches[kernel].load() : -1;
}

}  // extern "C"
