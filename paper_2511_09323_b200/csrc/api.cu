// C ABI of the MoC FFN library: argument validation, workspace carving, kernel plans.
// Everything here is host code that only enqueues kernels on the caller's stream.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <atomic>
#include <cstdint>
#include <cstring>
#include <mutex>
#include <unordered_map>
#include <vector>

#include "decode_coop.cuh"
#include "decode_kernels.cuh"
#include "gather_kernels.cuh"
#include "grouped_select.cuh"
#include "moc_common.cuh"
#include "small_batch.cuh"
#include "small_batch_fused.cuh"
#include "tc_gemm.cuh"
#include "tc_gemm_sp.cuh"
#include "tc_plan.cuh"
#include "topk_select.cuh"

namespace moc {

// ---- device status word ---------------------------------------------------------------------------
__device__ int g_status_word = 0;

int *device_status_ptr() {
    // the symbol has one instance per device; its address is looked up once per device (several host threads may
    // race to look it up: they store the same value)
    static std::atomic<int *> cache[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    int *have = cache[dev].load(std::memory_order_relaxed);
    if (!have) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_status_word) != cudaSuccess) return nullptr;
        have = static_cast<int *>(p);
        cache[dev].store(have, std::memory_order_relaxed);
    }
    return have;
}

// State that the one-kernel small-batch form keeps from one run to the next (the counters of its column blocks, the
// flags its CTAs signal with and a mark that says both are zero): kept in the library's own device memory rather than
// in the caller's workspace, whose contents between calls are the caller's.  One block of kFusedStateWords words per
// workspace address -- a workspace serves one call at a time, so a block is never used by two runs at once.
constexpr int kFusedStateWords = 128, kFusedStateSlots = 1024;
__device__ unsigned int g_fused_state[kFusedStateSlots * kFusedStateWords];

unsigned int *fused_state_for(const void *workspace) {
    static std::mutex mu;
    static std::unordered_map<uint64_t, int> slot_of[64];
    static unsigned int *base[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!base[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_fused_state) != cudaSuccess) return nullptr;
        base[dev] = static_cast<unsigned int *>(p);
    }
    auto &m = slot_of[dev];
    auto it = m.find(reinterpret_cast<uint64_t>(workspace));
    if (it == m.end()) {
        if ((int)m.size() >= kFusedStateSlots) return nullptr;  // (the multi-kernel forms serve further workspaces)
        it = m.emplace(reinterpret_cast<uint64_t>(workspace), (int)m.size()).first;
    }
    return base[dev] + (size_t)it->second * kFusedStateWords;
}

// ---- launch bookkeeping --------------------------------------------------------------------------
// Every kernel the library launches goes through MOC_LAUNCH: it counts the launch and, while a
// profiling window is open, brackets it with a pair of CUDA events on the caller's stream so that
// a benchmark can read per-kernel device time without a profiler attached.
enum KernelId {
    KID_GATE_GEMM_ALU = 0,
    KID_SELECT_ROWS,
    KID_FORWARD_TOKEN,
    KID_BACKWARD_TOKEN,
    KID_CSR_COUNT,
    KID_CSR_SCAN_BLOCKS,
    KID_CSR_SCAN_CHANNELS,
    KID_CSR_FILL,
    KID_WGRAD_ROWS,
    KID_TOPK_SELECT,
    KID_TC_GATE_UP_GEMM,
    KID_TC_SELECT_MASK,
    KID_TC_DOWN_GEMM,
    KID_TC_BWD_SAMPLE,
    KID_TC_DZ_GEMM,
    KID_TC_WGRAD_GEMM,
    KID_TC_DX_GEMM,
    KID_TC_TEST_GEMM,
    KID_TC_SELECT_HINT,
    KID_DEC_GATE_GEMV,
    KID_DEC_SELECT,
    KID_DEC_UP,
    KID_DEC_DOWN,
    KID_SB_GATE_UP,
    KID_SB_SELECT,
    KID_SB_DOWN,
    KID_RECOMPUTE_UP,
    KID_DEC_COOP,
    KID_DEC_RMSNORM,
    KID_TC_COMPRESS,
    KID_TC_SP_DOWN_GEMM,
    KID_TC_SP_DX_GEMM,
    KID_STREAM_PROBE,
    KID_SB_FUSED,
    KID_TC_SPLIT_SUM,
    KID_COUNT
};
static const char *const kKernelNames[KID_COUNT] = {
    "gate_gemm_alu", "select_rows",       "forward_token", "backward_token", "csr_count",
    "csr_scan_blocks", "csr_scan_channels", "csr_fill",      "wgrad_rows",     "topk_select",
    "tc_gate_up_gemm", "tc_select_mask",  "tc_down_gemm",  "tc_bwd_sample",  "tc_dz_gemm",
    "tc_wgrad_gemm",   "tc_dx_gemm",      "tc_test_gemm",  "tc_select_hint", "dec_gate_gemv",
    "dec_select",      "dec_up",          "dec_down",      "sb_gate_up",     "sb_select",
    "sb_down",         "recompute_up",    "dec_coop",      "dec_rmsnorm",    "tc_compress_2of4",
    "tc_sp_down_gemm", "tc_sp_dx_gemm", "stream_probe",    "sb_fused",
    "tc_split_sum",
};

struct Profiler {
    static constexpr int kMaxPairs = 8192;
    std::atomic<int64_t> launches{0};
    bool on = false;
    std::vector<cudaEvent_t> ev;  // 2 * kMaxPairs, created on first use
    int used = 0, dropped = 0;
    int ids[kMaxPairs];
    double ms[KID_COUNT] = {};
    int64_t count[KID_COUNT] = {};
};
static Profiler g_prof;

static bool prof_begin(int kid, cudaStream_t st) {
    g_prof.launches.fetch_add(1, std::memory_order_relaxed);
    if (!g_prof.on) return false;
    if (g_prof.used >= Profiler::kMaxPairs) {
        ++g_prof.dropped;
        return false;
    }
    g_prof.ids[g_prof.used] = kid;
    return cudaEventRecord(g_prof.ev[2 * g_prof.used], st) == cudaSuccess;
}
static void prof_end(bool rec, cudaStream_t st) {
    if (!rec) return;
    cudaEventRecord(g_prof.ev[2 * g_prof.used + 1], st);
    ++g_prof.used;
}
#define MOC_LAUNCH(kid, st, ...)                   \
    do {                                           \
        const bool moc_rec_ = prof_begin(kid, st); \
        __VA_ARGS__;                               \
        prof_end(moc_rec_, st);                    \
    } while (0)

namespace {

constexpr size_t kAlign = 256;
constexpr int kMaxDynSmem = 227 * 1024;

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool good_ptr(const void *p) { return p != nullptr && aligned16(p); }
inline size_t esize(int dtype) { return dtype == MOC_BF16 ? 2 : 4; }

int check_desc(const moc_ffn_desc *d) {
    if (!d) return MOC_ERR_INVALID_ARG;
    if (d->tokens < 0 || d->d_model < 1 || d->d_ff < 1 || d->d_ff_ld < d->d_ff || d->k < 1 || d->k > d->d_ff)
        return MOC_ERR_INVALID_ARG;
    if (d->dtype != MOC_F32 && d->dtype != MOC_BF16) return MOC_ERR_UNSUPPORTED;
    if (d->flags & ~(MOC_FLAG_ACCUMULATE_WGRAD | MOC_FLAG_SELECT_2_OF_8 | MOC_FLAG_SELECT_POST_SILU))
        return MOC_ERR_INVALID_ARG;
    if ((d->flags & MOC_FLAG_SELECT_2_OF_8) && (d->flags & MOC_FLAG_SELECT_POST_SILU)) return MOC_ERR_INVALID_ARG;
    if ((d->flags & MOC_FLAG_SELECT_2_OF_8) && (d->d_ff % 8 != 0 || d->k != d->d_ff / 4)) return MOC_ERR_INVALID_ARG;
    if (d->d_ff > 32768) return MOC_ERR_UNSUPPORTED;     // int16 channel indices
    if (d->d_model % 8 != 0) return MOC_ERR_UNSUPPORTED;  // 16-byte row vectors
    if ((double)d->tokens * (double)d->k >= 4294967296.0) return MOC_ERR_UNSUPPORTED;  // 32-bit pair ids
    return MOC_OK;
}

// ---- workspace layouts ------------------------------------------------------------------------------
struct Carver {
    size_t off = 0;
    size_t take(size_t bytes) {
        size_t o = off;
        off = align_up(off + bytes, kAlign);
        return o;
    }
};

struct ForwardPlan {
    int64_t chunk;   // tokens per gate-projection chunk
    size_t off_g;    // fp32 [chunk, F]
    size_t off_idx;  // int16 [T, K] when the caller keeps nothing
    size_t total;
};

ForwardPlan plan_forward(const moc_ffn_desc &d) {
    ForwardPlan p{};
    const size_t row = (size_t)d.d_ff * 4;
    int64_t chunk = (int64_t)std::max<size_t>(1, ((size_t)256 << 20) / row);
    chunk = std::min<int64_t>(chunk, 1 << 20);  // keeps the gate GEMM's grid.y in range
    p.chunk = std::max<int64_t>(1, std::min<int64_t>(d.tokens, chunk));
    Carver c;
    p.off_g = c.take((size_t)p.chunk * row);
    p.off_idx = c.take((size_t)d.tokens * d.k * sizeof(int16_t));
    p.total = c.off;
    return p;
}

struct BackwardPlan {
    int tb, nb;  // tokens per block / number of token blocks of the channel-list build
    size_t off_coef, off_counts, off_totals, off_rowstart, off_pairs, total;
};

BackwardPlan plan_backward(const moc_ffn_desc &d) {
    BackwardPlan p{};
    const int64_t T = d.tokens;
    int64_t nb = std::min<int64_t>(1184, (T + 7) / 8);
    nb = std::max<int64_t>(1, nb);
    p.tb = (int)((T + nb - 1) / nb);
    if (p.tb < 1) p.tb = 1;
    p.nb = (int)((T + p.tb - 1) / p.tb);
    if (p.nb < 1) p.nb = 1;
    const size_t TK = (size_t)T * d.k;
    Carver c;
    p.off_coef = c.take(3 * TK * sizeof(float));
    p.off_counts = c.take((size_t)p.nb * d.d_ff * sizeof(uint32_t));
    p.off_totals = c.take((size_t)d.d_ff * sizeof(uint32_t));
    p.off_rowstart = c.take(((size_t)d.d_ff + 1) * sizeof(uint32_t));
    p.off_pairs = c.take(TK * sizeof(uint32_t));
    p.total = c.off;
    return p;
}

template <typename K>
int set_smem(K kernel, size_t bytes, size_t kStaticReserve = 48 * 1024) {
    // by default room is left for the selector's static shared state (up to 47 KiB with 1024 threads), which
    // most kernels that call this hold
    if (bytes + kStaticReserve > (size_t)kMaxDynSmem) return MOC_ERR_UNSUPPORTED;
    if (bytes + kStaticReserve > 48 * 1024) {
        // the attribute only ever grows; remember what was set so that steady-state calls make no driver call
        static std::mutex mu;
        static std::unordered_map<const void *, size_t> configured;
        std::lock_guard<std::mutex> lock(mu);
        size_t &have = configured[reinterpret_cast<const void *>(kernel)];
        if (have < bytes) {
            if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess)
                return MOC_ERR_CUDA;
            have = bytes;
        }
    }
    return MOC_OK;
}

inline int launch_ok() { return cudaGetLastError() == cudaSuccess ? MOC_OK : MOC_ERR_CUDA; }

size_t token_red_floats(int d) {
    const int nvec = d / 8;
    const int lanes_v = std::min(nvec, kTokenThreads);
    const int G = kTokenThreads / lanes_v;
    return G > 1 ? (size_t)G * d : 0;
}

// ---- forward (gathered plan) -------------------------------------------------------------------------
template <typename T>
int forward_gather(const moc_ffn_desc &d, const T *x, const T *wg, const T *wu, const T *wd, T *out,
                   int16_t *idx, T *tg, T *tu, char *ws, cudaStream_t st) {
    const ForwardPlan p = plan_forward(d);
    float *G = reinterpret_cast<float *>(ws + p.off_g);
    if (!idx) idx = reinterpret_cast<int16_t *>(ws + p.off_idx);
    const int F = d.d_ff, K = d.k, dm = d.d_model;

    const size_t sel_smem = (size_t)F * sizeof(uint32_t);
    int rc = set_smem(select_rows_kernel<T>, sel_smem);
    if (rc != MOC_OK) return rc;
    const size_t tok_smem = ((size_t)dm + 2 * (size_t)K + token_red_floats(dm)) * sizeof(float);
    rc = set_smem(forward_token_kernel<T>, tok_smem);
    if (rc != MOC_OK) return rc;

    for (int64_t t0 = 0; t0 < d.tokens; t0 += p.chunk) {
        const int64_t n = std::min<int64_t>(p.chunk, d.tokens - t0);
        dim3 grid((F + 63) / 64, (unsigned)((n + 63) / 64));
        MOC_LAUNCH(KID_GATE_GEMM_ALU, st, (gemm_nt_alu_kernel<T><<<grid, 256, 0, st>>>(x + t0 * dm, wg, G, (int)n, F, dm, F)));
        if ((rc = launch_ok()) != MOC_OK) return rc;
        if (d.flags & MOC_FLAG_SELECT_2_OF_8) {
            const unsigned grp_grid = (unsigned)std::min<int64_t>((n * (F / 8) + 255) / 256, 148 * 32);
            MOC_LAUNCH(KID_SELECT_ROWS, st,
                       (select_grouped_idx_kernel<T><<<grp_grid, 256, 0, st>>>(G, n, F, F, idx + t0 * K,
                                                                                tg ? tg + t0 * K : nullptr)));
        } else {
            const unsigned sel_grid = (unsigned)std::min<int64_t>(n, 148 * 32);
            MOC_LAUNCH(KID_SELECT_ROWS, st,
                       (select_rows_kernel<T><<<sel_grid, kSelectThreads, sel_smem, st>>>(
                           G, n, F, F, K, idx + t0 * K, tg ? tg + t0 * K : nullptr,
                           (d.flags & MOC_FLAG_SELECT_POST_SILU) ? 1 : 0)));
        }
        if ((rc = launch_ok()) != MOC_OK) return rc;
        MOC_LAUNCH(KID_FORWARD_TOKEN, st,
                   (forward_token_kernel<T><<<(unsigned)n, kTokenThreads, tok_smem, st>>>(
                       x + t0 * dm, wu, wd, G, F, idx + t0 * K, dm, K, out + t0 * dm, tu ? tu + t0 * K : nullptr,
                       0)));
        if ((rc = launch_ok()) != MOC_OK) return rc;
    }
    return MOC_OK;
}

// ---- backward (gathered plan) ------------------------------------------------------------------------
template <typename T>
int backward_gather(const moc_ffn_desc &d, const T *x, const T *wg, const T *wu, const T *wd,
                    const int16_t *idx, const T *tg, const T *tu, const T *dout, T *gx, T *gwg, T *gwu, T *gwd,
                    char *ws, cudaStream_t st, cudaEvent_t wgrad_done) {
    const BackwardPlan p = plan_backward(d);
    const int F = d.d_ff, K = d.k, dm = d.d_model;
    const int64_t TK = d.tokens * (int64_t)K;
    const bool want_w = gwg || gwu || gwd;
    float *coef = reinterpret_cast<float *>(ws + p.off_coef);
    int *status = device_status_ptr();
    if (!status) return MOC_ERR_CUDA;

    const size_t tok_smem = ((size_t)dm + 3 * (size_t)K + token_red_floats(dm)) * sizeof(float);
    int rc = set_smem(backward_token_kernel<T>, tok_smem);
    if (rc != MOC_OK) return rc;
    MOC_LAUNCH(KID_BACKWARD_TOKEN, st,
               (backward_token_kernel<T><<<(unsigned)d.tokens, kTokenThreads, tok_smem, st>>>(
                   wg, wu, wd, idx, tg, tu, dout, dm, F, K, TK, gx, want_w ? coef : nullptr, status)));
    if ((rc = launch_ok()) != MOC_OK) return rc;
    if (!want_w) {
        if (wgrad_done && cudaEventRecord(wgrad_done, st) != cudaSuccess) return MOC_ERR_CUDA;
        return MOC_OK;
    }

    uint32_t *counts = reinterpret_cast<uint32_t *>(ws + p.off_counts);
    uint32_t *totals = reinterpret_cast<uint32_t *>(ws + p.off_totals);
    uint32_t *row_start = reinterpret_cast<uint32_t *>(ws + p.off_rowstart);
    uint32_t *pairs = reinterpret_cast<uint32_t *>(ws + p.off_pairs);
    const size_t f_smem = (size_t)F * sizeof(uint32_t);
    if ((rc = set_smem(csr_count_kernel, f_smem)) != MOC_OK) return rc;
    if ((rc = set_smem(csr_fill_kernel, f_smem)) != MOC_OK) return rc;
    MOC_LAUNCH(KID_CSR_COUNT, st, (csr_count_kernel<<<p.nb, 256, f_smem, st>>>(idx, d.tokens, K, F, p.tb, counts)));
    if ((rc = launch_ok()) != MOC_OK) return rc;
    MOC_LAUNCH(KID_CSR_SCAN_BLOCKS, st,
               (csr_scan_blocks_kernel<<<(F + 255) / 256, 256, 0, st>>>(counts, p.nb, F, totals)));
    if ((rc = launch_ok()) != MOC_OK) return rc;
    MOC_LAUNCH(KID_CSR_SCAN_CHANNELS, st, (csr_scan_channels_kernel<<<1, 1024, 0, st>>>(totals, F, row_start)));
    if ((rc = launch_ok()) != MOC_OK) return rc;
    MOC_LAUNCH(KID_CSR_FILL, st,
               (csr_fill_kernel<<<p.nb, 256, f_smem, st>>>(idx, d.tokens, K, F, p.tb, counts, row_start, pairs)));
    if ((rc = launch_ok()) != MOC_OK) return rc;

    const size_t red = token_red_floats(dm) * 3 * sizeof(float);
    if ((rc = set_smem(wgrad_rows_kernel<T>, red)) != MOC_OK) return rc;
    MOC_LAUNCH(KID_WGRAD_ROWS, st,
               (wgrad_rows_kernel<T><<<d.d_ff_ld, kTokenThreads, red, st>>>(
                   x, dout, coef, TK, row_start, pairs, dm, F, K, gwg, gwu, gwd,
                   (d.flags & MOC_FLAG_ACCUMULATE_WGRAD) ? 1 : 0)));
    if ((rc = launch_ok()) != MOC_OK) return rc;
    if (wgrad_done && cudaEventRecord(wgrad_done, st) != cudaSuccess) return MOC_ERR_CUDA;
    return MOC_OK;
}

// ---- tensor-core plan (bf16 training shapes) ---------------------------------------------------------
bool use_tc_plan(const moc_ffn_desc &d) {
    // bf16 at every token count: even for a handful of tokens the dense contractions on the tensor cores (one
    // padded 128-row tile, weights read once) beat the gathered ALU kernels, 10x at the LLaMA-7B shape
    if (d.dtype != MOC_BF16 || d.tokens < 1) return false;
    // the forward selector keeps F keys and K packed entries in shared memory
    return ((size_t)d.d_ff + (size_t)d.k) * 4 <= 170 * 1024;
}

// The forward pass of the tensor-core plan selects on the gate values themselves: the post-SiLU ablation variant
// takes the gathered kernels (the backward pass does not select and keeps its plan).
bool use_tc_forward(const moc_ffn_desc &d) { return use_tc_plan(d) && !(d.flags & MOC_FLAG_SELECT_POST_SILU); }

inline int ceil_div(int64_t a, int64_t b) { return (int)((a + b - 1) / b); }

// ---- the row Top-K selector of the tensor-core plan: which kernel form serves a row of F channels with K kept ----
// A team of warps per token while at least two tokens' rows fit an SM's shared memory (each team stages its token's
// rows in its own slice: as many teams per SM as fit, in one or two CTAs; rows too long for that with separate gate
// and up buffers let the two rows share one buffer), else one CTA per token.  Teams of four warps for long rows (few
// tokens fit an SM there), pairs otherwise (measured: LLaMA-1B width 0.59 -> 0.50 ms and LLaMA-7B width 0.56 -> 0.41 ms
// with four; 2048 channels 0.080 -> 0.124 ms, so short rows keep pairs).
struct TcSelect {
    int nv;             // 128-channel groups of a row
    int team;           // warps per token (2 or 4)
    bool team_select;   // false: one CTA per token (select_mask_rows_kernel)
    bool shared_u;      // gate and up row share one buffer
    int tokens_per_cta, ctas_per_sm;
    size_t smem;        // dynamic shared memory of the launch
    int variant;        // MOC_SELECT_VARIANT_* (what a test hook reports)
};

enum {
    MOC_SELECT_VARIANT_CTA_PER_ROW = 0,   // select_mask_rows_kernel
    MOC_SELECT_VARIANT_TEAM2 = 1,         // teams of two warps, separate gate / up buffers
    MOC_SELECT_VARIANT_TEAM4 = 2,         // teams of four warps, separate buffers
    MOC_SELECT_VARIANT_TEAM4_SHARED = 3,  // teams of four, one buffer for both rows
};

TcSelect tc_select_config(int F, int K) {
    using namespace tc;
    TcSelect c{};
    c.nv = ceil_div(F, 128);
    c.team = c.nv >= 40 ? 4 : 2;
    const auto units_fit = [&](bool shared) {  // tokens in flight per SM
        return (int)std::min<size_t>(
            (size_t)220 * 1024 / (pair_select_words(c.nv, K, shared, c.team) * sizeof(uint32_t)), 16);
    };
    const bool parks = pair_select_parks_gates(c.nv, K, c.team);
    const int min_units = 2;  // at least two tokens in flight per SM
    // (rows short enough for teams of two always fit with separate buffers: the shared form exists for teams of four)
    c.shared_u = c.team == 4 && units_fit(false) < min_units && parks && units_fit(true) >= min_units;
    const size_t team_bytes = pair_select_words(c.nv, K, c.shared_u, c.team) * sizeof(uint32_t);
    const int per_sm = units_fit(c.shared_u);
    const int units_per_cta = kPairSelMaxWarps / c.team;
    c.team_select = per_sm >= min_units;
    if (c.team_select) {
        c.ctas_per_sm = per_sm > units_per_cta ? 2 : 1;
        c.tokens_per_cta = std::min(per_sm / c.ctas_per_sm, units_per_cta);
        c.smem = (size_t)c.tokens_per_cta * team_bytes;
        c.variant = c.team == 4 ? (c.shared_u ? MOC_SELECT_VARIANT_TEAM4_SHARED : MOC_SELECT_VARIANT_TEAM4)
                                : MOC_SELECT_VARIANT_TEAM2;
    } else {
        c.ctas_per_sm = 6;
        c.tokens_per_cta = 1;
        c.smem = ((size_t)F + K) * sizeof(uint32_t);
        c.variant = MOC_SELECT_VARIANT_CTA_PER_ROW;
    }
    return c;
}

// the usual row lengths get their loops unrolled (the template's first parameter)
#define MOC_TC_SELECT_DISPATCH(c, DO)                                                   \
    do {                                                                                \
        if ((c).team == 4) {                                                            \
            if ((c).shared_u) DO((tc::select_mask_rows_pair_kernel<0, true, 4>), 128);  \
            else if ((c).nv == 43) DO((tc::select_mask_rows_pair_kernel<43, false, 4>), 128); \
            else DO((tc::select_mask_rows_pair_kernel<0, false, 4>), 128);              \
        } else {                                                                        \
            if ((c).nv == 8) DO((tc::select_mask_rows_pair_kernel<8, false, 2>), 64);   \
            else if ((c).nv == 16) DO((tc::select_mask_rows_pair_kernel<16, false, 2>), 64); \
            else if ((c).nv == 32) DO((tc::select_mask_rows_pair_kernel<32, false, 2>), 64); \
            else DO((tc::select_mask_rows_pair_kernel<0, false, 2>), 64);               \
        }                                                                               \
    } while (0)

int tc_select_prepare(const TcSelect &c, int F, int K) {
    int rc = MOC_OK;
    if (c.team_select) {
#define MOC_DO_SET(KERN, TPT) rc = set_smem(KERN, c.smem, 2048)
        MOC_TC_SELECT_DISPATCH(c, MOC_DO_SET);
#undef MOC_DO_SET
    } else {
        rc = set_smem(tc::select_mask_rows_kernel, c.smem);
    }
    if (rc != MOC_OK) return rc;
    return set_smem(tc::select_hint_kernel, (size_t)F * sizeof(uint32_t));
}

// Team selector: every launch works with one bracket kept in the workspace ({center, width, tag} at hint[0..2]); it
// gathers the statistics of its thresholds (hint[4..6], CTA counter at hint[8]) and its last CTA rewrites the bracket
// for the next launch.  The bracket is only a hint: a stale or garbage one costs time (rows take the general exact
// path), never correctness; the statistics and the counter reset themselves at the end of every launch.
// CTA-per-token selector: hint[0..1] is the guess select_hint_kernel left.
void tc_select_launch(const TcSelect &c, const float *G, int ldg, __nv_bfloat16 *U, int ldu, int64_t n, int F, int K,
                      int16_t *o_idx, __nv_bfloat16 *o_g, __nv_bfloat16 *o_u, float *hint, int *status, cudaStream_t st) {
    using namespace tc;
    if (c.team_select) {
        SelectMeta meta{};
        meta.bracket = hint;
        meta.acc = hint + 4;
        meta.done = reinterpret_cast<unsigned int *>(hint + 8);
        const unsigned grid = (unsigned)std::min<int64_t>((n + c.tokens_per_cta - 1) / c.tokens_per_cta,
                                                          (int64_t)sm_count() * c.ctas_per_sm);
#define MOC_DO_LAUNCH(KERN, TPT)                                                                     \
    MOC_LAUNCH(KID_TC_SELECT_MASK, st,                                                               \
               (KERN<<<grid, c.tokens_per_cta * TPT, c.smem, st>>>(G, ldg, U, ldu, n, F, c.nv, K, o_idx, o_g, o_u, \
                                                                    meta, status)))
        MOC_TC_SELECT_DISPATCH(c, MOC_DO_LAUNCH);
#undef MOC_DO_LAUNCH
    } else {
        const unsigned grid = (unsigned)std::min<int64_t>(n, (int64_t)sm_count() * 6);
        MOC_LAUNCH(KID_TC_SELECT_MASK, st,
                   (select_mask_rows_kernel<<<grid, kSelectThreads, c.smem, st>>>(G, ldg, U, ldu, n, F, K, o_idx, o_g,
                                                                                   o_u, hint)));
    }
}

// ---- 2:4-sparse contractions (tcgen05.mma.sp): compressed operand + metadata in the workspace -----------------
struct SparseOperandLayout {
    int kc_ld;          // leading dimension of the compressed rows (elements): K / 2 rounded up to 64
    int k_stages;       // stages of 128 logical contraction elements
    size_t comp_bytes, meta_bytes;
};
SparseOperandLayout sparse_operand_layout(int64_t rows, int K) {
    SparseOperandLayout L{};
    L.k_stages = ceil_div(K, tcsp::SBKL);
    L.kc_ld = L.k_stages * (tcsp::SBKL / 2);
    const int64_t blocks = (rows + 127) / 128;
    L.comp_bytes = align_up((size_t)blocks * 128 * L.kc_ld * sizeof(__nv_bfloat16), kAlign);
    L.meta_bytes = align_up((size_t)blocks * L.k_stages * 128 * 4 * sizeof(uint32_t), kAlign);
    return L;
}

// MOC_FFN_SPARSE=0 in the environment keeps every contraction on the dense MMA (comparisons)
bool sparse_mma_enabled() {
    static const bool on = [] {
        const char *e = getenv("MOC_FFN_SPARSE");
        return !(e && strcmp(e, "0") == 0);
    }();
    return on && tc::pair_mode();
}

// dense [rows, ld] (at most 2 non-zero values per group of 4) -> compressed rows + metadata
int sparse_compress(const __nv_bfloat16 *dense, int64_t rows, int K, int ld, const SparseOperandLayout &L,
                    __nv_bfloat16 *comp, uint32_t *meta, tcsp::Overflow *overflow, int overflow_cap,
                    unsigned int *overflow_n, cudaStream_t st, int *bad_status = nullptr) {
    const int64_t jobs = ((rows + 127) / 128) * L.k_stages;
    const unsigned grid = (unsigned)std::min<int64_t>(jobs, (int64_t)tc::sm_count() * 8);
    MOC_LAUNCH(KID_TC_COMPRESS, st,
               (tcsp::compress_2of4_kernel<<<grid, 512, 0, st>>>(dense, rows, K, ld, comp, L.kc_ld, meta, L.k_stages,
                                                                  overflow, overflow_cap, overflow_n, bad_status)));
    return launch_ok();
}

// C [M, N] bf16 = sum over segments of A_seg (compressed, [M, K]) * B_seg ([K, N], N contiguous)
int sparse_gemm_pair(int64_t M, int N, int K, int segments, const __nv_bfloat16 *const comp[2],
                     const uint32_t *const meta[2], const SparseOperandLayout &L, const __nv_bfloat16 *const b[2],
                     int ldb, __nv_bfloat16 *c, int ldc, bool accumulate, int kid, int *status, cudaStream_t st) {
    using namespace tcsp;
    using tc::EncodeTiledFn;
    using tc::encode_fn;
    SpPairParams p;
    memset(&p, 0, sizeof(p));
    for (int sgm = 0; sgm < segments; ++sgm) {
        // (columns K / 2 .. kc_ld of the compressed rows are never written: the map ends at K / 2)
        if (!tc::make_map(&p.a_map[sgm], comp[sgm], M, K / 2, L.kc_ld, 64, SBM) ||
            !tc::make_map(&p.b_map[sgm], b[sgm], K, N, ldb, 64, 64))
            return MOC_ERR_CUDA;
        // the metadata as a matrix of 32-bit words, 4 per row: one stage of one 128-row block is a box of 4 x 128
        EncodeTiledFn fn = encode_fn();
        if (!fn) return MOC_ERR_CUDA;
        const int64_t blocks = (M + 127) / 128;
        cuuint64_t dims[2] = {4, (cuuint64_t)(blocks * L.k_stages * 128)};
        cuuint64_t strides[1] = {16};
        cuuint32_t box[2] = {4, 128};
        cuuint32_t estr[2] = {1, 1};
        if (fn(&p.e_map[sgm], CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<uint32_t *>(meta[sgm]), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return MOC_ERR_CUDA;
    }
    p.segments = segments;
    p.k_stages = L.k_stages;
    p.M = (int)M;
    p.N = N;
    p.m_pairs = ceil_div(M, 2 * SBM);
    p.n_tiles = ceil_div(N, PBN);
    p.c = c;
    p.ldc = ldc;
    p.accumulate = accumulate ? 1 : 0;
    p.status = status;
    static int max_pairs = 0;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.blockDim = dim3(PTHREADS);
    cfg.dynamicSmemBytes = PSMEM_BYTES;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (!max_pairs) {
        if (cudaFuncSetAttribute(gemm_sp_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PSMEM_BYTES) != cudaSuccess)
            return MOC_ERR_CUDA;
        cfg.gridDim = dim3(2 * (unsigned)tc::sm_count());
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, gemm_sp_pair_kernel, &cfg) != cudaSuccess || n <= 0) return MOC_ERR_CUDA;
        max_pairs = n;
    }
    const int tiles = p.m_pairs * p.n_tiles;
    const int pairs = std::min(tiles, max_pairs);
    if (pairs <= 0) return MOC_OK;
    cfg.gridDim = dim3(2 * (unsigned)pairs);
    int rc = MOC_OK;
    MOC_LAUNCH(kid, st, (rc = cudaLaunchKernelEx(&cfg, gemm_sp_pair_kernel, p) == cudaSuccess ? MOC_OK : MOC_ERR_CUDA));
    return rc;
}

// out = bf16(a + b), 8 elements per thread (the two halves of a contraction that was split, see below)
__global__ void __launch_bounds__(256) split_sum_kernel(const float *__restrict__ a, const float *__restrict__ b,
                                                        __nv_bfloat16 *__restrict__ out, int64_t n8) {
    for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < n8; i += (int64_t)gridDim.x * 256) {
        const float4 a0 = __ldcs(reinterpret_cast<const float4 *>(a) + 2 * i), a1 = __ldcs(reinterpret_cast<const float4 *>(a) + 2 * i + 1);
        const float4 b0 = __ldcs(reinterpret_cast<const float4 *>(b) + 2 * i), b1 = __ldcs(reinterpret_cast<const float4 *>(b) + 2 * i + 1);
        reinterpret_cast<uint4 *>(out)[i] = make_uint4(tc::pack_bf16(a0.x + b0.x, a0.y + b0.y), tc::pack_bf16(a0.z + b0.z, a0.w + b0.w),
                                                      tc::pack_bf16(a1.x + b1.x, a1.y + b1.y), tc::pack_bf16(a1.z + b1.z, a1.w + b1.w));
    }
}

// (see tc::split_contraction_pays) -- here with the room the caller has for the partial outputs
bool split_contraction(int64_t T, int n_cols, size_t scratch_floats) {
    return tc::split_contraction_pays(T, n_cols) && (size_t)2 * T * n_cols <= scratch_floats;
}

int launch_split_sum(const float *partial, int64_t T, int n_cols, __nv_bfloat16 *out, cudaStream_t st) {
    const int64_t n8 = T * n_cols / 8;
    const unsigned grid = (unsigned)std::min<int64_t>((n8 + 255) / 256, (int64_t)tc::sm_count() * 8);
    MOC_LAUNCH(KID_TC_SPLIT_SUM, st, (split_sum_kernel<<<grid, 256, 0, st>>>(partial, partial + T * n_cols, out, n8)));
    return launch_ok();
}

// D = Z' W_down over all tokens: A = Z' [T, F] (K-major), B = Wd [F, d] (its contiguous dimension is N).
// scratch: fp32 words of dead workspace for the partial outputs of a split contraction (or none)
int forward_tc_down(const moc_ffn_desc &d, const __nv_bfloat16 *Z, int ldz, const __nv_bfloat16 *wd, __nv_bfloat16 *out,
                    int *status, cudaStream_t st, float *scratch = nullptr, size_t scratch_floats = 0) {
    using namespace tc;
    const int F = d.d_ff, dm = d.d_model;
    const int64_t T = d.tokens;
    int rc = MOC_OK;
    Params q;
    init_params(q);
    if (scratch && F >= 4 * BK && split_contraction(T, dm, scratch_floats)) {
        const int Kc = ceil_div(ceil_div(F, 2), BK) * BK;  // channels of the first half: whole 64-channel blocks
        for (int h = 0; h < 2; ++h) {
            const int k0 = h * Kc, kn = std::min(Kc, F - k0);
            if (!map_k_major(&q.a_map[h], Z + k0, T, kn, ldz, BM) || !map_mn_major(&q.b_map[h], wd + (int64_t)k0 * dm, kn, dm, dm))
                return MOC_ERR_CUDA;
            q.a_idx[h][0] = q.b_idx[h][0] = (int8_t)h;
            q.c[h] = scratch + (int64_t)h * T * dm;
            q.ldc[h] = dm;
        }
        q.num_problems = 2;
        q.k_blocks = Kc / BK;
        q.M = (int)T;
        q.N = dm;
        q.m_tiles = ceil_div(T, BM);
        q.n_tiles = ceil_div(dm, BN);
        q.status = status;
        MOC_LAUNCH(KID_TC_DOWN_GEMM, st, (rc = launch_gemm<false, true, EPI_F32>(q, st)));
        if (rc != MOC_OK) return rc;
        return launch_split_sum(scratch, T, dm, out, st);
    }
    if (!map_k_major(&q.a_map[0], Z, T, F, ldz, BM) || !map_mn_major(&q.b_map[0], wd, F, dm, dm)) return MOC_ERR_CUDA;
    q.k_blocks = ceil_div(F, BK);
    q.M = (int)T;
    q.N = dm;
    q.m_tiles = ceil_div(T, BM);
    q.n_tiles = ceil_div(dm, BN);
    q.c[0] = out;
    q.ldc[0] = dm;
    q.status = status;
    MOC_LAUNCH(KID_TC_DOWN_GEMM, st, (rc = launch_gemm<false, true, EPI_BF16>(q, st)));
    return rc;
}

int forward_tc(const moc_ffn_desc &d, const __nv_bfloat16 *x, const __nv_bfloat16 *wg, const __nv_bfloat16 *wu,
               const __nv_bfloat16 *wd, __nv_bfloat16 *out, int16_t *idx, __nv_bfloat16 *tg, __nv_bfloat16 *tu,
               char *ws, cudaStream_t st) {
    using namespace tc;
    const TcForwardLayout L = tc_forward_layout(d);
    float *G = reinterpret_cast<float *>(ws + L.off_g);
    __nv_bfloat16 *U = reinterpret_cast<__nv_bfloat16 *>(ws + L.off_u);
    const int F = d.d_ff, K = d.k, dm = d.d_model;
    const int64_t T = d.tokens;
    const int f_tiles = ceil_div(F, BN);

    const TcSelect sel = tc_select_config(F, K);
    float *hint = reinterpret_cast<float *>(ws + L.off_hint);
    int rc = tc_select_prepare(sel, F, K);
    if (rc != MOC_OK) return rc;

    int *status = device_status_ptr();
    if (!status) return MOC_ERR_CUDA;
    if ((d.flags & MOC_FLAG_SELECT_2_OF_8) && pair_mode()) {
        // MoC 2:8: the mask is local to groups of eight channels, so it is applied in the epilogue of one GEMM whose
        // tiles hold the gate and the up projection of the same 128 channels side by side: Z' and the saved triple
        // are all that reaches memory, and no selector kernel runs
        Params q;
        init_params(q);
        if (!map_k_major(&q.a_map[0], x, T, dm, dm, BM) || !map_k_major(&q.b_map[0], wg, F, dm, dm, BN / 2) ||
            !map_k_major(&q.b_map[1], wu, F, dm, dm, BN / 2))
            return MOC_ERR_CUDA;
        q.status = status;
        q.k_blocks = ceil_div(dm, BK);
        q.M = (int)T;
        q.N = F;
        q.m_tiles = ceil_div(T, BM);
        q.n_tiles = ceil_div(F, BN / 2);
        q.c[0] = U;
        q.ldc[0] = L.ldf;
        q.sv_idx = idx;
        q.sv_g = idx ? tg : nullptr;
        q.sv_u = idx ? tu : nullptr;
        // Every 4 consecutive channels of a 2:8 row hold at most 2 kept values: the epilogue hands Z' over in the
        // compressed form of the 2:4-sparse MMA, and the down projection contracts over twice the channels per instruction
        const SparseOperandLayout SL = sparse_operand_layout(T, F);
        // (the compressed rows live in U's buffer; with few output columns the GEMM is too short for its 1.5 x to pay
        // for the slower epilogue of the gate + up GEMM: LLaMA-130M shape 0.170 -> 0.174 ms, LLaMA-1B shape 1.57 -> 1.43 ms)
        const bool sparse_down = sparse_mma_enabled() && SL.kc_ld <= L.ldf && dm >= 1024;
        uint32_t *zmeta = reinterpret_cast<uint32_t *>(ws + L.off_meta);
        if (sparse_down) {
            q.zc = U;
            q.zc_ld = SL.kc_ld;
            q.zmeta = zmeta;
            q.zmeta_stages = SL.k_stages;
        }
        MOC_LAUNCH(KID_TC_GATE_UP_GEMM, st, (rc = launch_gemm<false, false, EPI_GATE_UP_2OF8>(q, st)));
        if (rc != MOC_OK) return rc;
        if (sparse_down) {
            const __nv_bfloat16 *comps[2] = {U, nullptr};
            const uint32_t *metas[2] = {zmeta, nullptr};
            const __nv_bfloat16 *bs[2] = {wd, nullptr};
            return sparse_gemm_pair(T, dm, F, 1, comps, metas, SL, bs, dm, out, dm, false, KID_TC_SP_DOWN_GEMM, status, st);
        }
        return forward_tc_down(d, U, L.ldf, wd, out, status, st);
    }
    Params p;
    init_params(p);
    if (!map_k_major(&p.b_map[0], wg, F, dm, dm, b_box_rows()) || !map_k_major(&p.b_map[1], wu, F, dm, dm, b_box_rows()))
        return MOC_ERR_CUDA;
    p.status = status;
    p.num_problems = 2;
    p.b_idx[1][0] = 1;
    p.k_blocks = ceil_div(dm, BK);
    p.N = F;
    p.n_tiles = f_tiles;
    p.ldc[0] = p.ldc[1] = L.ldf;
    for (int64_t t0 = 0; t0 < T; t0 += L.chunk) {
        const int64_t n = std::min<int64_t>(L.chunk, T - t0);
        if (!map_k_major(&p.a_map[0], x + t0 * dm, n, dm, dm, BM)) return MOC_ERR_CUDA;
        p.M = (int)n;
        p.m_tiles = ceil_div(n, BM);
        p.c[0] = G;
        p.c[1] = U + t0 * L.ldf;
        MOC_LAUNCH(KID_TC_GATE_UP_GEMM, st, (rc = launch_gemm<false, false, EPI_GATE_UP>(p, st)));
        if (rc != MOC_OK) return rc;
        if (t0 == 0 && !sel.team_select) {
            MOC_LAUNCH(KID_TC_SELECT_HINT, st,
                       (select_hint_kernel<<<1, kSelectThreads, (size_t)F * sizeof(uint32_t), st>>>(G, F, K, hint)));
            if ((rc = launch_ok()) != MOC_OK) return rc;
        }
        int16_t *o_idx = idx ? idx + t0 * K : nullptr;
        __nv_bfloat16 *o_g = idx ? tg + t0 * K : nullptr, *o_u = idx ? tu + t0 * K : nullptr;
        __nv_bfloat16 *Uc = U + t0 * L.ldf;
        if (d.flags & MOC_FLAG_SELECT_2_OF_8) {
            // local mask: one thread per group of eight channels, no search
            const unsigned grid = (unsigned)std::min<int64_t>((n * (F / 8) + 255) / 256, (int64_t)sm_count() * 64);
            MOC_LAUNCH(KID_TC_SELECT_MASK, st,
                       (select_grouped_mask_kernel<<<grid, 256, 0, st>>>(G, L.ldf, Uc, L.ldf, n, F, o_idx, o_g, o_u)));
        } else {
            tc_select_launch(sel, G, L.ldf, Uc, L.ldf, n, F, K, o_idx, o_g, o_u, hint, status, st);
        }
        if ((rc = launch_ok()) != MOC_OK) return rc;
    }
    // (the fp32 gate values are dead by now: their buffer takes the partial outputs of a split contraction)
    return forward_tc_down(d, U, L.ldf, wd, out, status, st, G, (size_t)std::min<int64_t>(L.chunk, T) * L.ldf);
}

int small_batch_dx(const moc_ffn_desc &d, const __nv_bfloat16 *dG, const __nv_bfloat16 *dU, int ldf,
                   const __nv_bfloat16 *wg, const __nv_bfloat16 *wu, __nv_bfloat16 *gx, char *small, cudaStream_t st);

int backward_tc(const moc_ffn_desc &d, const __nv_bfloat16 *x, const __nv_bfloat16 *wg, const __nv_bfloat16 *wu,
                const __nv_bfloat16 *wd, const int16_t *idx, const __nv_bfloat16 *tg, const __nv_bfloat16 *tu,
                const __nv_bfloat16 *dout, __nv_bfloat16 *gx, __nv_bfloat16 *gwg, __nv_bfloat16 *gwu,
                __nv_bfloat16 *gwd, char *ws, cudaStream_t st, cudaEvent_t wgrad_done) {
    using namespace tc;
    const TcBackwardLayout L = tc_backward_layout(d);
    __nv_bfloat16 *Zp = reinterpret_cast<__nv_bfloat16 *>(ws + L.off_z);
    __nv_bfloat16 *dUp = reinterpret_cast<__nv_bfloat16 *>(ws + L.off_du);
    __nv_bfloat16 *dGp = reinterpret_cast<__nv_bfloat16 *>(ws + L.off_dg);
    const int F = d.d_ff, K = d.k, dm = d.d_model;
    const int64_t T = d.tokens;
    int *status = device_status_ptr();
    if (!status) return MOC_ERR_CUDA;
    int rc;
    // MoC 2:8: dG' and dU' are 2:4-sparse rows; grad_x can contract them on the sparse MMA (the element-wise kernel then
    // also writes them in compressed form).  With few output columns the shorter GEMM does not pay for that.
    const bool sparse_dx = gx && L.sp_bytes != 0 && sparse_mma_enabled() && dm >= 1024;

    // dZ = dD Wd^T (dense, bf16), then the element-wise step at the saved indices -> masked Z', dU', dG'
    {
        Params p;
        init_params(p);
        if (!map_k_major(&p.a_map[0], dout, T, dm, dm, BM) || !map_k_major(&p.b_map[0], wd, F, dm, dm, b_box_rows()))
            return MOC_ERR_CUDA;
        p.k_blocks = ceil_div(dm, BK);
        p.M = (int)T;
        p.N = F;
        p.m_tiles = ceil_div(T, BM);
        p.n_tiles = ceil_div(F, BN);
        p.c[0] = Zp;
        p.ldc[0] = L.ldf;
        p.status = status;
        MOC_LAUNCH(KID_TC_DZ_GEMM, st, (rc = launch_gemm<false, false, EPI_BF16>(p, st)));
        if (rc != MOC_OK) return rc;
        // one warp per token with the token's rows staged in shared memory while at least four such warps fit an
        // SM; else one CTA per token working in global memory
        const size_t sw_bytes = sample_warp_words(L.ldf, K) * sizeof(uint32_t);
        const int sw_per_sm = (int)std::min<size_t>((size_t)220 * 1024 / sw_bytes, 2 * kSampleMaxWarps);  // tokens in flight
        if (sw_per_sm >= 2 && F <= 65535) {
            // two warps per token unless that many tokens fit that one warp each already fills the SM
            const int team = sw_per_sm <= 12 ? 2 : 1;
            const int per_cta_max = kSampleMaxWarps / team;
            const int ctas_per_sm = (sw_per_sm + per_cta_max - 1) / per_cta_max, wpc = sw_per_sm / ctas_per_sm;
            const size_t smem = (size_t)wpc * sw_bytes;
            auto kern = team == 2 ? backward_sample_rows_warp_kernel<2> : backward_sample_rows_warp_kernel<1>;
            if ((rc = set_smem(kern, smem, 2048)) != MOC_OK) return rc;
            const unsigned grid = (unsigned)std::min<int64_t>((T + wpc - 1) / wpc, (int64_t)sm_count() * ctas_per_sm);
            MOC_LAUNCH(KID_TC_BWD_SAMPLE, st,
                       (kern<<<grid, wpc * team * 32, smem, st>>>(idx, tg, tu, T, K, F, L.ldf, Zp, dUp, dGp, status)));
        } else {
            const size_t smem = (size_t)K * 8;
            if ((rc = set_smem(backward_sample_rows_kernel, smem)) != MOC_OK) return rc;
            const unsigned grid = (unsigned)std::min<int64_t>(T, (int64_t)sm_count() * 8);
            MOC_LAUNCH(KID_TC_BWD_SAMPLE, st,
                       (backward_sample_rows_kernel<<<grid, 256, smem, st>>>(idx, tg, tu, T, K, F, L.ldf, Zp, dUp, dGp,
                                                                             status)));
        }
        if ((rc = launch_ok()) != MOC_OK) return rc;
    }
    // weight gradients: dWd = Z'^T dD, dWu = dU'^T x, dWg = dG'^T x   (Eqs. (bp-1), (bp-4)); contraction over tokens
    if (gwd || gwu || gwg) {
        Params p;
        init_params(p);
        if (!map_mn_major(&p.b_map[0], dout, T, dm, dm) || !map_mn_major(&p.b_map[1], x, T, dm, dm))
            return MOC_ERR_CUDA;
        int np = 0;
        auto add = [&](__nv_bfloat16 *dst, const __nv_bfloat16 *a, int bsel) {
            if (!dst) return true;
            if (!map_mn_major(&p.a_map[np], a, T, F, L.ldf)) return false;
            p.a_idx[np][0] = (int8_t)np;
            p.b_idx[np][0] = (int8_t)bsel;
            p.c[np] = dst;
            p.ldc[np] = dm;
            ++np;
            return true;
        };
        if (!add(gwd, Zp, 0) || !add(gwu, dUp, 1) || !add(gwg, dGp, 1)) return MOC_ERR_CUDA;
        p.num_problems = np;
        p.k_blocks = ceil_div(T, BK);
        p.M = d.d_ff_ld;  // padding rows read zeros from the maps and are written as zeros
        p.N = dm;
        p.m_tiles = ceil_div(d.d_ff_ld, BM);
        p.n_tiles = ceil_div(dm, BN);
        p.accumulate = (d.flags & MOC_FLAG_ACCUMULATE_WGRAD) ? 1 : 0;
        // long contraction, few tiles: the finer tile granularity of single CTAs fills the last wave better
        p.single_cta = 1;
        static const bool problem_major = [] {
            const char *e = getenv("MOC_FFN_WGRAD_ORDER");  // "m": the m-block-major order (comparisons)
            return !(e && strcmp(e, "m") == 0);
        }();
        p.problem_major = problem_major ? 1 : 0;
        p.status = status;
        MOC_LAUNCH(KID_TC_WGRAD_GEMM, st, (rc = launch_gemm<true, true, EPI_BF16>(p, st)));
        if (rc != MOC_OK) return rc;
    }
    // the weight gradients are complete in stream order here; the grad_x kernel that follows does not touch them
    if (wgrad_done && cudaEventRecord(wgrad_done, st) != cudaSuccess) return MOC_ERR_CUDA;
    // dX = dG' Wg + dU' Wu   (Eq. (bp-5)): one accumulator, two contraction segments
    if (sparse_dx) {
        // dG' and dU' rows are 2:4-sparse (the caller's promise): compress both, then one sparse GEMM over two segments.
        // Values a row holds beyond two per group of 4 are counted and reported as a broken promise.
        const SparseOperandLayout SL = sparse_operand_layout(T, F);
        __nv_bfloat16 *gc = reinterpret_cast<__nv_bfloat16 *>(ws + L.off_gc), *uc = reinterpret_cast<__nv_bfloat16 *>(ws + L.off_uc);
        uint32_t *gmeta = reinterpret_cast<uint32_t *>(ws + L.off_gmeta), *umeta = reinterpret_cast<uint32_t *>(ws + L.off_umeta);
        if ((rc = sparse_compress(dGp, T, F, L.ldf, SL, gc, gmeta, nullptr, 0, nullptr, st, status)) != MOC_OK) return rc;
        if ((rc = sparse_compress(dUp, T, F, L.ldf, SL, uc, umeta, nullptr, 0, nullptr, st, status)) != MOC_OK) return rc;
        const __nv_bfloat16 *comps[2] = {gc, uc};
        const uint32_t *metas[2] = {gmeta, umeta};
        const __nv_bfloat16 *bs[2] = {wg, wu};
        if ((rc = sparse_gemm_pair(T, dm, F, 2, comps, metas, SL, bs, dm, gx, dm, false, KID_TC_SP_DX_GEMM, status, st)) != MOC_OK)
            return rc;
    } else if (gx && L.small_bytes) {
        // a small batch: the weight-streaming kernel of the small-batch plan (a 256-row tile of tokens would leave
        // most SMs without work: d_model / 256 tiles in all)
        if ((rc = small_batch_dx(d, dGp, dUp, L.ldf, wg, wu, gx, ws + L.off_small, st)) != MOC_OK) return rc;
    } else if (gx) {
        Params p;
        init_params(p);
        if (!map_k_major(&p.a_map[0], dGp, T, F, L.ldf, BM) || !map_k_major(&p.a_map[1], dUp, T, F, L.ldf, BM) ||
            !map_mn_major(&p.b_map[0], wg, F, dm, dm) || !map_mn_major(&p.b_map[1], wu, F, dm, dm))
            return MOC_ERR_CUDA;
        p.k_blocks = ceil_div(F, BK);
        p.M = (int)T;
        p.N = dm;
        p.m_tiles = ceil_div(T, BM);
        p.n_tiles = ceil_div(dm, BN);
        p.status = status;
        if (L.split_bytes) {
            // a few hundred tokens: the two segments as two problems of the launch, fp32 partial outputs, added behind it
            float *partial = reinterpret_cast<float *>(ws + L.off_split);
            p.num_problems = 2;
            p.a_idx[1][0] = 1;
            p.b_idx[1][0] = 1;
            p.c[0] = partial;
            p.c[1] = partial + T * dm;
            p.ldc[0] = p.ldc[1] = dm;
            MOC_LAUNCH(KID_TC_DX_GEMM, st, (rc = launch_gemm<false, true, EPI_F32>(p, st)));
            if (rc != MOC_OK) return rc;
            if ((rc = launch_split_sum(partial, T, dm, gx, st)) != MOC_OK) return rc;
        } else {
            p.k_segments = 2;
            p.a_idx[0][1] = 1;
            p.b_idx[0][1] = 1;
            p.c[0] = gx;
            p.ldc[0] = dm;
            MOC_LAUNCH(KID_TC_DX_GEMM, st, (rc = launch_gemm<false, true, EPI_BF16>(p, st)));
            if (rc != MOC_OK) return rc;
        }
    }
    return MOC_OK;
}

// ---- decode plan (bf16, tokens <= 16) ------------------------------------------------------------------
struct DecodeLayout {
    int ldf, slices, parts, gemv_grid;
    size_t off_g, off_zb, off_mask, off_list, off_count, off_acc, off_cnt, total;
};

DecodeLayout decode_layout(const moc_ffn_desc &d) {
    DecodeLayout L{};
    L.ldf = (d.d_ff + 7) & ~7;
    L.slices = (d.d_model + dec::kSliceCols - 1) / dec::kSliceCols;
    // about two CTAs per SM in the down kernel; a CTA's share of the list is bounded by its shared arrays
    const int sms = tc::sm_count();
    L.parts = std::max(std::max(1, 2 * sms / L.slices), (d.d_ff + dec::kMaxPart - 1) / dec::kMaxPart);
    // GEMV kernels: two CTAs per SM, never more than 64 rows per CTA
    L.gemv_grid = std::max(std::max(1, std::min(2 * sms, (d.d_ff + 7) / 8)), (d.d_ff + 63) / 64);
    Carver c;
    L.off_g = c.take((size_t)d.tokens * L.ldf * sizeof(float));
    L.off_zb = c.take((size_t)((d.d_ff + 15) / 16) * 256 * sizeof(__nv_bfloat16));
    L.off_mask = c.take((size_t)d.tokens * ((d.d_ff + 31) / 32) * sizeof(uint32_t));  // per-token selection bitmaps
    L.off_list = c.take((size_t)(d.d_ff + 1) * sizeof(uint16_t));
    L.off_count = c.take(sizeof(int));
    L.off_acc = c.take((size_t)d.tokens * d.d_model * sizeof(float));
    L.off_cnt = c.take((size_t)(L.slices + 1) * sizeof(int));  // + arrivals of the select kernel
    L.total = c.off;
    return L;
}

bool use_small_batch_plan(const moc_ffn_desc &d);
bool small_batch_preferred(const moc_ffn_desc &d);

bool use_decode_plan(const moc_ffn_desc &d) {
    return !(d.flags & MOC_FLAG_SELECT_POST_SILU) && d.dtype == MOC_BF16 && d.tokens >= 1 && d.tokens <= 16 && d.d_model <= 256 * dec::kSliceCols &&
           !(use_small_batch_plan(d) && small_batch_preferred(d));
}

// Launch with programmatic stream serialization allowed: the kernel may become resident while its predecessor in
// the stream drains (every kernel launched this way calls pdl_wait before it touches global data).
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, unsigned block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

// ---- cooperative decode (bf16, one or two tokens, d_model <= 4096): one kernel, every SM keeps its channels ----
struct CoopLayout {
    int grid, unit, stages;
    size_t smem, off_hist, off_n, off_cand, off_acc, total;
};

// ok == false: the problem or the device does not admit the cooperative kernel (the four-kernel plan runs then)
CoopLayout coop_layout(const moc_ffn_desc &d, bool &ok) {
    CoopLayout L{};
    ok = false;
    static const bool off = [] {
        const char *e = getenv("MOC_FFN_DECODE");  // "chain": the four-kernel decode plan (comparisons, tests)
        return e && strcmp(e, "chain") == 0;
    }();
    if (off || d.dtype != MOC_BF16 || d.tokens < 1 || d.tokens > dc::kMaxTokens || d.d_model > dc::kMaxD) return L;
    static const int coop_ok = [] {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess) return 0;
        return v;
    }();
    if (!coop_ok) return L;
    const int T = (int)d.tokens, dm = d.d_model, F = d.d_ff;
    L.unit = (F % 8 == 0) ? 8 : 1;
    if ((d.flags & MOC_FLAG_SELECT_2_OF_8) && L.unit != 8) return L;
    const int units = (F + L.unit - 1) / L.unit;
    L.grid = std::min(tc::sm_count(), units);
    if (((units + L.grid - 1) / L.grid) * L.unit > dc::kMaxRows) return L;
    const size_t fixed = (size_t)T * dm * 2 + (size_t)2 * T * dc::kMaxRows * 4;
    const size_t budget = (size_t)216 * 1024;
    if (fixed + (size_t)4 * dm * 2 > budget) return L;
    // a multiple of the consumer warps: every stage is then always consumed by the same warp (see the kernel)
    L.stages = (int)std::min<size_t>(dc::kMaxStages, (budget - fixed) / ((size_t)dm * 2)) / dc::kConsumerWarps * dc::kConsumerWarps;
    if (L.stages < dc::kConsumerWarps) return L;
    L.smem = dc::smem_bytes(T, dm, L.stages);
    Carver c;
    L.off_hist = c.take((size_t)T * dc::kBins * sizeof(uint32_t));
    L.off_n = c.take((size_t)T * sizeof(uint32_t));
    L.off_cand = c.take((size_t)T * F * sizeof(uint2));
    L.off_acc = c.take((size_t)T * dm * sizeof(float));
    L.total = c.off;
    ok = true;
    return L;
}

template <int T>
int launch_coop(const dc::Params &prm, const CoopLayout &L, cudaStream_t st) {
    auto kern = dc::decode_coop_kernel<T>;
    int rc;
    if ((rc = set_smem(kern, L.smem, 8 * 1024)) != MOC_OK) return rc;
    // all CTAs must be resident at once (the launch would be refused otherwise); asked once per shared-memory size
    static std::mutex mu;
    static std::unordered_map<size_t, int> per_sm_of;
    int per_sm = 0;
    {
        std::lock_guard<std::mutex> lock(mu);
        auto it = per_sm_of.find(L.smem);
        if (it == per_sm_of.end()) {
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, dc::kThreads, L.smem) != cudaSuccess)
                return MOC_ERR_CUDA;
            per_sm_of[L.smem] = per_sm;
        } else {
            per_sm = it->second;
        }
    }
    if (per_sm < 1 || L.grid > per_sm * tc::sm_count()) return MOC_ERR_UNSUPPORTED;
    dc::Params local = prm;
    void *args[] = {&local};
    cudaError_t err = cudaSuccess;
    MOC_LAUNCH(KID_DEC_COOP, st,
               err = cudaLaunchCooperativeKernel(reinterpret_cast<void *>(kern), dim3(L.grid), dim3(dc::kThreads), args, L.smem, st));
    if (err != cudaSuccess) {  // refused: nothing ran, the four-kernel plan serves the call
        (void)cudaGetLastError();
        return MOC_ERR_UNSUPPORTED;
    }
    return launch_ok();
}

// rms_w != nullptr: the block form (x is the residual stream h: RMSNorm in front, h added behind)
int decode_coop(const moc_ffn_desc &d, const CoopLayout &L, const __nv_bfloat16 *x, const __nv_bfloat16 *wg,
                const __nv_bfloat16 *wu, const __nv_bfloat16 *wd, __nv_bfloat16 *out, char *wsp, cudaStream_t st,
                const __nv_bfloat16 *rms_w = nullptr, float rms_eps = 0.f, uint8_t *kept_out = nullptr) {
    int *status = device_status_ptr();
    if (!status) return MOC_ERR_CUDA;
    dc::Params prm{};
    prm.x = x;
    prm.wg = wg;
    prm.wu = wu;
    prm.wd = wd;
    prm.out = out;
    prm.T = (int)d.tokens;
    prm.d = d.d_model;
    prm.F = d.d_ff;
    prm.K = d.k;
    prm.grouped = (d.flags & MOC_FLAG_SELECT_2_OF_8) ? 1 : 0;
    prm.unit = L.unit;
    prm.stages = L.stages;
    prm.rms_w = rms_w;
    prm.rms_eps = rms_eps;
    prm.kept_out = kept_out;
    prm.hist = reinterpret_cast<uint32_t *>(wsp + L.off_hist);
    prm.cand_n = reinterpret_cast<uint32_t *>(wsp + L.off_n);
    prm.cand = reinterpret_cast<uint2 *>(wsp + L.off_cand);
    prm.acc = reinterpret_cast<float *>(wsp + L.off_acc);
    prm.status = status;
    switch (prm.T) {
        case 1: return launch_coop<1>(prm, L, st);
        case 2: return launch_coop<2>(prm, L, st);
        default: return MOC_ERR_UNSUPPORTED;
    }
}

// resid != nullptr: added to the layer's output before the rounding (the block form)
int decode_bf16(const moc_ffn_desc &d, const __nv_bfloat16 *x, const __nv_bfloat16 *wg, const __nv_bfloat16 *wu,
                const __nv_bfloat16 *wd, __nv_bfloat16 *out, char *wsp, cudaStream_t st,
                const __nv_bfloat16 *resid = nullptr) {
    const DecodeLayout L = decode_layout(d);
    const int T = (int)d.tokens, F = d.d_ff, K = d.k, dm = d.d_model;
    int *status = device_status_ptr();
    if (!status) return MOC_ERR_CUDA;
    dec::Workspace ws;
    ws.G = reinterpret_cast<float *>(wsp + L.off_g);
    ws.Zb = reinterpret_cast<__nv_bfloat16 *>(wsp + L.off_zb);
    ws.sel_bits = reinterpret_cast<uint32_t *>(wsp + L.off_mask);
    ws.sel_words = (F + 31) / 32;
    ws.list = reinterpret_cast<uint16_t *>(wsp + L.off_list);
    ws.list_count = reinterpret_cast<int *>(wsp + L.off_count);
    ws.out_acc = reinterpret_cast<float *>(wsp + L.off_acc);
    ws.counters = reinterpret_cast<int *>(wsp + L.off_cnt);
    ws.ldf = L.ldf;
    int rc;
    const size_t sel_smem = ((size_t)((F + 3) & ~3) + 2 * dec::kSelListCap) * sizeof(uint32_t);
    if ((rc = set_smem(dec::select_mask_kernel, sel_smem)) != MOC_OK) return rc;
    if ((rc = set_smem(dec::select_grouped_bits_kernel, sel_smem)) != MOC_OK) return rc;
    if ((rc = set_smem(dec::down_rows_kernel, dec::kDownSmem)) != MOC_OK) return rc;
    if ((rc = set_smem(dec::gemv_rows_kernel<false>, dec::kGemvSmem)) != MOC_OK) return rc;
    if ((rc = set_smem(dec::gemv_rows_kernel<true>, dec::kGemvSmem)) != MOC_OK) return rc;

    MOC_LAUNCH(KID_DEC_GATE_GEMV, st,
               launch_pdl(dec::gemv_rows_kernel<false>, dim3(L.gemv_grid), dec::kGemvThreads, dec::kGemvSmem, st, x, wg, T,
                          dm, F, ws, L.slices, status));
    if ((rc = launch_ok()) != MOC_OK) return rc;
    if (d.flags & MOC_FLAG_SELECT_2_OF_8) {
        MOC_LAUNCH(KID_DEC_SELECT, st,
                   launch_pdl(dec::select_grouped_bits_kernel, dim3(T), dec::kSelThreads, sel_smem, st, ws, F,
                              ws.counters + L.slices));
    } else {
        MOC_LAUNCH(KID_DEC_SELECT, st,
                   launch_pdl(dec::select_mask_kernel, dim3(T), dec::kSelThreads, sel_smem, st, ws, F, K,
                              ws.counters + L.slices, status));
    }
    if ((rc = launch_ok()) != MOC_OK) return rc;
    MOC_LAUNCH(KID_DEC_UP, st,
               launch_pdl(dec::gemv_rows_kernel<true>, dim3(L.gemv_grid), dec::kGemvThreads, dec::kGemvSmem, st, x, wu, T,
                          dm, F, ws, L.slices, status));
    if ((rc = launch_ok()) != MOC_OK) return rc;
    MOC_LAUNCH(KID_DEC_DOWN, st,
               launch_pdl(dec::down_rows_kernel, dim3(L.slices, L.parts), dec::kGemvThreads, dec::kDownSmem, st, wd, T, dm,
                          F, ws, out, resid, status));
    return launch_ok();
}

// ---- small-batch plan (bf16, up to 256 tokens): three weight-streaming tcgen05 kernels ----------------------
struct SmallBatchLayout {
    int ldf, ldz;
    int rows, ctas_per_matrix;                   // gate + up: channels per CTA, CTAs per weight matrix
    int accs, m_tiles, splits, k_blocks_down;    // down: 128 * accs columns per CTA, CTAs = m_tiles * splits
    bool stage_u;                                // the selector holds the token's up row in shared memory
    size_t off_g, off_u, off_z, off_acc, off_cnt, total;
};

// Grid of sb_down_kernel for `d_model` output columns and `k_blocks` channel blocks in all: about one CTA per SM,
// every CTA at least one channel block; 256-column blocks (accs = 2) when they still fill the GPU, else 128.
void down_geometry(int d_model, int k_blocks, int &accs, int &m_tiles, int &splits, int sms = 0) {
    if (sms <= 0) sms = tc::sm_count();
    auto ctas = [&](int a, int &mt, int &sp) {
        mt = (d_model + sb::kTile * a - 1) / (sb::kTile * a);
        sp = std::max(1, std::min(sms / mt, k_blocks));
        return mt * sp;
    };
    int m1, s1, m2, s2;
    const int c1 = ctas(1, m1, s1), c2 = ctas(2, m2, s2);
    const bool wide = d_model > sb::kTile && (c2 >= c1 || 20 * c2 >= 17 * sms);
    accs = wide ? 2 : 1;
    m_tiles = wide ? m2 : m1;
    splits = wide ? s2 : s1;
}

SmallBatchLayout small_batch_layout(const moc_ffn_desc &d) {
    SmallBatchLayout L{};
    const int sms = tc::sm_count();
    L.ldf = (d.d_ff + 7) & ~7;
    L.ldz = (d.d_ff + 7) & ~7;
    // gate + up: one CTA per SM, half of them per matrix
    const int per = std::max(1, sms / 2);
    L.rows = std::min(sb::kMaxRows, std::max(8, (((d.d_ff + per - 1) / per) + 7) & ~7));
    L.ctas_per_matrix = (d.d_ff + L.rows - 1) / L.rows;
    L.k_blocks_down = (d.d_ff + sb::kBK - 1) / sb::kBK;
    down_geometry(d.d_model, L.k_blocks_down, L.accs, L.m_tiles, L.splits);
    L.stage_u = sb::select_smem(d.d_ff, true) + 48 * 1024 <= (size_t)kMaxDynSmem;
    Carver c;
    L.off_g = c.take((size_t)d.tokens * L.ldf * sizeof(float));
    L.off_u = c.take((size_t)d.tokens * L.ldf * sizeof(float));
    L.off_z = c.take((size_t)d.tokens * L.ldz * sizeof(__nv_bfloat16));
    L.off_acc = c.take((size_t)d.tokens * d.d_model * sizeof(float));
    L.off_cnt = c.take((size_t)L.m_tiles * sizeof(int));
    L.total = c.off;
    return L;
}

// Which of the two small-batch forms reads fewer bytes: the decode plan reads W_gate and the rows of W_up / W_down
// that some token selected, (1 + 2 u) F d elements with u = 1 - (1 - K/F)^T the expected share of used channels; the
// small-batch plan reads all 3 F d but is one kernel without gathers.  Measured on the LLaMA-7B shape the two cross
// between 4 and 5 tokens at K = F/8 (58.3 / 63.4 us for the chain, 58.9 / 59.7 us for the one-kernel form), i.e. where u
// passes 0.45; from 17 tokens on only the small-batch plan exists.
// MOC_FFN_SB_MIN_TOKENS=n in the environment moves the boundary to n tokens (measurements only).
bool small_batch_preferred(const moc_ffn_desc &d) {
    static const int forced = [] {
        const char *e = getenv("MOC_FFN_SB_MIN_TOKENS");
        return e ? atoi(e) : 0;
    }();
    if (forced >= 1) return d.tokens >= forced;
    if (d.tokens > 16) return true;
    const double unused = std::pow(1.0 - (double)d.k / (double)d.d_ff, (double)d.tokens);
    return 1.0 - unused >= 0.45;
}

// moc_ffn_forward takes the small-batch plan for every bf16 batch it can serve (the tensor-core plan's tiles need
// thousands of tokens); moc_ffn_decode takes it where small_batch_preferred says so, else the decode plan.
bool use_small_batch_plan(const moc_ffn_desc &d) {
    return !(d.flags & MOC_FLAG_SELECT_POST_SILU) && d.dtype == MOC_BF16 && d.tokens >= 1 && d.tokens <= sb::kMaxTokens &&
           sb::select_smem(d.d_ff, false) + 48 * 1024 <= (size_t)kMaxDynSmem;
}

int small_batch_down(const moc_ffn_desc &d, const SmallBatchLayout &L, const sb::GemmShape &ds, const __nv_bfloat16 *wd,
                     const __nv_bfloat16 *Z, float *acc, int *counters, __nv_bfloat16 *out, const __nv_bfloat16 *resid,
                     int *status, cudaStream_t st);

// The overlapped form of the small-batch plan, for calls that keep nothing: the gate matrix is streamed by ALL SMs
// first, and the selection (one CTA per token, a dozen microseconds during which HBM would idle) then runs beside the
// kernel that streams the up matrix on the remaining SMs; that kernel's epilogue waits for the selection and forms the
// masked hidden state Z' from its accumulators, the gate values and the selection bitmaps.  Four kernels:
//   gate (all SMs) -> select (T CTAs, bitmaps only) || up + mask (SMs - ceil(T/2) CTAs) -> down.
// MOC_FFN_SB_OVERLAP=0 in the environment keeps the three-kernel form everywhere (comparisons); =n: up to n tokens.
bool small_batch_overlapped(const moc_ffn_desc &d, bool saving) {
    static const int limit = [] {
        const char *e = getenv("MOC_FFN_SB_OVERLAP");
        return e ? atoi(e) : 32;  // measured on the LLaMA-7B shape: 67 / 70 us against 70 / 72 us at 16 / 32 tokens, but 86 against 76 us at 64
    }();
    return !saving && !(d.flags & MOC_FLAG_SELECT_2_OF_8) && d.tokens <= limit && tc::sm_count() >= 32;
}

// channels per CTA when `ctas` CTAs share the F channels of one matrix: a multiple of 8, at most sb::kMaxRows
int sb_rows_for(int F, int ctas) {
    return std::min(sb::kMaxRows, std::max(8, (((F + ctas - 1) / ctas) + 7) & ~7));
}

int forward_small_batch_overlapped(const moc_ffn_desc &d, const SmallBatchLayout &L, const __nv_bfloat16 *x,
                                   const __nv_bfloat16 *wg, const __nv_bfloat16 *wu, const __nv_bfloat16 *wd,
                                   __nv_bfloat16 *out, char *wsp, cudaStream_t st, const __nv_bfloat16 *resid) {
    const int T = (int)d.tokens, F = d.d_ff, dm = d.d_model;
    int *status = device_status_ptr();
    if (!status) return MOC_ERR_CUDA;
    const int sms = tc::sm_count();
    // a selector CTA per SM (asking for more than half an SM's shared memory keeps a second one away: two of them on
    // one SM would halve each other's pace); the up kernel gets the other SMs
    const int sel_sms = std::min(T, sms / 2);
    const int rows_g = sb_rows_for(F, sms), rows_u = sb_rows_for(F, sms - sel_sms);
    const int ctas_g = (F + rows_g - 1) / rows_g, ctas_u = (F + rows_u - 1) / rows_u;
    const int boxes = 2;  // two 64-element blocks per stage: the CTAs' row counts are small here
    const sb::GemmShape gg = sb::gemm_shape(T, rows_g, boxes), gu = sb::gemm_shape(T, rows_u, boxes),
                        ds = sb::gemm_shape(T, sb::kTile * L.accs);
    if (gg.stages < 2 || gu.stages < 2 || ds.stages < 2) return MOC_ERR_UNSUPPORTED;
    float *G = reinterpret_cast<float *>(wsp + L.off_g);
    uint32_t *kept = reinterpret_cast<uint32_t *>(wsp + L.off_u);  // the bitmaps live where the three-kernel form keeps U
    const int kept_words = (F + 31) / 32;
    __nv_bfloat16 *Z = reinterpret_cast<__nv_bfloat16 *>(wsp + L.off_z);
    float *acc = reinterpret_cast<float *>(wsp + L.off_acc);
    int *counters = reinterpret_cast<int *>(wsp + L.off_cnt);
    int rc;
    const size_t sel_smem = std::max(sb::select_smem(F, false), (size_t)116 * 1024);
    if ((rc = set_smem(sb::sb_gate_up_kernel, std::max(gg.smem, gu.smem), 1024)) != MOC_OK) return rc;
    if ((rc = set_smem(sb::sb_down_kernel, ds.smem, 1024)) != MOC_OK) return rc;
    if ((rc = set_smem(sb::sb_select_kernel, sel_smem)) != MOC_OK) return rc;

    auto gate_up_params = [&](sb::GateUpParams &gp, const sb::GemmShape &gs, int rows, int ctas) {
        memset(&gp, 0, sizeof(gp));
        if (!tc::make_map(&gp.w_map[0], wg, F, dm, dm, sb::kBK, rows) ||
            !tc::make_map(&gp.w_map[1], wu, F, dm, dm, sb::kBK, rows) ||
            !tc::make_map(&gp.x_map, x, T, dm, dm, sb::kBK, gs.tn))
            return false;
        gp.T = T;
        gp.tn = gs.tn;
        gp.tmem_cols = gs.tmem_cols;
        gp.stages = gs.stages;
        gp.w_bytes = gs.w_bytes;
        gp.stage_bytes = gs.stage_bytes;
        gp.F = F;
        gp.boxes = boxes;
        gp.k_blocks = (dm + sb::kBK * boxes - 1) / (sb::kBK * boxes);
        gp.rows = rows;
        gp.ctas_per_matrix = ctas;
        gp.G = G;
        gp.ldf = L.ldf;
        gp.status = status;
        return true;
    };
    sb::GateUpParams gp;
    if (!gate_up_params(gp, gg, rows_g, ctas_g)) return MOC_ERR_CUDA;
    gp.counters = counters;
    gp.n_counters = L.m_tiles;
    MOC_LAUNCH(KID_SB_GATE_UP, st, launch_pdl(sb::sb_gate_up_kernel, dim3(ctas_g), sb::kThreads, gg.smem, st, gp));
    if ((rc = launch_ok()) != MOC_OK) return rc;

    sb::SelectParams sp{G, nullptr, L.ldf, F, d.k, dm, Z, L.ldz, acc, nullptr, nullptr, nullptr, 0, status, kept, kept_words};
    MOC_LAUNCH(KID_SB_SELECT, st, launch_pdl(sb::sb_select_kernel, dim3(T), dec::kSelThreads, sel_smem, st, sp));
    if ((rc = launch_ok()) != MOC_OK) return rc;

    sb::GateUpParams up;
    if (!gate_up_params(up, gu, rows_u, ctas_u)) return MOC_ERR_CUDA;
    up.prob0 = 1;
    up.mask_mode = 1;
    up.kept_bits = kept;
    up.kept_words = kept_words;
    up.Z = Z;
    up.ldz = L.ldz;
    MOC_LAUNCH(KID_SB_GATE_UP, st, launch_pdl(sb::sb_gate_up_kernel, dim3(ctas_u), sb::kThreads, gu.smem, st, up));
    if ((rc = launch_ok()) != MOC_OK) return rc;
    return small_batch_down(d, L, ds, wd, Z, acc, counters, out, resid, status, st);
}

// The one-kernel form of the small-batch plan (small_batch_fused.cuh), for calls of up to 32 tokens that keep nothing:
// T selector CTAs and SMs - T streamer CTAs in one cooperative launch.  ok == false: the problem or the device does not
// admit it (the multi-kernel forms run then).  MOC_FFN_SB_FUSED=0 in the environment switches it off (comparisons).
struct FusedLayout {
    int tn, n_stream, n_gu, rows, gu_boxes, gu_stages, accs, m_tiles, splits, stages;
    uint32_t w_pitch, slot_bytes, tail_off;
    size_t smem;
};

FusedLayout fused_layout(const moc_ffn_desc &d, bool saving, bool &ok) {
    FusedLayout L{};
    ok = false;
    static const bool off = [] {
        const char *e = getenv("MOC_FFN_SB_FUSED");
        return e && atoi(e) == 0;
    }();
    static const int coop_ok = [] {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess) return 0;
        return v;
    }();
    const int T = (int)d.tokens, F = d.d_ff, dm = d.d_model, sms = tc::sm_count();
    const bool grouped = (d.flags & MOC_FLAG_SELECT_2_OF_8) != 0;  // local mask: no selector CTAs
    if (off || !coop_ok || saving || T < 1 || T > sbf::kMaxTokens || sms < 4 * T || (grouped && F % 8 != 0)) return L;
    L.n_stream = grouped ? sms : sms - T;
    L.tn = T <= 16 ? 16 : 32;
    const uint32_t xbox = (uint32_t)L.tn * sb::kBK * 2;
    L.rows = (F + L.n_stream - 1) / L.n_stream;
    if (L.rows > sb::kTile || grouped) L.rows = (L.rows + 7) & ~7;  // the second MMA tile starts at a whole swizzle group; whole groups of 8
    if (L.rows > sb::kMaxRows) return L;
    L.n_gu = (F + L.rows - 1) / L.rows;
    L.w_pitch = ((uint32_t)L.rows * sb::kBK * 2 + 1023u) & ~1023u;
    down_geometry(dm, (F + sb::kBK - 1) / sb::kBK, L.accs, L.m_tiles, L.splits, L.n_stream);
    if (L.m_tiles > L.n_stream) return L;
    // a stage of phases G and U holds as many 64-element blocks as make it about the size of a stage of phase D (the
    // ring's slots have one size): few large stages keep more bytes in flight than many small ones that leave slots half used
    const uint32_t d_slot = (uint32_t)L.accs * 16384u + xbox, gu_box = xbox + L.w_pitch;
    static const int forced_boxes = [] {
        const char *e = getenv("MOC_FFN_SB_FUSED_BOXES");
        return e ? atoi(e) : 0;
    }();
    L.gu_boxes = forced_boxes > 0 ? forced_boxes : std::max(1, std::min(8, (int)((d_slot + gu_box / 2) / gu_box)));
    L.gu_stages = (dm + L.gu_boxes * sb::kBK - 1) / (L.gu_boxes * sb::kBK);
    const uint32_t gu_slot = (uint32_t)L.gu_boxes * gu_box;
    L.slot_bytes = std::max(gu_slot, d_slot);
    // behind the ring: the gate values and the barriers, and at least as many bytes as an MMA over a short weight box
    // reads past the ring's end (it always reads 128 rows)
    const uint32_t past = (uint32_t)L.gu_boxes * xbox + (uint32_t)(L.gu_boxes - 1) * L.w_pitch + (uint32_t)sb::kTile * sb::kBK * 2;
    const uint32_t tail = std::max<uint32_t>((uint32_t)sbf::kTn * L.rows * 4 + 512, past > L.slot_bytes ? past - L.slot_bytes : 0);
    const size_t budget = (size_t)kMaxDynSmem - 2048 /*static state of the selector role*/ - 1024 /*alignment*/;
    if (tail + 2 * (size_t)L.slot_bytes > budget) return L;
    L.stages = (int)std::min<size_t>(sbf::kStagesMax, (budget - tail) / L.slot_bytes);
    L.tail_off = (uint32_t)L.stages * L.slot_bytes;
    L.smem = std::max((size_t)1024 + L.tail_off + tail, sbf::selector_smem(F));
    if (L.smem + 2048 > (size_t)kMaxDynSmem) return L;
    ok = true;
    return L;
}

int forward_small_batch_fused(const moc_ffn_desc &d, const SmallBatchLayout &L, const FusedLayout &FL, const __nv_bfloat16 *x,
                              const __nv_bfloat16 *wg, const __nv_bfloat16 *wu, const __nv_bfloat16 *wd, __nv_bfloat16 *out,
                              char *wsp, cudaStream_t st, const __nv_bfloat16 *resid, long long wait_limit = tc::kWaitLimitCycles,
                              int stall = 0, const __nv_bfloat16 *rms_h = nullptr, const __nv_bfloat16 *rms_w = nullptr,
                              float rms_eps = 0.f) {
    const int T = (int)d.tokens, F = d.d_ff, dm = d.d_model;
    int *status = device_status_ptr();
    if (!status) return MOC_ERR_CUDA;
    int rc;
    const bool grouped = (d.flags & MOC_FLAG_SELECT_2_OF_8) != 0;
    void (*const kern)(sbf::FusedParams) = grouped ? sbf::sb_fused_kernel<true> : sbf::sb_fused_kernel<false>;
    if ((rc = set_smem(kern, FL.smem, 2048)) != MOC_OK) return rc;
    // all CTAs must be resident at once (the launch would be refused otherwise); asked once per form and shared-memory size
    static std::mutex mu;
    static std::unordered_map<size_t, int> per_sm_of;
    int per_sm = 0;
    {
        std::lock_guard<std::mutex> lock(mu);
        auto it = per_sm_of.find(2 * FL.smem + (grouped ? 1 : 0));
        if (it == per_sm_of.end()) {
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, sbf::kBlock, FL.smem) != cudaSuccess)
                return MOC_ERR_CUDA;
            per_sm_of[2 * FL.smem + (grouped ? 1 : 0)] = per_sm;
        } else {
            per_sm = it->second;
        }
    }
    if (per_sm < 1) return MOC_ERR_UNSUPPORTED;
    sbf::FusedParams fp;
    memset(&fp, 0, sizeof(fp));
    __nv_bfloat16 *Z = reinterpret_cast<__nv_bfloat16 *>(wsp + L.off_z);
    if (!tc::make_map(&fp.wg_map, wg, F, dm, dm, sb::kBK, FL.rows) || !tc::make_map(&fp.wu_map, wu, F, dm, dm, sb::kBK, FL.rows) ||
        !tc::make_map(&fp.x_map, x, T, dm, dm, sb::kBK, FL.tn) || !tc::make_map(&fp.wd_map, wd, F, dm, dm, 64, sb::kBK) ||
        !tc::make_map(&fp.z_map, Z, T, F, L.ldz, sb::kBK, FL.tn))
        return MOC_ERR_CUDA;
    fp.T = T;
    fp.F = F;
    fp.K = d.k;
    fp.d = dm;
    fp.tn = FL.tn;
    fp.grouped = grouped ? 1 : 0;
    fp.n_stream = FL.n_stream;
    fp.n_gu = FL.n_gu;
    fp.rows = FL.rows;
    fp.w_pitch = FL.w_pitch;
    fp.gu_boxes = FL.gu_boxes;
    fp.gu_stages = FL.gu_stages;
    fp.accs = FL.accs;
    fp.m_tiles = FL.m_tiles;
    fp.splits = FL.splits;
    fp.kb_down = (F + sb::kBK - 1) / sb::kBK;
    fp.slot_bytes = FL.slot_bytes;
    fp.stages = FL.stages;
    fp.tail_off = FL.tail_off;
    fp.G = reinterpret_cast<float *>(wsp + L.off_g);
    fp.ldf = L.ldf;
    fp.kept_bits = reinterpret_cast<uint32_t *>(wsp + L.off_u);  // the bitmaps live where the three-kernel form keeps U
    fp.kept_words = (F + 31) / 32;
    fp.Z = Z;
    fp.ldz = L.ldz;
    fp.acc = reinterpret_cast<float *>(wsp + L.off_acc);
    fp.out = out;
    fp.resid = resid;
    unsigned int *state = fused_state_for(wsp);
    if (!state || FL.m_tiles > sbf::kStateCounters) return MOC_ERR_UNSUPPORTED;
    fp.counters = reinterpret_cast<int *>(state);
    fp.flags = state + sbf::kStateCounters;
    fp.status = status;
    fp.wait_limit = wait_limit;
    fp.stall = stall;
    if (rms_w) {  // x is where the selector CTAs will write RMSNorm(rms_h)
        if (grouped) return MOC_ERR_UNSUPPORTED;
        fp.rms_h = rms_h;
        fp.rms_w = rms_w;
        fp.rms_eps = rms_eps;
        fp.xn = const_cast<__nv_bfloat16 *>(x);
    }
    // cooperative, and allowed to become resident while the previous kernel in the stream drains (the kernel waits for
    // that kernel's completion before it touches anything but the weights); a driver that refuses the combination gets
    // the plain cooperative launch from then on
    static std::atomic<int> pdl_ok{1};
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(FL.n_stream + (fp.grouped ? 0 : T));
    cfg.blockDim = dim3(sbf::kBlock);
    cfg.dynamicSmemBytes = FL.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    void *args[] = {&fp};
    cudaError_t err = cudaErrorUnknown;
    if (pdl_ok.load(std::memory_order_relaxed)) {
        cfg.numAttrs = 2;
        MOC_LAUNCH(KID_SB_FUSED, st, err = cudaLaunchKernelExC(&cfg, reinterpret_cast<const void *>(kern), args));
        if (err != cudaSuccess) {
            (void)cudaGetLastError();
            pdl_ok.store(0, std::memory_order_relaxed);
        }
    }
    if (err != cudaSuccess) {
        cfg.numAttrs = 1;
        MOC_LAUNCH(KID_SB_FUSED, st, err = cudaLaunchKernelExC(&cfg, reinterpret_cast<const void *>(kern), args));
    }
    if (err != cudaSuccess) {  // the launch was refused (SMs reserved by others, ...): nothing ran, the multi-kernel forms serve the call
        (void)cudaGetLastError();
        return MOC_ERR_UNSUPPORTED;
    }
    return launch_ok();
}

int forward_small_batch(const moc_ffn_desc &d, const __nv_bfloat16 *x, const __nv_bfloat16 *wg,
                        const __nv_bfloat16 *wu, const __nv_bfloat16 *wd, __nv_bfloat16 *out, int16_t *idx,
                        __nv_bfloat16 *tg, __nv_bfloat16 *tu, char *wsp, cudaStream_t st,
                        const __nv_bfloat16 *resid = nullptr) {
    const SmallBatchLayout L = small_batch_layout(d);
    const int T = (int)d.tokens, F = d.d_ff, dm = d.d_model;
    int *status = device_status_ptr();
    if (!status) return MOC_ERR_CUDA;
    const sb::GemmShape gs = sb::gemm_shape(T, L.rows), ds = sb::gemm_shape(T, sb::kTile * L.accs);
    if (gs.stages < 2 || ds.stages < 2) return MOC_ERR_UNSUPPORTED;
    float *G = reinterpret_cast<float *>(wsp + L.off_g), *U = reinterpret_cast<float *>(wsp + L.off_u);
    __nv_bfloat16 *Z = reinterpret_cast<__nv_bfloat16 *>(wsp + L.off_z);
    float *acc = reinterpret_cast<float *>(wsp + L.off_acc);
    int *counters = reinterpret_cast<int *>(wsp + L.off_cnt);
    int rc;
    const size_t sel_smem = sb::select_smem(F, L.stage_u);
    if ((rc = set_smem(sb::sb_gate_up_kernel, gs.smem, 1024)) != MOC_OK) return rc;
    if ((rc = set_smem(sb::sb_down_kernel, ds.smem, 1024)) != MOC_OK) return rc;
    if ((rc = set_smem(sb::sb_select_kernel, sel_smem)) != MOC_OK) return rc;

    {
        bool fused_ok = false;
        const FusedLayout FL = fused_layout(d, idx != nullptr, fused_ok);
        if (fused_ok) {
            rc = forward_small_batch_fused(d, L, FL, x, wg, wu, wd, out, wsp, st, resid);
            if (rc != MOC_ERR_UNSUPPORTED) return rc;
        }
    }
    if (small_batch_overlapped(d, idx != nullptr))
        return forward_small_batch_overlapped(d, L, x, wg, wu, wd, out, wsp, st, resid);

    sb::GateUpParams gp;
    memset(&gp, 0, sizeof(gp));
    if (!tc::make_map(&gp.w_map[0], wg, F, dm, dm, sb::kBK, L.rows) ||
        !tc::make_map(&gp.w_map[1], wu, F, dm, dm, sb::kBK, L.rows) ||
        !tc::make_map(&gp.x_map, x, T, dm, dm, sb::kBK, gs.tn))
        return MOC_ERR_CUDA;
    gp.T = T;
    gp.tn = gs.tn;
    gp.tmem_cols = gs.tmem_cols;
    gp.stages = gs.stages;
    gp.w_bytes = gs.w_bytes;
    gp.stage_bytes = gs.stage_bytes;
    gp.F = F;
    gp.k_blocks = (dm + sb::kBK - 1) / sb::kBK;
    gp.rows = L.rows;
    gp.boxes = 1;
    gp.ctas_per_matrix = L.ctas_per_matrix;
    gp.G = G;
    gp.U = U;
    gp.ldf = L.ldf;
    gp.counters = counters;
    gp.n_counters = L.m_tiles;
    gp.status = status;
    MOC_LAUNCH(KID_SB_GATE_UP, st,
               launch_pdl(sb::sb_gate_up_kernel, dim3(2 * L.ctas_per_matrix), sb::kThreads, gs.smem, st, gp));
    if ((rc = launch_ok()) != MOC_OK) return rc;

    sb::SelectParams sp{G, U, L.ldf, F, d.k, dm, Z, L.ldz, acc, idx, tg, tu, L.stage_u ? 1 : 0, status, nullptr, 0};
    if (d.flags & MOC_FLAG_SELECT_2_OF_8) {
        MOC_LAUNCH(KID_SB_SELECT, st,
                   launch_pdl(sb::sb_select_grouped_kernel, dim3(T), dec::kSelThreads, 0, st, sp));
    } else {
        MOC_LAUNCH(KID_SB_SELECT, st, launch_pdl(sb::sb_select_kernel, dim3(T), dec::kSelThreads, sel_smem, st, sp));
    }
    if ((rc = launch_ok()) != MOC_OK) return rc;

    return small_batch_down(d, L, ds, wd, Z, acc, counters, out, resid, status, st);
}

// D = Z' W_down of the small-batch plan (both forms end with it)
int small_batch_down(const moc_ffn_desc &d, const SmallBatchLayout &L, const sb::GemmShape &ds, const __nv_bfloat16 *wd,
                     const __nv_bfloat16 *Z, float *acc, int *counters, __nv_bfloat16 *out, const __nv_bfloat16 *resid,
                     int *status, cudaStream_t st) {
    const int T = (int)d.tokens, F = d.d_ff, dm = d.d_model;
    sb::DownParams dp;
    memset(&dp, 0, sizeof(dp));
    if (!tc::make_map(&dp.wd_map[0], wd, F, dm, dm, 64, sb::kBK) ||
        !tc::make_map(&dp.z_map[0], Z, T, F, L.ldz, sb::kBK, ds.tn))
        return MOC_ERR_CUDA;
    dp.segments = 1;
    dp.T = T;
    dp.tn = ds.tn;
    dp.tmem_cols = ds.tmem_cols;
    dp.stages = ds.stages;
    dp.w_bytes = ds.w_bytes;
    dp.stage_bytes = ds.stage_bytes;
    dp.d = dm;
    dp.k_blocks = L.k_blocks_down;
    dp.m_tiles = L.m_tiles;
    dp.splits = L.splits;
    dp.accs = L.accs;
    dp.acc = acc;
    dp.out = out;
    dp.resid = resid;
    dp.counters = counters;
    dp.status = status;
    MOC_LAUNCH(KID_SB_DOWN, st,
               launch_pdl(sb::sb_down_kernel, dim3(L.m_tiles * L.splits), sb::kThreads, ds.smem, st, dp));
    return launch_ok();
}

// dX = dG' Wg + dU' Wu for a small batch with sb_down_kernel: two contraction segments into one accumulator.
// `small`: T * d floats (the accumulator) followed by the column blocks' counters; both are cleared here.
int small_batch_dx(const moc_ffn_desc &d, const __nv_bfloat16 *dG, const __nv_bfloat16 *dU, int ldf,
                   const __nv_bfloat16 *wg, const __nv_bfloat16 *wu, __nv_bfloat16 *gx, char *small, cudaStream_t st) {
    const int T = (int)d.tokens, F = d.d_ff, dm = d.d_model;
    int *status = device_status_ptr();
    if (!status) return MOC_ERR_CUDA;
    const size_t acc_bytes = (size_t)T * dm * sizeof(float);
    float *acc = reinterpret_cast<float *>(small);
    int *counters = reinterpret_cast<int *>(small + acc_bytes);
    const int k_blocks = (F + sb::kBK - 1) / sb::kBK;
    int accs, m_tiles, splits;
    down_geometry(dm, 2 * k_blocks, accs, m_tiles, splits);
    if ((size_t)m_tiles * sizeof(int) > 1024) return MOC_ERR_UNSUPPORTED;
    const sb::GemmShape ds = sb::gemm_shape(T, sb::kTile * accs);
    if (ds.stages < 2) return MOC_ERR_UNSUPPORTED;
    int rc;
    if ((rc = set_smem(sb::sb_down_kernel, ds.smem, 1024)) != MOC_OK) return rc;
    if (cudaMemsetAsync(small, 0, acc_bytes + (size_t)m_tiles * sizeof(int), st) != cudaSuccess) return MOC_ERR_CUDA;
    sb::DownParams dp;
    memset(&dp, 0, sizeof(dp));
    if (!tc::make_map(&dp.wd_map[0], wg, F, dm, dm, 64, sb::kBK) || !tc::make_map(&dp.wd_map[1], wu, F, dm, dm, 64, sb::kBK) ||
        !tc::make_map(&dp.z_map[0], dG, T, F, ldf, sb::kBK, ds.tn) || !tc::make_map(&dp.z_map[1], dU, T, F, ldf, sb::kBK, ds.tn))
        return MOC_ERR_CUDA;
    dp.segments = 2;
    dp.T = T;
    dp.tn = ds.tn;
    dp.tmem_cols = ds.tmem_cols;
    dp.stages = ds.stages;
    dp.w_bytes = ds.w_bytes;
    dp.stage_bytes = ds.stage_bytes;
    dp.d = dm;
    dp.k_blocks = k_blocks;
    dp.m_tiles = m_tiles;
    dp.splits = splits;
    dp.accs = accs;
    dp.acc = acc;
    dp.out = gx;
    dp.counters = counters;
    dp.status = status;
    MOC_LAUNCH(KID_TC_DX_GEMM, st, (sb::sb_down_kernel<<<m_tiles * splits, sb::kThreads, ds.smem, st>>>(dp)));
    return launch_ok();
}

}  // namespace
}  // namespace moc

using namespace moc;

// =====================================================================================================
extern "C" {

// The block form runs on the three weight-streaming plans for small bf16 batches.
static bool block_form_supported(const moc_ffn_desc &d) {
    return d.dtype == MOC_BF16 && d.tokens >= 1 && d.tokens <= sb::kMaxTokens && d.d_model % 8 == 0 &&
           (use_decode_plan(d) || use_small_batch_plan(d));
}

size_t moc_ffn_workspace_bytes(const moc_ffn_desc *desc, int op) {
    if (check_desc(desc) != MOC_OK) return 0;
    if (desc->tokens == 0) return 0;
    switch (op) {
        case MOC_OP_DECODE:
            if (desc->tokens > sb::kMaxTokens) return 0;
            if (use_decode_plan(*desc)) {
                bool coop = false;
                const CoopLayout C = coop_layout(*desc, coop);
                return std::max(decode_layout(*desc).total, coop ? C.total : (size_t)0);
            }
            // fall through: the forward with nothing saved
        case MOC_OP_FORWARD:
            if (use_small_batch_plan(*desc)) return small_batch_layout(*desc).total;
            return use_tc_forward(*desc) ? tc::tc_forward_layout(*desc).total : plan_forward(*desc).total;
        case MOC_OP_BACKWARD:
            return use_tc_plan(*desc) ? tc::tc_backward_layout(*desc).total : plan_backward(*desc).total;
        case MOC_OP_DECODE_BLOCK: {
            // the decode workspace followed by the normalised activations [tokens, d_model]
            if (!block_form_supported(*desc)) return 0;
            return align_up(moc_ffn_workspace_bytes(desc, MOC_OP_DECODE), 256) +
                   align_up((size_t)desc->tokens * desc->d_model * sizeof(__nv_bfloat16), 256);
        }
        default:
            return 0;
    }
}

size_t moc_ffn_saved_bytes_per_token(const moc_ffn_desc *desc) {
    if (check_desc(desc) != MOC_OK) return 0;
    return (size_t)desc->k * (sizeof(int16_t) + 2 * esize(desc->dtype));
}

int moc_ffn_forward(const moc_ffn_desc *desc, const void *x, const void *w_gate, const void *w_up,
                    const void *w_down, void *out, int16_t *topk_idx, void *topk_gate, void *topk_up,
                    void *workspace, size_t workspace_bytes, void *cuda_stream) {
    int rc = check_desc(desc);
    if (rc != MOC_OK) return rc;
    const bool save_all = topk_idx && topk_gate && topk_up;
    const bool save_none = !topk_idx && !topk_gate && !topk_up;
    if (!save_all && !save_none) return MOC_ERR_INVALID_ARG;
    if (desc->tokens == 0) return MOC_OK;
    if (!good_ptr(x) || !good_ptr(w_gate) || !good_ptr(w_up) || !good_ptr(w_down) || !good_ptr(out))
        return MOC_ERR_INVALID_ARG;
    if (save_all && (!aligned16(topk_idx) || !aligned16(topk_gate) || !aligned16(topk_up)))
        return MOC_ERR_INVALID_ARG;
    const size_t need = moc_ffn_workspace_bytes(desc, MOC_OP_FORWARD);
    if (need && (!good_ptr(workspace) || workspace_bytes < need)) return MOC_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char *ws = static_cast<char *>(workspace);
    if (desc->dtype == MOC_BF16) {
        using T = __nv_bfloat16;
        if (use_small_batch_plan(*desc))
            return forward_small_batch(*desc, (const T *)x, (const T *)w_gate, (const T *)w_up, (const T *)w_down,
                                       (T *)out, topk_idx, (T *)topk_gate, (T *)topk_up, ws, st);
        if (use_tc_forward(*desc))
            return forward_tc(*desc, (const T *)x, (const T *)w_gate, (const T *)w_up, (const T *)w_down, (T *)out,
                              topk_idx, (T *)topk_gate, (T *)topk_up, ws, st);
        return forward_gather<T>(*desc, (const T *)x, (const T *)w_gate, (const T *)w_up, (const T *)w_down,
                                 (T *)out, topk_idx, (T *)topk_gate, (T *)topk_up, ws, st);
    }
    return forward_gather<float>(*desc, (const float *)x, (const float *)w_gate, (const float *)w_up,
                                 (const float *)w_down, (float *)out, topk_idx, (float *)topk_gate,
                                 (float *)topk_up, ws, st);
}

int moc_ffn_backward(const moc_ffn_desc *desc, const void *x, const void *w_gate, const void *w_up,
                     const void *w_down, const int16_t *topk_idx, const void *topk_gate, const void *topk_up,
                     const void *grad_out, void *grad_x, void *grad_w_gate, void *grad_w_up, void *grad_w_down,
                     void *workspace, size_t workspace_bytes, void *cuda_stream) {
    return moc_ffn_backward_overlap(desc, x, w_gate, w_up, w_down, topk_idx, topk_gate, topk_up, grad_out, grad_x,
                                    grad_w_gate, grad_w_up, grad_w_down, workspace, workspace_bytes, cuda_stream, nullptr);
}

int moc_ffn_backward_overlap(const moc_ffn_desc *desc, const void *x, const void *w_gate, const void *w_up,
                             const void *w_down, const int16_t *topk_idx, const void *topk_gate, const void *topk_up,
                             const void *grad_out, void *grad_x, void *grad_w_gate, void *grad_w_up,
                             void *grad_w_down, void *workspace, size_t workspace_bytes, void *cuda_stream,
                             void *wgrad_done_event) {
    cudaEvent_t wgrad_done = static_cast<cudaEvent_t>(wgrad_done_event);
    int rc = check_desc(desc);
    if (rc != MOC_OK) return rc;
    if (desc->tokens == 0) {
        // no tokens: weight gradients are zero unless they accumulate
        if (desc->flags & MOC_FLAG_ACCUMULATE_WGRAD) return MOC_OK;
        cudaStream_t st0 = static_cast<cudaStream_t>(cuda_stream);
        const size_t wbytes = (size_t)desc->d_ff_ld * desc->d_model * esize(desc->dtype);
        void *gw[3] = {grad_w_gate, grad_w_up, grad_w_down};
        for (void *g : gw) {
            if (g && !aligned16(g)) return MOC_ERR_INVALID_ARG;
        }
        for (void *g : gw) {
            if (g && cudaMemsetAsync(g, 0, wbytes, st0) != cudaSuccess) return MOC_ERR_CUDA;
        }
        if (wgrad_done && cudaEventRecord(wgrad_done, st0) != cudaSuccess) return MOC_ERR_CUDA;
        return MOC_OK;
    }
    if (!good_ptr(x) || !good_ptr(w_gate) || !good_ptr(w_up) || !good_ptr(w_down) || !good_ptr(topk_idx) ||
        !good_ptr(topk_gate) || !good_ptr(topk_up) || !good_ptr(grad_out))
        return MOC_ERR_INVALID_ARG;
    if (!aligned16(grad_x) || !aligned16(grad_w_gate) || !aligned16(grad_w_up) || !aligned16(grad_w_down))
        return MOC_ERR_INVALID_ARG;
    if (!grad_x && !grad_w_gate && !grad_w_up && !grad_w_down) {
        if (wgrad_done && cudaEventRecord(wgrad_done, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
            return MOC_ERR_CUDA;
        return MOC_OK;
    }
    const size_t need = moc_ffn_workspace_bytes(desc, MOC_OP_BACKWARD);
    if (need && (!good_ptr(workspace) || workspace_bytes < need)) return MOC_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char *ws = static_cast<char *>(workspace);
    if (desc->dtype == MOC_BF16) {
        using T = __nv_bfloat16;
        if (use_tc_plan(*desc))
            return backward_tc(*desc, (const T *)x, (const T *)w_gate, (const T *)w_up, (const T *)w_down, topk_idx,
                               (const T *)topk_gate, (const T *)topk_up, (const T *)grad_out, (T *)grad_x,
                               (T *)grad_w_gate, (T *)grad_w_up, (T *)grad_w_down, ws, st, wgrad_done);
        return backward_gather<T>(*desc, (const T *)x, (const T *)w_gate, (const T *)w_up, (const T *)w_down,
                                  topk_idx, (const T *)topk_gate, (const T *)topk_up, (const T *)grad_out,
                                  (T *)grad_x, (T *)grad_w_gate, (T *)grad_w_up, (T *)grad_w_down, ws, st, wgrad_done);
    }
    using T = float;
    return backward_gather<T>(*desc, (const T *)x, (const T *)w_gate, (const T *)w_up, (const T *)w_down,
                              topk_idx, (const T *)topk_gate, (const T *)topk_up, (const T *)grad_out,
                              (T *)grad_x, (T *)grad_w_gate, (T *)grad_w_up, (T *)grad_w_down, ws, st, wgrad_done);
}

int moc_ffn_decode(const moc_ffn_desc *desc, const void *x, const void *w_gate, const void *w_up,
                   const void *w_down, void *out, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    int rc = check_desc(desc);
    if (rc != MOC_OK) return rc;
    if (desc->tokens > sb::kMaxTokens) return MOC_ERR_UNSUPPORTED;
    if (!use_decode_plan(*desc))  // more than 16 tokens, or fp32 storage: the forward with nothing saved
        return moc_ffn_forward(desc, x, w_gate, w_up, w_down, out, nullptr, nullptr, nullptr, workspace,
                               workspace_bytes, cuda_stream);
    if (!good_ptr(x) || !good_ptr(w_gate) || !good_ptr(w_up) || !good_ptr(w_down) || !good_ptr(out))
        return MOC_ERR_INVALID_ARG;
    const size_t need = moc_ffn_workspace_bytes(desc, MOC_OP_DECODE);
    if (!good_ptr(workspace) || workspace_bytes < need) return MOC_ERR_WORKSPACE;
    using T = __nv_bfloat16;
    {
        // a handful of tokens: one cooperative kernel; where the device or the problem does not admit it, or its
        // launch is refused, the four-kernel plan
        bool coop = false;
        const CoopLayout C = coop_layout(*desc, coop);
        if (coop) {
            const int rc2 = decode_coop(*desc, C, (const T *)x, (const T *)w_gate, (const T *)w_up, (const T *)w_down,
                                        (T *)out, static_cast<char *>(workspace), static_cast<cudaStream_t>(cuda_stream));
            if (rc2 != MOC_ERR_UNSUPPORTED) return rc2;
        }
    }
    return decode_bf16(*desc, (const T *)x, (const T *)w_gate, (const T *)w_up, (const T *)w_down, (T *)out,
                       static_cast<char *>(workspace), static_cast<cudaStream_t>(cuda_stream));
}

int moc_ffn_decode_block(const moc_ffn_desc *desc, const void *h, const void *rms_weight, float rms_eps,
                         const void *w_gate, const void *w_up, const void *w_down, void *out, void *workspace,
                         size_t workspace_bytes, void *cuda_stream) {
    int rc = check_desc(desc);
    if (rc != MOC_OK) return rc;
    if (desc->tokens == 0) return MOC_OK;
    if (!block_form_supported(*desc)) return MOC_ERR_UNSUPPORTED;
    if (!good_ptr(h) || !good_ptr(rms_weight) || !good_ptr(w_gate) || !good_ptr(w_up) || !good_ptr(w_down) ||
        !good_ptr(out) || !(rms_eps >= 0.f))
        return MOC_ERR_INVALID_ARG;
    const size_t need = moc_ffn_workspace_bytes(desc, MOC_OP_DECODE_BLOCK);
    if (!good_ptr(workspace) || workspace_bytes < need) return MOC_ERR_WORKSPACE;
    using T = __nv_bfloat16;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char *wsp = static_cast<char *>(workspace);
    if (use_decode_plan(*desc)) {
        // one or two tokens: the cooperative kernel normalises its staged rows and adds h itself
        bool coop = false;
        const CoopLayout C = coop_layout(*desc, coop);
        if (coop) {
            const int rc2 = decode_coop(*desc, C, (const T *)h, (const T *)w_gate, (const T *)w_up, (const T *)w_down,
                                        (T *)out, wsp, st, (const T *)rms_weight, rms_eps);
            if (rc2 != MOC_ERR_UNSUPPORTED) return rc2;
        }
    }
    // otherwise a small kernel writes RMSNorm(h) behind the decode workspace, the plan's first kernel reads it as
    // its x, and the plan's last step adds h before it rounds
    T *xn = reinterpret_cast<T *>(wsp + align_up(moc_ffn_workspace_bytes(desc, MOC_OP_DECODE), 256));
    if (!use_decode_plan(*desc) && !(desc->flags & MOC_FLAG_SELECT_2_OF_8)) {
        // 6 to 32 tokens: the one-kernel form, whose selector CTAs -- idle until the gate values exist -- normalise the
        // tokens themselves
        bool fused_ok = false;
        const FusedLayout FL = fused_layout(*desc, false, fused_ok);
        if (fused_ok) {
            const SmallBatchLayout L = small_batch_layout(*desc);
            const int rc2 = forward_small_batch_fused(*desc, L, FL, xn, (const T *)w_gate, (const T *)w_up, (const T *)w_down,
                                                      (T *)out, wsp, st, (const T *)h, tc::kWaitLimitCycles, 0, (const T *)h,
                                                      (const T *)rms_weight, rms_eps);
            if (rc2 != MOC_ERR_UNSUPPORTED) return rc2;
        }
    }
    MOC_LAUNCH(KID_DEC_RMSNORM, st,
               launch_pdl(dec::rmsnorm_rows_kernel, dim3((unsigned)desc->tokens), 256, 0, st, (const T *)h,
                          (const T *)rms_weight, rms_eps, desc->d_model, xn));
    if ((rc = launch_ok()) != MOC_OK) return rc;
    if (use_decode_plan(*desc))
        return decode_bf16(*desc, xn, (const T *)w_gate, (const T *)w_up, (const T *)w_down, (T *)out, wsp, st,
                           (const T *)h);
    return forward_small_batch(*desc, xn, (const T *)w_gate, (const T *)w_up, (const T *)w_down, (T *)out, nullptr,
                               nullptr, nullptr, wsp, st, (const T *)h);
}

int moc_ffn_recompute_up(const moc_ffn_desc *desc, const void *x, const void *w_up, const int16_t *topk_idx,
                         void *topk_up, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    int rc = check_desc(desc);
    if (rc != MOC_OK) return rc;
    if (desc->tokens == 0) return MOC_OK;
    if (!good_ptr(x) || !good_ptr(w_up) || !good_ptr(topk_idx) || !good_ptr(topk_up)) return MOC_ERR_INVALID_ARG;
    const size_t need = moc_ffn_workspace_bytes(desc, MOC_OP_BACKWARD);
    if (need && (!good_ptr(workspace) || workspace_bytes < need)) return MOC_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int *status = device_status_ptr();
    if (!status) return MOC_ERR_CUDA;
    const int64_t T = desc->tokens;
    const int F = desc->d_ff, K = desc->k, dm = desc->d_model;
    const int64_t total = T * K;
    if (desc->dtype == MOC_BF16 && use_tc_plan(*desc)) {
        // dense U = x Wu^T with the GEMM of the forward pass (same contraction order: the same bf16 values), then a gather
        using namespace tc;
        using B16 = __nv_bfloat16;
        const TcBackwardLayout L = tc_backward_layout(*desc);
        B16 *U = reinterpret_cast<B16 *>(static_cast<char *>(workspace) + L.off_z);
        Params p;
        init_params(p);
        if (!map_k_major(&p.a_map[0], x, T, dm, dm, BM) || !map_k_major(&p.b_map[0], w_up, F, dm, dm, b_box_rows()))
            return MOC_ERR_CUDA;
        p.k_blocks = ceil_div(dm, BK);
        p.M = (int)T;
        p.N = F;
        p.m_tiles = ceil_div(T, BM);
        p.n_tiles = ceil_div(F, BN);
        p.c[0] = U;
        p.ldc[0] = L.ldf;
        p.status = status;
        MOC_LAUNCH(KID_RECOMPUTE_UP, st, (rc = launch_gemm<false, false, EPI_BF16>(p, st)));
        if (rc != MOC_OK) return rc;
        const unsigned grid = (unsigned)std::min<int64_t>((total + 255) / 256, 148 * 16);
        MOC_LAUNCH(KID_RECOMPUTE_UP, st,
                   (recompute_up_kernel<B16><<<grid, 256, 0, st>>>((const B16 *)x, (const B16 *)w_up, U, L.ldf, topk_idx, T,
                                                                    K, F, dm, (B16 *)topk_up, status)));
        return launch_ok();
    }
    const unsigned grid = (unsigned)std::min<int64_t>((total + 7) / 8, 148 * 32);
    if (desc->dtype == MOC_BF16) {
        using B16 = __nv_bfloat16;
        MOC_LAUNCH(KID_RECOMPUTE_UP, st,
                   (recompute_up_kernel<B16><<<grid, 256, 0, st>>>((const B16 *)x, (const B16 *)w_up, nullptr, 0, topk_idx,
                                                                    T, K, F, dm, (B16 *)topk_up, status)));
    } else {
        MOC_LAUNCH(KID_RECOMPUTE_UP, st,
                   (recompute_up_kernel<float><<<grid, 256, 0, st>>>((const float *)x, (const float *)w_up, nullptr, 0,
                                                                      topk_idx, T, K, F, dm, (float *)topk_up, status)));
    }
    return launch_ok();
}

int moc_topk_select(int64_t rows, int32_t n, int32_t n_ld, int32_t k, const float *gate, int16_t *idx_out,
                    void *cuda_stream) {
    if (rows < 0 || n < 1 || n_ld < n || k < 1 || k > n) return MOC_ERR_INVALID_ARG;
    if (n > 32768) return MOC_ERR_UNSUPPORTED;
    if (rows == 0) return MOC_OK;
    if (!good_ptr(gate) || !idx_out || (reinterpret_cast<uintptr_t>(idx_out) & 1u)) return MOC_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (rows <= sb::kMaxTokens) {
        // as in the plans: a small batch of rows goes to the selector that gives a whole CTA to each row
        const size_t smem1 = ((size_t)((n + 3) & ~3) + 2 * dec::kSelListCap) * sizeof(uint32_t);
        int *status = device_status_ptr();
        if (!status) return MOC_ERR_CUDA;
        int rc1 = set_smem(dec::cta_select_idx_kernel, smem1);
        if (rc1 != MOC_OK) return rc1;
        MOC_LAUNCH(KID_TOPK_SELECT, st,
                   (dec::cta_select_idx_kernel<<<(unsigned)rows, dec::kSelThreads, smem1, st>>>(gate, n, n_ld, k, idx_out,
                                                                                                  status)));
        return launch_ok();
    }
    const size_t smem = (size_t)n * sizeof(uint32_t);
    int rc = set_smem(topk_select_kernel<kSelectThreads>, smem);
    if (rc != MOC_OK) return rc;
    const unsigned grid = (unsigned)std::min<int64_t>(rows, 148 * 32);
    MOC_LAUNCH(KID_TOPK_SELECT, st,
               (topk_select_kernel<kSelectThreads><<<grid, kSelectThreads, smem, st>>>(gate, rows, n, n_ld, k,
                                                                                        idx_out)));
    return launch_ok();
}

// ---- test hooks: the selectors of the tensor-core plan and of the cooperative decode kernel on their own ----------
namespace moc {
namespace {
__global__ void set_hint_kernel(float *hint, float center, float width, float tag) {
    hint[0] = center;
    hint[1] = width;
    hint[2] = tag;
}

struct SelectTcLayout {
    size_t off_u, off_g, off_v, off_hint, total;
};
SelectTcLayout select_tc_layout(int64_t rows, int n_ld, int k) {
    SelectTcLayout L{};
    Carver c;
    L.off_u = c.take((size_t)rows * n_ld * sizeof(__nv_bfloat16));
    L.off_g = c.take((size_t)rows * k * sizeof(__nv_bfloat16));
    L.off_v = c.take((size_t)rows * k * sizeof(__nv_bfloat16));
    L.off_hint = c.take(256);
    L.total = c.off;
    return L;
}
bool select_tc_shape_ok(int64_t rows, int n, int n_ld, int k) {
    return rows >= 0 && n >= 1 && k >= 1 && k <= n && n <= 32768 && n_ld >= n && n_ld % 8 == 0 &&
           n_ld <= ((n + 127) / 128) * 128 && ((size_t)n + (size_t)k) * 4 <= 170 * 1024;
}
}  // namespace
}  // namespace moc

size_t moc_topk_select_tc_workspace_bytes(int64_t rows, int32_t n, int32_t n_ld, int32_t k) {
    if (!select_tc_shape_ok(rows, n, n_ld, k)) return 0;
    return select_tc_layout(rows, n_ld, k).total;
}

int moc_topk_select_tc(int64_t rows, int32_t n, int32_t n_ld, int32_t k, const float *gate, int16_t *idx_out,
                       const float *bracket, int *variant, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!select_tc_shape_ok(rows, n, n_ld, k)) return MOC_ERR_INVALID_ARG;
    const TcSelect sel = tc_select_config(n, k);
    if (variant) *variant = sel.variant;
    if (rows == 0) return MOC_OK;
    if (!good_ptr(gate) || !good_ptr(idx_out)) return MOC_ERR_INVALID_ARG;
    const SelectTcLayout L = select_tc_layout(rows, n_ld, k);
    if (!good_ptr(workspace) || workspace_bytes < L.total) return MOC_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char *ws = static_cast<char *>(workspace);
    int *status = device_status_ptr();
    if (!status) return MOC_ERR_CUDA;
    int rc = tc_select_prepare(sel, n, k);
    if (rc != MOC_OK) return rc;
    using B16 = __nv_bfloat16;
    B16 *U = reinterpret_cast<B16 *>(ws + L.off_u);
    float *hint = reinterpret_cast<float *>(ws + L.off_hint);
    // a zero up row: the selector forms SiLU(g) * 0 for its masked row, which nobody reads here
    if (cudaMemsetAsync(U, 0, (size_t)rows * n_ld * sizeof(B16), st) != cudaSuccess) return MOC_ERR_CUDA;
    if (cudaMemsetAsync(hint, 0, 256, st) != cudaSuccess) return MOC_ERR_CUDA;
    if (bracket) {
        set_hint_kernel<<<1, 1, 0, st>>>(hint, bracket[0], bracket[1], tc::kBracketTag);
    } else if (!sel.team_select) {
        // as in the forward pass: the CTA-per-row form starts from the exact threshold of the first row
        tc::select_hint_kernel<<<1, kSelectThreads, (size_t)n * sizeof(uint32_t), st>>>(gate, n, k, hint);
    }
    if ((rc = launch_ok()) != MOC_OK) return rc;
    tc_select_launch(sel, gate, n_ld, U, n_ld, rows, n, k, idx_out, reinterpret_cast<B16 *>(ws + L.off_g),
                     reinterpret_cast<B16 *>(ws + L.off_v), hint, status, st);
    return launch_ok();
}

size_t moc_ffn_decode_probe_workspace_bytes(const moc_ffn_desc *desc) {
    if (check_desc(desc) != MOC_OK || desc->tokens < 1) return 0;
    bool coop = false;
    const CoopLayout C = coop_layout(*desc, coop);
    return coop ? C.total : 0;
}

int moc_ffn_decode_probe(const moc_ffn_desc *desc, const void *x, const void *w_gate, const void *w_up,
                         const void *w_down, void *out, uint8_t *kept, void *workspace, size_t workspace_bytes,
                         void *cuda_stream) {
    int rc = check_desc(desc);
    if (rc != MOC_OK) return rc;
    // (whatever form moc_ffn_decode would prefer for this K: the probe exists to look at this kernel's selection)
    bool coop = false;
    const bool plain = desc->tokens >= 1 && desc->dtype == MOC_BF16 && !(desc->flags & MOC_FLAG_SELECT_POST_SILU);
    const CoopLayout C = plain ? coop_layout(*desc, coop) : CoopLayout{};
    if (!coop) return MOC_ERR_UNSUPPORTED;
    if (!good_ptr(x) || !good_ptr(w_gate) || !good_ptr(w_up) || !good_ptr(w_down) || !good_ptr(out) || !kept)
        return MOC_ERR_INVALID_ARG;
    if (!good_ptr(workspace) || workspace_bytes < C.total) return MOC_ERR_WORKSPACE;
    using T = __nv_bfloat16;
    return decode_coop(*desc, C, (const T *)x, (const T *)w_gate, (const T *)w_up, (const T *)w_down, (T *)out,
                       static_cast<char *>(workspace), static_cast<cudaStream_t>(cuda_stream), nullptr, 0.f, kept);
}

// ---- decode without a caller workspace --------------------------------------------------------------
// Scratch for moc_ffn_decode_static.  In host code the name below is only a handle for the runtime,
// not a device address: the address is asked for once per device and that pointer goes to the kernels.
static __device__ __align__(256) unsigned char g_static_scratch[MOC_STATIC_SCRATCH_BYTES];

static char *static_scratch_ptr() {
    static std::atomic<char *> cache[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    char *have = cache[dev].load(std::memory_order_relaxed);
    if (!have) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return nullptr;
        have = static_cast<char *>(p);
        cache[dev].store(have, std::memory_order_relaxed);
    }
    return have;
}

int moc_ffn_decode_static(const moc_ffn_desc *desc, const void *x, const void *w_gate, const void *w_up,
                          const void *w_down, void *out, void *cuda_stream) {
    int rc = check_desc(desc);
    if (rc != MOC_OK) return rc;
    if (desc->tokens > MOC_STATIC_MAX_TOKENS || desc->d_ff > MOC_STATIC_MAX_DFF) return MOC_ERR_STATIC_LIMIT;
    if (desc->tokens == 0) return MOC_OK;
    if (!good_ptr(x) || !good_ptr(w_gate) || !good_ptr(w_up) || !good_ptr(w_down) || !good_ptr(out))
        return MOC_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // bf16: the decode plan's kernels whenever their workspace fits the array (the LLaMA-7B layer does at 16 tokens)
    // (the post-SiLU selection key exists on the gathered kernels only, as for moc_ffn_decode)
    if (desc->dtype == MOC_BF16 && !(desc->flags & MOC_FLAG_SELECT_POST_SILU) && desc->d_model <= 256 * dec::kSliceCols &&
        decode_layout(*desc).total <= MOC_STATIC_SCRATCH_BYTES) {
        char *wsd = static_scratch_ptr();
        if (!wsd) return MOC_ERR_CUDA;
        using T = __nv_bfloat16;
        return decode_bf16(*desc, (const T *)x, (const T *)w_gate, (const T *)w_up, (const T *)w_down, (T *)out, wsd, st);
    }
    // otherwise the gathered kernels: same carving as the workspace variant; the limits above bound it by the array's size
    if (plan_forward(*desc).total > MOC_STATIC_SCRATCH_BYTES) return MOC_ERR_STATIC_LIMIT;
    char *ws = static_scratch_ptr();
    if (!ws) return MOC_ERR_CUDA;
    if (desc->dtype == MOC_BF16) {
        using T = __nv_bfloat16;
        return forward_gather<T>(*desc, (const T *)x, (const T *)w_gate, (const T *)w_up, (const T *)w_down,
                                 (T *)out, nullptr, nullptr, nullptr, ws, st);
    }
    return forward_gather<float>(*desc, (const float *)x, (const float *)w_gate, (const float *)w_up,
                                 (const float *)w_down, (float *)out, nullptr, nullptr, nullptr, ws, st);
}

int moc_tc_gemm_bf16(int64_t m, int64_t n, int64_t k, const void *a, int a_mn_major, int64_t lda, const void *b,
                     int b_mn_major, int64_t ldb, float *c, int64_t ldc, void *cuda_stream) {
    using namespace tc;
    if (m < 1 || n < 1 || k < 1 || m > INT32_MAX || n > INT32_MAX || k > INT32_MAX) return MOC_ERR_INVALID_ARG;
    if (!good_ptr(a) || !good_ptr(b) || !good_ptr(c) || lda % 8 || ldb % 8 || ldc < n) return MOC_ERR_INVALID_ARG;
    int *status = device_status_ptr();
    if (!status) return MOC_ERR_CUDA;
    Params p;
    init_params(p);
    const bool ok_a = a_mn_major ? map_mn_major(&p.a_map[0], a, k, m, lda) : map_k_major(&p.a_map[0], a, m, k, lda, BM);
    const bool ok_b = b_mn_major ? map_mn_major(&p.b_map[0], b, k, n, ldb) : map_k_major(&p.b_map[0], b, n, k, ldb, b_box_rows());
    if (!ok_a || !ok_b) return MOC_ERR_CUDA;
    p.k_blocks = ceil_div(k, BK);
    p.M = (int)m;
    p.N = (int)n;
    p.m_tiles = ceil_div(m, BM);
    p.n_tiles = ceil_div(n, BN);
    p.c[0] = c;
    p.ldc[0] = (int)ldc;
    p.status = status;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int rc = MOC_OK;
    if (!a_mn_major && !b_mn_major)
        MOC_LAUNCH(KID_TC_TEST_GEMM, st, (rc = launch_gemm<false, false, EPI_F32>(p, st)));
    else if (!a_mn_major && b_mn_major)
        MOC_LAUNCH(KID_TC_TEST_GEMM, st, (rc = launch_gemm<false, true, EPI_F32>(p, st)));
    else if (a_mn_major && b_mn_major)
        MOC_LAUNCH(KID_TC_TEST_GEMM, st, (rc = launch_gemm<true, true, EPI_F32>(p, st)));
    else
        MOC_LAUNCH(KID_TC_TEST_GEMM, st, (rc = launch_gemm<true, false, EPI_F32>(p, st)));
    return rc;
}

int moc_tc_gemm_sp_bf16(int64_t m, int64_t n, int64_t k, const void *a_compressed, const void *metadata, const void *b,
                        int b_mn_major, int64_t ldb, float *c, int64_t ldc, void *cuda_stream) {
    using namespace tcsp;
    if (m < 1 || n < 1 || k < 16 || k % 16 != 0 || m > INT32_MAX || n > INT32_MAX || k > INT32_MAX) return MOC_ERR_INVALID_ARG;
    if (!good_ptr(a_compressed) || !good_ptr(metadata) || !good_ptr(b) || !good_ptr(c) || ldb % 8 || ldc < n)
        return MOC_ERR_INVALID_ARG;
    int *status = device_status_ptr();
    if (!status) return MOC_ERR_CUDA;
    SpParams p;
    memset(&p, 0, sizeof(p));
    if (!tc::make_map(&p.a_map, a_compressed, m, k / 2, k / 2, 64, SBM)) return MOC_ERR_CUDA;
    const bool ok_b = b_mn_major ? tc::make_map(&p.b_map, b, k, n, ldb, 64, 64) : tc::make_map(&p.b_map, b, n, k, ldb, 64, SBN);
    if (!ok_b) return MOC_ERR_CUDA;
    p.e = static_cast<const uint4 *>(metadata);
    p.k_stages = ceil_div(k, SBKL);
    p.M = (int)m;
    p.N = (int)n;
    p.m_tiles = ceil_div(m, SBM);
    p.n_tiles = ceil_div(n, SBN);
    p.c = c;
    p.ldc = (int)ldc;
    p.out_bf16 = 0;
    p.status = status;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int grid = std::min(p.m_tiles * p.n_tiles, tc::sm_count());
    if (b_mn_major) {
        if (cudaFuncSetAttribute(gemm_sp_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SSMEM_BYTES) != cudaSuccess)
            return MOC_ERR_CUDA;
        MOC_LAUNCH(KID_TC_TEST_GEMM, st, (gemm_sp_kernel<true><<<grid, STHREADS, SSMEM_BYTES, st>>>(p)));
    } else {
        if (cudaFuncSetAttribute(gemm_sp_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SSMEM_BYTES) != cudaSuccess)
            return MOC_ERR_CUDA;
        MOC_LAUNCH(KID_TC_TEST_GEMM, st, (gemm_sp_kernel<false><<<grid, STHREADS, SSMEM_BYTES, st>>>(p)));
    }
    return launch_ok();
}

size_t moc_tc_gemm_sp_dense_workspace_bytes(int64_t m, int64_t k) {
    if (m < 1 || k < 8 || k % 8 != 0 || k > INT32_MAX) return 0;
    const SparseOperandLayout L = sparse_operand_layout(m, (int)k);
    return L.comp_bytes + L.meta_bytes + 256 + 4096 * sizeof(tcsp::Overflow);
}

int moc_tc_gemm_sp_dense_bf16(int64_t m, int64_t n, int64_t k, const void *a_dense, int64_t lda, const void *b, int64_t ldb,
                              void *c, int64_t ldc, int accumulate, int64_t *overflow_count, void *workspace,
                              size_t workspace_bytes, void *cuda_stream) {
    if (m < 1 || n < 1 || k < 8 || k % 8 != 0 || m > INT32_MAX || n > INT32_MAX || k > INT32_MAX) return MOC_ERR_INVALID_ARG;
    if (!good_ptr(a_dense) || !good_ptr(b) || !c || lda % 8 || ldb % 8 || lda < k || ldb < n || ldc < n) return MOC_ERR_INVALID_ARG;
    if (!tc::pair_mode()) return MOC_ERR_UNSUPPORTED;
    const size_t need = moc_tc_gemm_sp_dense_workspace_bytes(m, k);
    if (!good_ptr(workspace) || workspace_bytes < need) return MOC_ERR_WORKSPACE;
    int *status = device_status_ptr();
    if (!status) return MOC_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    using B16 = __nv_bfloat16;
    const SparseOperandLayout L = sparse_operand_layout(m, (int)k);
    char *ws = static_cast<char *>(workspace);
    B16 *comp = reinterpret_cast<B16 *>(ws);
    uint32_t *meta = reinterpret_cast<uint32_t *>(ws + L.comp_bytes);
    unsigned int *ovf_n = reinterpret_cast<unsigned int *>(ws + L.comp_bytes + L.meta_bytes);
    tcsp::Overflow *ovf = reinterpret_cast<tcsp::Overflow *>(ws + L.comp_bytes + L.meta_bytes + 256);
    if (cudaMemsetAsync(ovf_n, 0, 256, st) != cudaSuccess) return MOC_ERR_CUDA;
    // rows beyond m of the last 128-row block and columns beyond k / 2 are never read as values (the maps clip), but
    // the metadata of clipped rows must be valid nibbles: the kernel writes fillers for them
    int rc = sparse_compress(static_cast<const B16 *>(a_dense), m, (int)k, (int)lda, L, comp, meta, ovf, 4096, ovf_n, st);
    if (rc != MOC_OK) return rc;
    const B16 *comps[2] = {comp, nullptr};
    const uint32_t *metas[2] = {meta, nullptr};
    const B16 *bs[2] = {static_cast<const B16 *>(b), nullptr};
    rc = sparse_gemm_pair(m, (int)n, (int)k, 1, comps, metas, L, bs, (int)ldb, static_cast<B16 *>(c), (int)ldc,
                          accumulate != 0, KID_TC_TEST_GEMM, status, st);
    if (rc != MOC_OK) return rc;
    if (overflow_count) {
        unsigned int h = 0;
        if (cudaMemcpyAsync(&h, ovf_n, sizeof(h), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
            cudaStreamSynchronize(st) != cudaSuccess)
            return MOC_ERR_CUDA;
        *overflow_count = h;
    }
    return MOC_OK;
}

int moc_test_small_batch_stall(const moc_ffn_desc *desc, const void *x, const void *w_gate, const void *w_up,
                               const void *w_down, void *out, void *workspace, size_t workspace_bytes, int64_t limit_cycles,
                               void *cuda_stream) {
    int rc = check_desc(desc);
    if (rc != MOC_OK) return rc;
    if (limit_cycles < 1 || limit_cycles > tc::kWaitLimitCycles) return MOC_ERR_INVALID_ARG;
    if (!good_ptr(x) || !good_ptr(w_gate) || !good_ptr(w_up) || !good_ptr(w_down) || !good_ptr(out)) return MOC_ERR_INVALID_ARG;
    if (!use_small_batch_plan(*desc) || (desc->flags & MOC_FLAG_SELECT_2_OF_8)) return MOC_ERR_UNSUPPORTED;
    const size_t need = moc_ffn_workspace_bytes(desc, MOC_OP_DECODE);
    if (!good_ptr(workspace) || workspace_bytes < need) return MOC_ERR_WORKSPACE;
    bool ok = false;
    const FusedLayout FL = fused_layout(*desc, false, ok);
    if (!ok) return MOC_ERR_UNSUPPORTED;
    using T = __nv_bfloat16;
    const SmallBatchLayout L = small_batch_layout(*desc);
    return forward_small_batch_fused(*desc, L, FL, (const T *)x, (const T *)w_gate, (const T *)w_up, (const T *)w_down, (T *)out,
                                     static_cast<char *>(workspace), static_cast<cudaStream_t>(cuda_stream), nullptr,
                                     (long long)limit_cycles, 1);
}

int moc_test_bounded_wait(int64_t limit_cycles, void *cuda_stream) {
    if (limit_cycles < 1 || limit_cycles > tc::kWaitLimitCycles) return MOC_ERR_INVALID_ARG;
    int *status = device_status_ptr();
    if (!status) return MOC_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    tc::bounded_wait_probe_kernel<<<1, 32, 0, st>>>((long long)limit_cycles, status, nullptr);
    return launch_ok();
}

int moc_last_device_status(void *cuda_stream) {
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return MOC_ERR_CUDA;
    int *p = device_status_ptr();
    if (!p) return MOC_ERR_CUDA;
    int v = 0;
    if (cudaMemcpy(&v, p, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return MOC_ERR_CUDA;
    if (v != 0) {
        if (cudaMemset(p, 0, sizeof(int)) != cudaSuccess) return MOC_ERR_CUDA;
    }
    return v;
}

#ifdef MOC_TIMELINE
extern "C" __attribute__((visibility("default"))) int moc_debug_timeline(unsigned long long *out, int n) {
    if (cudaDeviceSynchronize() != cudaSuccess) return MOC_ERR_CUDA;
    return cudaMemcpyFromSymbol(out, g_timeline, sizeof(unsigned long long) * (size_t)std::min(n, 4096)) == cudaSuccess
               ? MOC_OK : MOC_ERR_CUDA;
}

// development probe: W [rows_total, cols] bf16 is read once in TMA boxes of rows_per_cta rows x 64 columns, `boxes`
// adjacent boxes per stage through a ring of `stages` stages, nothing computed
namespace moc { namespace {
struct BoxProbe {
    CUtensorMap map;
    int rows, cols, boxes, stages;
    uint32_t pitch;
    int *status;
};
__global__ void __launch_bounds__(64, 1) box_probe_kernel(const __grid_constant__ BoxProbe p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[64];
    __shared__ int s_abort;
    const uint32_t base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
    auto full_bar = [&](int s) { return tc::smem_u32(&bars[s]); };
    auto empty_bar = [&](int s) { return tc::smem_u32(&bars[32 + s]); };
    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            tc::mbar_init(full_bar(s), 1);
            tc::mbar_init(empty_bar(s), 1);
        }
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    const int n = (p.cols / 64 + p.boxes - 1) / p.boxes;
    const int row0 = (int)blockIdx.x * p.rows;
    if (threadIdx.x == 0) {
        int stage = 0;
        uint32_t phase = 0;
        for (int i = 0; i < n; ++i) {
            if (!tc::mbar_wait(empty_bar(stage), phase ^ 1u, &s_abort, p.status)) return;
            tc::mbar_expect_tx(full_bar(stage), (uint32_t)p.boxes * (uint32_t)p.rows * 128u);
            for (int b = 0; b < p.boxes; ++b)
                tc::tma_load_2d(base + (uint32_t)stage * p.boxes * p.pitch + (uint32_t)b * p.pitch, &p.map, full_bar(stage),
                                (i * p.boxes + b) * 64, row0);
            if (++stage == p.stages) {
                stage = 0;
                phase ^= 1u;
            }
        }
    } else if (threadIdx.x == 32) {
        int stage = 0;
        uint32_t phase = 0;
        for (int i = 0; i < n; ++i) {
            if (!tc::mbar_wait(full_bar(stage), phase, &s_abort, p.status)) return;
            tc::mbar_arrive(empty_bar(stage));
            if (++stage == p.stages) {
                stage = 0;
                phase ^= 1u;
            }
        }
    }
}
} }
extern "C" MOC_API int moc_debug_stream_boxes(const void *w, int rows_total, int cols, int rows_per_cta, int boxes, int stages,
                                              void *cuda_stream) {
    BoxProbe p;
    memset(&p, 0, sizeof(p));
    if (stages > 32 || rows_per_cta > 256) return MOC_ERR_INVALID_ARG;
    if (!tc::make_map(&p.map, static_cast<const __nv_bfloat16 *>(w), rows_total, cols, cols, 64, rows_per_cta)) return MOC_ERR_CUDA;
    p.rows = rows_per_cta;
    p.cols = cols;
    p.boxes = boxes;
    p.stages = stages;
    p.pitch = ((uint32_t)rows_per_cta * 128u + 1023u) & ~1023u;
    p.status = device_status_ptr();
    const size_t smem = 1024 + (size_t)stages * boxes * p.pitch;
    int rc = set_smem(box_probe_kernel, smem, 1024);
    if (rc != MOC_OK) return rc;
    box_probe_kernel<<<(rows_total + rows_per_cta - 1) / rows_per_cta, 64, smem, static_cast<cudaStream_t>(cuda_stream)>>>(p);
    return launch_ok();
}

// development probe: cycles per MMA, seen by the issuing thread, of `count` MMAs of shape M x N x 16 (bf16, operands in
// shared memory, K-major, all zero) issued back to back with a tcgen05.commit after every `per_commit` of them.
// mode bit 0: the thread waits for every commit's barrier (else only for the last); bit 1: a second thread issues the same
// sequence at the same time into its own TMEM columns and barriers (the figure is still the first thread's).
namespace moc { namespace {
__global__ void __launch_bounds__(128, 1) mma_probe_kernel(int m, int n, int count, int per_commit, int mode, long long *cycles, int *status) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars4[4];
    __shared__ uint32_t holder;
    __shared__ int s_abort;
    const uint32_t base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
    for (int i = threadIdx.x; i < 96 * 1024 / 4; i += 128) reinterpret_cast<uint32_t *>(smem_raw + (base - tc::smem_u32(smem_raw)))[i] = 0u;
    if (threadIdx.x == 0) {
        for (int i = 0; i < 4; ++i) tc::mbar_init(tc::smem_u32(&bars4[i]), 1);
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (threadIdx.x < 32) {
        tc::tmem_alloc(tc::smem_u32(&holder), 512);
        tc::tmem_relinquish();
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t who = threadIdx.x >> 5;
    const uint32_t tmem = holder + who * 256;
    const uint32_t bar = tc::smem_u32(&bars4[2 * who]), bar_unwaited = tc::smem_u32(&bars4[2 * who + 1]);
    if (threadIdx.x == 0 || ((mode & 2) && threadIdx.x == 32)) {
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
        uint32_t parity = 0;
        // eight descriptor pairs held in registers: A walks over three 11 KiB regions, so that the loop is nothing but MMAs
        const uint64_t ad0 = tc::make_smem_desc(base, 16, 1024), bd0 = tc::make_smem_desc(base + 49152, 16, 1024);
        uint64_t ad[8], bd[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            ad[e] = ad0 + (uint64_t)((e & 3) * 2 + (e >> 2) * 704);
            bd[e] = bd0 + (uint64_t)((e & 3) * 2);
        }
        const long long t0 = clock64();
        for (int i = 0; i < count; i += per_commit) {
            for (int j = 0; j < per_commit; j += 8) {
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    asm volatile(
                        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 1, 0;\n\t"
                        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem), "l"(ad[e]), "l"(bd[e]), "r"(idesc)
                        : "memory");
            }
            if (!(mode & 1) && i + per_commit < count) {
                tc::umma_commit(bar_unwaited);  // nobody waits for this one
                continue;
            }
            tc::umma_commit(bar);
            if (!tc::mbar_wait(bar, parity, &s_abort, status)) break;
            parity ^= 1u;
        }
        if (blockIdx.x == 0 && threadIdx.x == 0) *cycles = clock64() - t0;
    }
    tc::tc_fence_before();
    __syncthreads();
    if (threadIdx.x < 32) {
        tc::tc_fence_after();
        tc::tmem_dealloc(holder, 512);
    }
}
} }
extern "C" MOC_API long long moc_debug_mma_cycles(int m, int n, int count, int per_commit, int mode) {
    if (m != 64 && m != 128) return -4;
    if (n < 16 || n > 256 || n % 16 || count < 8 || per_commit < 8 || per_commit % 8 || count % per_commit) return -4;
    long long *dev = nullptr, host = -1;
    if (cudaMalloc(&dev, sizeof(long long)) != cudaSuccess) return -1;
    const size_t smem = 100 * 1024;  // A within the first 48 KiB, B (up to 256 rows of 128 bytes) behind it
    if (set_smem(mma_probe_kernel, smem, 1024) != MOC_OK) return -2;
    mma_probe_kernel<<<tc::sm_count(), 128, smem>>>(m, n, count, per_commit, mode, dev, device_status_ptr());
    if (cudaMemcpy(&host, dev, sizeof(host), cudaMemcpyDeviceToHost) != cudaSuccess) host = -3;
    cudaFree(dev);
    return host;
}
#endif

int moc_profile_stream_read(const void *a, size_t a_bytes, const void *b, size_t b_bytes, const void *c, size_t c_bytes,
                            void *cuda_stream) {
    const void *ptr[3] = {a, b, c};
    const size_t n[3] = {a_bytes, b_bytes, c_bytes};
    dec::ProbeRanges r{};
    for (int i = 0; i < 3; ++i) {
        if (n[i] && (!good_ptr(ptr[i]) || n[i] % 16 != 0)) return MOC_ERR_INVALID_ARG;
        r.base[i] = static_cast<const uint8_t *>(ptr[i]);
        r.bytes[i] = n[i];
    }
    int *status = device_status_ptr();
    if (!status) return MOC_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const size_t smem = (size_t)dec::kProbeStages * dec::kProbeChunk;
    int rc = set_smem(dec::stream_probe_kernel, smem, 1024);
    if (rc != MOC_OK) return rc;
    MOC_LAUNCH(KID_STREAM_PROBE, st,
               launch_pdl(dec::stream_probe_kernel, dim3(2 * tc::sm_count()), dec::kProbeThreads, smem, st, r, status));
    return launch_ok();
}

int64_t moc_launch_count(void) { return g_prof.launches.load(std::memory_order_relaxed); }

int moc_profile_enable(int on) {
    if (on) {
        if (g_prof.ev.empty()) {
            g_prof.ev.resize(2 * Profiler::kMaxPairs);
            for (auto &e : g_prof.ev) {
                if (cudaEventCreate(&e) != cudaSuccess) {
                    g_prof.ev.clear();
                    return MOC_ERR_CUDA;
                }
            }
        }
        g_prof.used = g_prof.dropped = 0;
        for (int i = 0; i < KID_COUNT; ++i) {
            g_prof.ms[i] = 0.0;
            g_prof.count[i] = 0;
        }
    }
    g_prof.on = on != 0;
    return MOC_OK;
}

int moc_profile_collect(void *cuda_stream) {
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return MOC_ERR_CUDA;
    for (int i = 0; i < g_prof.used; ++i) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, g_prof.ev[2 * i], g_prof.ev[2 * i + 1]) != cudaSuccess) return MOC_ERR_CUDA;
        g_prof.ms[g_prof.ids[i]] += ms;
        g_prof.count[g_prof.ids[i]] += 1;
    }
    const int dropped = g_prof.dropped;
    g_prof.used = g_prof.dropped = 0;
    return dropped;
}

int moc_profile_kernel_count(void) { return KID_COUNT; }

const char *moc_profile_kernel_name(int id) { return (id >= 0 && id < KID_COUNT) ? kKernelNames[id] : ""; }

int moc_profile_read(int id, int64_t *launches, double *total_ms) {
    if (id < 0 || id >= KID_COUNT || !launches || !total_ms) return MOC_ERR_INVALID_ARG;
    *launches = g_prof.count[id];
    *total_ms = g_prof.ms[id];
    return MOC_OK;
}

const char *moc_status_string(int status) {
    switch (status) {
        case MOC_OK: return "ok";
        case MOC_ERR_INVALID_ARG: return "invalid argument";
        case MOC_ERR_UNSUPPORTED: return "unsupported shape or type";
        case MOC_ERR_WORKSPACE: return "workspace missing or too small";
        case MOC_ERR_CUDA: return "CUDA runtime error";
        case MOC_ERR_TIMEOUT: return "a bounded device-side wait expired";
        case MOC_ERR_BAD_INDEX: return "saved channel index out of range";
        case MOC_ERR_STATIC_LIMIT: return "problem exceeds the built-in scratch of moc_ffn_decode_static";
        default: return "unknown status";
    }
}

}  // extern "C"

