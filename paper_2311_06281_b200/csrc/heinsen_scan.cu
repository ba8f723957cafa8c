// C-ABI of libheinsen_scan: argument validation, kernel selection, tensor maps, launches.
// See include/heinsen_scan.h for the contract of every entry point.
#include "../../include/heinsen_scan.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <climits>
#include <chrono>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "hs_kernels.cuh"

namespace {

using namespace hs;

std::atomic<int> g_path{HS_PATH_AUTO};
std::atomic<int> g_last_path{0};
std::atomic<long long> g_launches{0};
std::atomic<unsigned int> g_spin_limit{hs::kLookbackSpinLimit};
std::atomic<long long> g_mute_tile{-1};
thread_local char g_cuda_msg[256] = "";

constexpr long long kMaxN = (1ll << 31) - (1ll << 20);  // column indices and TMA coordinates are int32
constexpr long long kMaxTmaDim = kMaxN;
constexpr int kBatchedMinRowsPerSm = 8;  // fewer rows per SM than this: look-back kernel
constexpr int kBatchedMinWarpsPerSm = 12; // rows per warp are chosen to keep at least this many warps per SM
constexpr int kLookbackMinWarps = 8;     // fewest compute warps (= chunks per tile) of the look-back kernel
constexpr int kLookbackWarps = 14;       // default compute warps of the look-back kernel
constexpr size_t kMaxWarpSlots = 16 * 256;  // warp slots of the batched kernel, at most
constexpr int kMinChunk = 512;           // smallest chunk of the real storage types (32 lanes x 16 elements)
constexpr int kComplexChunk = 256;       // chunk of the complex-logarithm storage type (32 lanes x 8 elements)
constexpr hs_dtype kC64 = static_cast<hs_dtype>(2);  // internal: complex64 elements (heinsen_scan_log_complex)

unsigned long long next_call_id() {
    static std::atomic<unsigned long long> counter{[] {
        const auto t = std::chrono::high_resolution_clock::now().time_since_epoch().count();
        unsigned long long z = (unsigned long long)t * 0x9E3779B97F4A7C15ull;
        z ^= (unsigned long long)(uintptr_t)&g_path << 17;
        z ^= z >> 29;
        return z;
    }()};
    // 62 bits; never 0
    unsigned long long id = (counter.fetch_add(1) + 1) & ((1ull << 62) - 1);
    return id ? id : 1;
}

struct DeviceInfo {
    int sm_count = 0;
    int cc_major = 0;
    int max_smem_optin = 0;
    bool ok = false;
};

hs_status device_info(DeviceInfo& out) {
    static std::mutex mu;
    static DeviceInfo cache[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) {
        snprintf(g_cuda_msg, sizeof g_cuda_msg, "cudaGetDevice: %s", cudaGetErrorString(e));
        return HS_ERR_CUDA;
    }
    if (dev < 0 || dev >= 64) return HS_ERR_UNSUPPORTED_DEVICE;
    std::lock_guard<std::mutex> lk(mu);
    DeviceInfo& d = cache[dev];
    if (!d.ok) {
        if (cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&d.cc_major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&d.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) {
            snprintf(g_cuda_msg, sizeof g_cuda_msg, "cudaDeviceGetAttribute failed");
            return HS_ERR_CUDA;
        }
        d.ok = true;
    }
    out = d;
    return HS_OK;
}

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn encode_fn() {
    static EncodeFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeFn>(p);
    }();
    return fn;
}

// [rows, n] row-major as a 2-D tensor map whose box is {128 bytes of a row, box_rows rows}, 128-byte swizzle.
// flat: the same memory as (element in 128-byte line, whole line of the row, row), box = box_rows consecutive
// lines of one row; the hardware clips a box at the row's last whole line, the n % line elements after it
// are not part of this view.
bool encode_tmap(CUtensorMap* tm, const void* ptr, hs_dtype dt, long long rows, long long n, int box_rows, bool flat) {
    EncodeFn fn = encode_fn();
    if (!fn) return false;
    // complex64 rows are shown to TMA as rows of 2n floats
    if (dt == kC64) { dt = HS_F32; n *= 2; }
    const int es = (dt == HS_F32) ? 4 : 2;
    const CUtensorMapDataType type = dt == HS_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r;
    if (flat) {
        const cuuint64_t line = (cuuint64_t)(128 / es);
        cuuint64_t dims[3] = {line, (cuuint64_t)n / line, (cuuint64_t)rows};
        cuuint64_t strides[2] = {128, (cuuint64_t)n * es};
        cuuint32_t box[3] = {(cuuint32_t)line, (cuuint32_t)box_rows, 1};
        r = fn(tm, type, 3, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    } else {
        cuuint64_t dims[2] = {(cuuint64_t)n, (cuuint64_t)rows};
        cuuint64_t strides[1] = {(cuuint64_t)n * es};
        cuuint32_t box[2] = {(cuuint32_t)(128 / es), (cuuint32_t)box_rows};
        r = fn(tm, type, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
    return r == CUDA_SUCCESS;
}

// Encoding a tensor map costs about a microsecond and a call needs three; a map depends only on the
// arguments below (it holds an address and a geometry, no state), so the most recent ones are kept.
struct TmapKey {
    const void* ptr;
    long long rows, n;
    int dt, box_rows, flat, dev;
    bool operator==(const TmapKey& o) const {
        return ptr == o.ptr && rows == o.rows && n == o.n && dt == o.dt && box_rows == o.box_rows && flat == o.flat &&
               dev == o.dev;
    }
};
struct TmapSlot {
    TmapKey key;
    CUtensorMap map;
    bool used = false;
};
constexpr int kTmapSlots = 24;
std::mutex g_tmap_mu;
TmapSlot g_tmap_cache[kTmapSlots];
int g_tmap_next = 0;

bool make_tmap(CUtensorMap* tm, const void* ptr, hs_dtype dt, long long rows, long long n, int box_rows, bool flat) {
    int dev = 0;
    cudaGetDevice(&dev);
    const TmapKey key{ptr, rows, n, (int)dt, box_rows, flat ? 1 : 0, dev};
    {
        std::lock_guard<std::mutex> lk(g_tmap_mu);
        for (int i = 0; i < kTmapSlots; ++i)
            if (g_tmap_cache[i].used && g_tmap_cache[i].key == key) {
                *tm = g_tmap_cache[i].map;
                return true;
            }
    }
    if (!encode_tmap(tm, ptr, dt, rows, n, box_rows, flat)) return false;
    std::lock_guard<std::mutex> lk(g_tmap_mu);
    TmapSlot& slot = g_tmap_cache[g_tmap_next];
    g_tmap_next = (g_tmap_next + 1) % kTmapSlots;
    slot.key = key;
    slot.map = *tm;
    slot.used = true;
    return true;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Tuning knobs.  Each has a measured default chosen per call; a knob overrides it when it is set.  The
// environment (HEINSEN_SCAN_<NAME>) is read once, when the first knob is looked up; afterwards only
// heinsen_scan_tune() changes a knob, so that a launch costs no getenv().
enum Knob : int {
    kKnobNoTma = 0, kKnobRowsPerWarp, kKnobWarps, kKnobRowTickets, kKnobNoFlat, kKnobNoPdl, kKnobLbStages,
    kKnobLbWarps, kKnobLbSleepIdle, kKnobLbSleepReady, kKnobLbCtasPerSm, kKnobStages, kKnobSpans, kKnobCount
};
const char* const kKnobNames[kKnobCount] = {
    "NO_TMA", "ROWS_PER_WARP", "WARPS", "ROW_TICKETS", "NO_FLAT", "NO_PDL", "LB_STAGES",
    "LB_WARPS", "LB_SLEEP_IDLE", "LB_SLEEP_READY", "LB_CTAS_PER_SM", "STAGES", "SPANS"};
constexpr int kKnobUnset = INT_MIN;
std::atomic<int> g_knobs[kKnobCount];
std::once_flag g_knobs_once;

void load_knobs_from_env() {
    for (int k = 0; k < kKnobCount; ++k) {
        char name[64];
        snprintf(name, sizeof name, "HEINSEN_SCAN_%s", kKnobNames[k]);
        const char* v = std::getenv(name);
        g_knobs[k].store((v && *v) ? std::atoi(v) : kKnobUnset);
    }
}
// value of a knob clamped to [lo, hi], or `dflt` when it is not set
int knob(Knob k, int dflt, int lo, int hi) {
    std::call_once(g_knobs_once, load_knobs_from_env);
    const int x = g_knobs[k].load(std::memory_order_relaxed);
    if (x == kKnobUnset) return dflt;
    return x < lo ? lo : (x > hi ? hi : x);
}

// ---------------------------------------------------------------------------------------------
struct Problem {
    int mode;            // hs::Mode
    hs_dtype din, dout;
    Params p;
    bool tma;
};


struct KernelEntry {
    const void* batched;      // row groups stay with their warp slots
    const void* batched_tk;   // row groups handed out by tickets
    const void* batched_span; // one row per warp, the rows' chunks shared out evenly among the warp slots (or null)
    const void* lookback;
    int K;
    int warp_smem_per_stage;  // bytes of one input stage (both tensors) of one warp
    int warp_smem_out;        // bytes of both output buffers of one warp
    int (*lb_smem)(int, int); // dynamic shared memory of the look-back kernel for W compute warps, S stages
    int lb_K;                 // elements per lane per chunk in the look-back kernel
};

template <int MODE, typename TIn, typename TOut, int K, bool TMA>
KernelEntry entry() {
    KernelEntry e;
    constexpr int LBK = sizeof(TIn) == 8 ? 8 : 16;  // the look-back kernel parks fp32 partial sums: 16 per lane (8 for complex elements)
    e.batched = reinterpret_cast<const void*>(&batched_scan_kernel<MODE, TIn, TOut, K, TMA, false>);
    e.batched_tk = reinterpret_cast<const void*>(&batched_scan_kernel<MODE, TIn, TOut, K, TMA, true>);
    e.batched_span = reinterpret_cast<const void*>(&batched_span_kernel<MODE, TIn, TOut, K, TMA>);
    e.lookback = reinterpret_cast<const void*>(&lookback_scan_kernel<MODE, TIn, TOut, LBK, TMA>);
    e.lb_K = LBK;
    e.K = K;
    constexpr int PAD = TMA ? 0 : ChunkEngine<MODE, TIn, TOut, K>::WIDE_PAD;  // chunk buffers without TMA are one line longer
    e.warp_smem_per_stage = 2 * (32 * K * (int)sizeof(TIn) + PAD);
    e.warp_smem_out = 2 * (32 * K * (int)sizeof(TOut) + PAD);
    e.lb_smem = [](int W, int S) { return lb_total_smem_bytes<TIn, LBK, PAD>(W, S); };
    return e;
}

// Modes that exist for the row-batched kernel only.
template <int MODE, typename TIn, typename TOut, int K, bool TMA>
KernelEntry entry_batched_only() {
    KernelEntry e;
    e.batched = reinterpret_cast<const void*>(&batched_scan_kernel<MODE, TIn, TOut, K, TMA, false>);
    e.batched_tk = reinterpret_cast<const void*>(&batched_scan_kernel<MODE, TIn, TOut, K, TMA, true>);
    e.batched_span = nullptr;
    e.lookback = nullptr;
    e.lb_K = K;
    e.K = K;
    constexpr int PAD = TMA ? 0 : ChunkEngine<MODE, TIn, TOut, K>::WIDE_PAD;
    e.warp_smem_per_stage = 2 * (32 * K * (int)sizeof(TIn) + PAD);
    e.warp_smem_out = 2 * (32 * K * (int)sizeof(TOut) + PAD);
    e.lb_smem = nullptr;
    return e;
}

bool find_kernel(int mode, hs_dtype din, hs_dtype dout, bool tma, KernelEntry& e) {
#define HS_PICK(M, TI, TO, KK)                                               \
    do {                                                                     \
        e = tma ? entry<M, TI, TO, KK, true>() : entry<M, TI, TO, KK, false>(); \
        return true;                                                         \
    } while (0)
    using bf16 = __nv_bfloat16;
    if (mode == kLinear) {
        if (din == HS_F32 && dout == HS_F32) HS_PICK(kLinear, float, float, 16);
        return false;
    }
    if (mode == kPairs) {
        if (din == HS_F32 && dout == HS_F32) {
            e = tma ? entry_batched_only<kPairs, float, float, 16, true>()
                    : entry_batched_only<kPairs, float, float, 16, false>();
            return true;
        }
        return false;
    }
    if (mode == kLogUnsigned) {
        if (din == HS_F32 && dout == HS_F32) HS_PICK(kLogUnsigned, float, float, 16);
        if (din == HS_BF16 && dout == HS_BF16) HS_PICK(kLogUnsigned, bf16, bf16, 32);
        if (din == HS_F32 && dout == HS_BF16) HS_PICK(kLogUnsigned, float, bf16, 16);
        return false;
    }
    if (mode == kLogSigned) {
        if (din == kC64 && dout == kC64) HS_PICK(kLogSigned, cplx, cplx, 8);
        if (din == HS_F32 && dout == HS_F32) HS_PICK(kLogSigned, float, float, 16);
        if (din == HS_BF16 && dout == HS_BF16) HS_PICK(kLogSigned, bf16, bf16, 32);
        if (din == HS_F32 && dout == HS_BF16) HS_PICK(kLogSigned, float, bf16, 16);
        return false;
    }
    return false;
#undef HS_PICK
}

long long lookback_tiles_per_row(long long n, int chunk, int warps) {
    const long long tile = (long long)warps * chunk;
    return (n + tile - 1) / tile;
}

int choose_path(long long rows, const DeviceInfo& d) {
    const int forced = g_path.load();
    if (forced == HS_PATH_BATCHED || forced == HS_PATH_LOOKBACK) return forced;
    return rows >= (long long)kBatchedMinRowsPerSm * d.sm_count ? HS_PATH_BATCHED : HS_PATH_LOOKBACK;
}

size_t workspace_bytes_for(long long rows, long long n, int min_chunk = kMinChunk) {
    // sized for the smallest chunk so that it covers every type
    const long long tpr = lookback_tiles_per_row(n, min_chunk, kLookbackMinWarps);
    size_t words = (size_t)(rows * tpr * 3);  // a tile's aggregate (two words), and the value entering it
    // ... or, for the batched kernel that shares the rows' chunks out among its warp slots, one word per slot
    // (at most 16 warps on each of at most 256 SMs; only shapes with at least one row per slot use it)
    if (rows >= 128 && words < kMaxWarpSlots) words = kMaxWarpSlots;
    return sizeof(Header) + words * 16;
}

// cudaFuncSetAttribute and the occupancy query cost microseconds per call; remember what was set.
struct FnCache {
    const void* fn;
    int dev;
    int smem_set;
    int occ_threads, occ_smem, occ_value;
};
std::mutex g_fn_mu;
FnCache g_fn_cache[128];
int g_fn_count = 0;

FnCache* fn_slot(const void* fn) {
    int dev = 0;
    cudaGetDevice(&dev);
    for (int i = 0; i < g_fn_count; ++i)
        if (g_fn_cache[i].fn == fn && g_fn_cache[i].dev == dev) return &g_fn_cache[i];
    if (g_fn_count >= 128) return nullptr;
    FnCache* c = &g_fn_cache[g_fn_count++];
    c->fn = fn; c->dev = dev; c->smem_set = -1; c->occ_threads = c->occ_smem = c->occ_value = -1;
    return c;
}

cudaError_t ensure_smem_attr(const void* fn, int smem) {
    std::lock_guard<std::mutex> lk(g_fn_mu);
    FnCache* c = fn_slot(fn);
    if (c && c->smem_set >= smem) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess && c) c->smem_set = smem;
    return e;
}

cudaError_t cached_occupancy(int* per_sm, const void* fn, int threads, int smem) {
    std::lock_guard<std::mutex> lk(g_fn_mu);
    FnCache* c = fn_slot(fn);
    if (c && c->occ_threads == threads && c->occ_smem == smem) { *per_sm = c->occ_value; return cudaSuccess; }
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(per_sm, fn, threads, smem);
    if (e == cudaSuccess && c) { c->occ_threads = threads; c->occ_smem = smem; c->occ_value = *per_sm; }
    return e;
}

hs_status cuda_fail(const char* what, cudaError_t e) {
    snprintf(g_cuda_msg, sizeof g_cuda_msg, "%s: %s", what, cudaGetErrorString(e));
    return HS_ERR_CUDA;
}

hs_status validate_common(const void* a, const void* b, const void* x0, const void* out, int64_t rows, int64_t n) {
    if (rows < 0 || n < 0) return HS_ERR_INVALID_ARG;
    if (rows == 0 || n == 0) return HS_OK;
    if (!a || !b || !x0 || !out) return HS_ERR_INVALID_ARG;
    if (rows > 0x7fffffffll) return HS_ERR_INVALID_ARG;
    if (n > kMaxN || rows > (1ll << 62) / n) return HS_ERR_INVALID_ARG;
    return HS_OK;
}

hs_status run(Problem& pr, void* workspace, size_t workspace_bytes, cudaStream_t stream, int force_path = 0) {
    Params& p = pr.p;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return HS_ERR_INVALID_ARG;
    if (workspace_bytes < sizeof(Header)) return HS_ERR_WORKSPACE_TOO_SMALL;

    DeviceInfo dev;
    hs_status st = device_info(dev);
    if (st != HS_OK) return st;
    if (dev.cc_major != 10) return HS_ERR_UNSUPPORTED_DEVICE;

    auto elem_size = [](hs_dtype d) { return d == HS_F32 ? 4 : d == HS_BF16 ? 2 : 8; };
    const int es_in = elem_size(pr.din), es_out = elem_size(pr.dout);
    bool tma = aligned16(p.in_a) && aligned16(p.in_b) && aligned16(p.out) && (p.n * es_in) % 16 == 0 &&
               (p.n * es_out) % 16 == 0 && p.n <= kMaxTmaDim && encode_fn() != nullptr;
    if (knob(kKnobNoTma, 0, 0, 1)) tma = false;
    pr.tma = tma;

    KernelEntry ke;
    if (!find_kernel(pr.mode, pr.din, pr.dout, tma, ke)) return HS_ERR_INVALID_ARG;
    const int path = force_path ? force_path : choose_path(p.rows, dev);
    const int chunk = 32 * (path == HS_PATH_BATCHED ? ke.K : ke.lb_K);  // elements per warp per step
    p.nchunks = (int)((p.n + chunk - 1) / chunk);
    p.sign_vec_ok = (p.n % 16 == 0) && (!p.sign_a || aligned16(p.sign_a)) && (!p.sign_b || aligned16(p.sign_b)) &&
                    (!p.sign_x || aligned16(p.sign_x));
    p.call_id = next_call_id();
    p.spin_limit = g_spin_limit.load();
    p.mute_tile = g_mute_tile.load();
    p.ws = reinterpret_cast<Header*>(workspace);

    int warps, stages, grid, lb_smem = 0;
    const void* fn;
    if (path == HS_PATH_BATCHED) {
        // R rows per warp (32/R lanes per row): the largest R that still leaves about a dozen warps
        // per SM, so that rows with many steps use few scan steps and few rows still fill the GPU.
        // (16 only where a row's piece of the output chunk, 2 lanes x K elements, still fills a 128-byte line)
        int R = (2 * ke.K * es_out >= 128) ? 16 : 8;
        while (R > 1 && (p.rows + R - 1) / R < (long long)kBatchedMinWarpsPerSm * dev.sm_count) R >>= 1;
        const int full_chunk = 32 * ke.K;  // columns of a chunk when the warp holds one row
        if (R == 16 && p.n >= full_chunk / 8) R = 8;  // 16 rows per warp only for rows shorter than an eighth of a chunk
        if (p.n < full_chunk) {
            // short rows: among the R allowed, the one whose chunks (full_chunk / R columns wide) pad the row
            // least, the larger R on a tie (fewer scan steps); 262144 x 128: R = 1 1.7 TB/s, R = 4 5.8 TB/s
            int best = R;
            long long best_cols = -1;
            for (int r = R; r >= 1; r >>= 1) {
                const int w = full_chunk / r;
                const long long cols = (p.n + w - 1) / w * w;  // columns processed per row
                if (best_cols < 0 || cols < best_cols) { best_cols = cols; best = r; }
            }
            R = best;
        } else if (p.rows >= (long long)kBatchedMinWarpsPerSm * dev.sm_count) {
            // enough rows: one row per warp, each chunk one TMA box of 128-byte lines (or, where TMA cannot
            // address the rows, sixteen coalesced steps along one row instead of two along each of eight)
            R = 1;
        }
        R = knob(kKnobRowsPerWarp, R, 1, 16);
        while (R & (R - 1)) R &= R - 1;  // power of two
        if (!tma && es_in == 8) R = 1;   // complex elements without TMA: only the one-row-per-warp staging moves 8-byte elements
        p.rows_per_warp = R;
        p.nchunks = (int)((p.n + (32 / R) * ke.K - 1) / ((32 / R) * ke.K));
        const long long groups = (p.rows + R - 1) / R;
        // loads run one chunk ahead of the arithmetic (the kernel keeps one row group ahead): TMA boxes, or
        // asynchronous 4-byte copies where TMA cannot address the rows; 2-byte elements are staged in step
        stages = (tma || es_in == 4 || R == 1) ? 2 : 1;  // (one row per warp: asynchronous 16-byte copies whatever the type)
        if (tma) stages = knob(kKnobStages, stages, 2, kMaxStages);  // deeper TMA pipelines are a knob
        int max_warps = 16;
        while (max_warps > 1 && max_warps * (stages * ke.warp_smem_per_stage + ke.warp_smem_out) + max_warps * 8 * kMaxStages +
                                        1024 > dev.max_smem_optin)
            --max_warps;
        long long per_sm = (groups + dev.sm_count - 1) / dev.sm_count;
        warps = (int)(per_sm < 1 ? 1 : (per_sm > max_warps ? max_warps : per_sm));
        warps = knob(kKnobWarps, warps, 1, 16);
        const long long ctas_needed = (groups + warps - 1) / warps;
        grid = (int)(ctas_needed < dev.sm_count ? ctas_needed : dev.sm_count);
        // tickets balance SMs of unequal speed when every warp slot sees several groups; with fewer, a
        // greedy hand-out of the last round loses more than it gains (cfg4, 1.7 groups per slot: 81 vs 74 us)
        // ... and only for rows of at least four chunks, where a ticket can be drawn early enough to arrive in time
        int tickets = (groups >= 4ll * grid * warps && p.nchunks >= 4) ? 1 : 0;
        tickets = knob(kKnobRowTickets, tickets, 0, 1);
        fn = tickets ? ke.batched_tk : ke.batched;
        // Between one and a few rows per warp slot, whole rows per slot leave the last round of slots partly idle:
        // share the rows' chunks out evenly instead (one row per warp, rows of at least two chunks, at least one row
        // per slot so that every share begins or ends inside a row at most once; the hand-over words need 16 bytes
        // per slot behind the workspace header).
        const long long slots = (long long)grid * warps;
        const long long rounds = (groups + slots - 1) / slots;
        // (worth it when whole rows per slot would keep the slots busy less than four fifths of the time; closer to
        // full rounds than that, the plain assignment is as fast while HBM is the limit and its loop is a little shorter)
        int spans = (!tickets && R == 1 && ke.batched_span && p.nchunks >= 2 && groups >= slots && stages == 2 &&
                     groups * 5 <= rounds * slots * 4 && workspace_bytes >= sizeof(Header) + (size_t)slots * 16)
                        ? 1 : 0;
        spans = knob(kKnobSpans, spans, 0, 1);
        if (spans && !(R == 1 && ke.batched_span && groups >= slots && !tickets && stages == 2 &&
                       workspace_bytes >= sizeof(Header) + (size_t)slots * 16))
            spans = 0;  // (the knob cannot force it onto shapes it does not cover)
        if (spans) {
            fn = ke.batched_span;
            p.desc = reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(workspace) + sizeof(Header));
        }
    } else {
        p.rows_per_warp = 1;
        // S input stages per compute warp (phase 2 of a tile runs S-2 iterations after its phase 1),
        // W compute warps (as many as shared memory allows, at most the default), NLB look-back warps
        stages = knob(kKnobLbStages, 4, 3, kLbMaxStages);
        const int nlb = 1;  // look-back (poller) warps per CTA
        int W = knob(kKnobLbWarps, kLookbackWarps, kLookbackMinWarps, kLbMaxWarps);
        if (stages > 5) stages = 5;
        while (W > kLookbackMinWarps && (ke.lb_smem(W, stages) + 1024 > dev.max_smem_optin || W + nlb + 1 > 16)) --W;
        lb_smem = ke.lb_smem(W, stages) + 1024;
        p.lb_warps = nlb;
        p.lb_sleep_idle = (unsigned)knob(kKnobLbSleepIdle, 200, 0, 100000);
        p.lb_sleep_ready = (unsigned)knob(kKnobLbSleepReady, 0, 0, 100000);
        warps = W + nlb + 1;  // + the publisher warp
        p.tiles_per_row = (int)lookback_tiles_per_row(p.n, chunk, W);
        p.num_tiles = p.rows * p.tiles_per_row;
        // rows of several tiles: two words per tile for its aggregate and one for the value entering it; every word
        // carries the call's id, so what the workspace held before does not matter and nothing is cleared
        p.lb_server = p.tiles_per_row > 1 ? 1 : 0;
        const size_t need = sizeof(Header) + (p.lb_server ? (size_t)p.num_tiles * 3 * 16 : 0);
        if (workspace_bytes < need) return HS_ERR_WORKSPACE_TOO_SMALL;
        p.desc = reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(workspace) + sizeof(Header));
        p.edesc = p.desc + 2 * p.num_tiles;
        fn = ke.lookback;
        grid = 0;  // set below from occupancy
    }

    CUtensorMap tm_a, tm_b, tm_o;
    std::memset(&tm_a, 0, sizeof tm_a);
    std::memset(&tm_b, 0, sizeof tm_b);
    std::memset(&tm_o, 0, sizeof tm_o);
    if (tma) {
        // one row per warp, rows of at least one whole 128-byte line: move a chunk as a single box of lines
        const bool flat = p.rows_per_warp == 1 && p.n * es_in >= 128 && p.n * es_out >= 128 &&
                          !knob(kKnobNoFlat, 0, 0, 1);
        p.flat_boxes = flat ? 1 : 0;
        const int br_in = flat ? chunk * es_in / 128 : p.rows_per_warp;
        const int br_out = flat ? chunk * es_out / 128 : p.rows_per_warp;
        if (!make_tmap(&tm_a, p.in_a, pr.din, p.rows, p.n, br_in, flat) ||
            !make_tmap(&tm_b, p.in_b, pr.din, p.rows, p.n, br_in, flat) ||
            !make_tmap(&tm_o, p.out, pr.dout, p.rows, p.n, br_out, flat)) {
            snprintf(g_cuda_msg, sizeof g_cuda_msg, "cuTensorMapEncodeTiled failed");
            return HS_ERR_CUDA;
        }
    }
    p.stages = stages;
    const int smem = path == HS_PATH_LOOKBACK
                         ? lb_smem
                         : warps * (stages * ke.warp_smem_per_stage + ke.warp_smem_out) + warps * 8 * kMaxStages + 1024;
    if (smem > dev.max_smem_optin) return HS_ERR_INVALID_ARG;
    cudaError_t e = ensure_smem_attr(fn, smem);
    if (e != cudaSuccess) return cuda_fail("cudaFuncSetAttribute", e);

    void* args[] = {&p, &tm_a, &tm_b, &tm_o};
    if (path == HS_PATH_LOOKBACK) {
        // Tiles wait for their predecessors, so every CTA must be resident: size the grid from the
        // occupancy of this kernel and launch cooperatively (the launch fails rather than deadlocks).
        int per_sm = 0;
        e = cached_occupancy(&per_sm, fn, warps * 32, smem);
        if (e != cudaSuccess) return cuda_fail("cudaOccupancyMaxActiveBlocksPerMultiprocessor", e);
        if (per_sm < 1) return HS_ERR_INVALID_ARG;
        per_sm = knob(kKnobLbCtasPerSm, per_sm, 1, per_sm);
        // (with the carry server: one CTA of the grid is the server, the others take the tiles)
        long long g = (long long)per_sm * dev.sm_count;
        if (g > p.num_tiles + p.lb_server) g = p.num_tiles + p.lb_server;
        grid = (int)g;
        if (p.tiles_per_row == 1) {
            // every row is a single tile: no tile waits for another, so neither the descriptors nor the
            // co-residency guarantee of a cooperative launch are needed
            // (programmatic stream serialisation: back-to-back small calls overlap their set-up with the previous
            // kernel's tail; the kernel waits before its first access to global memory)
            cudaLaunchConfig_t cfg;
            std::memset(&cfg, 0, sizeof cfg);
            cfg.gridDim = dim3(grid);
            cfg.blockDim = dim3(warps * 32);
            cfg.dynamicSmemBytes = (size_t)smem;
            cfg.stream = stream;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[0].val.programmaticStreamSerializationAllowed = knob(kKnobNoPdl, 0, 0, 1) ? 0 : 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            e = cudaLaunchKernelExC(&cfg, fn, args);
        } else {
            e = cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(warps * 32), args, smem, stream);
        }
    } else {
        // programmatic stream serialisation: the kernel's set-up may overlap the end of the previous kernel
        // of the stream; it waits (griddepcontrol.wait) before its first access to global memory
        cudaLaunchConfig_t cfg;
        std::memset(&cfg, 0, sizeof cfg);
        cfg.gridDim = dim3(grid);
        cfg.blockDim = dim3(warps * 32);
        cfg.dynamicSmemBytes = (size_t)smem;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = knob(kKnobNoPdl, 0, 0, 1) ? 0 : 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelExC(&cfg, fn, args);
    }
    if (e != cudaSuccess) return cuda_fail("kernel launch", e);
    g_last_path.store(path);
    g_launches.fetch_add(1);
    return HS_OK;
}

// Scratch of heinsen_scan_log_static(): lives in the library image, so every GPU that loads the
// library holds these bytes until the process exits.  In host code `g_static_scratch` is only a
// handle for the runtime; the device address comes from cudaGetSymbolAddress().
constexpr size_t kStaticScratchBytes = 1u << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Device address of g_static_scratch on the current device, looked up once per device.
hs_status static_scratch_address(void** out) {
    static std::mutex mu;
    static void* addr[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail("cudaGetDevice", e);
    if (dev < 0 || dev >= 64) return HS_ERR_UNSUPPORTED_DEVICE;
    std::lock_guard<std::mutex> lk(mu);
    if (!addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return cuda_fail("cudaGetSymbolAddress", e);
        addr[dev] = p;
    }
    *out = addr[dev];
    return HS_OK;
}

// Roofline probe: nothing but MUFU work.  Every thread advances kProbeChains independent chains
// x <- ex2(x), x <- lg2(x) held in registers; the values stay in (0, 1] x [-1, 0] and never leave the SM
// (one store per thread at the very end keeps the chains alive).
constexpr int kProbeChains = 8;
__global__ void __launch_bounds__(256) mufu_probe_kernel(int iterations, float seed, float* sink) {
    float x[kProbeChains];
#pragma unroll
    for (int c = 0; c < kProbeChains; ++c) x[c] = seed + 0.01f * (float)c + 1e-6f * (float)threadIdx.x;
#pragma unroll 1
    for (int i = 0; i < iterations; ++i) {
#pragma unroll
        for (int c = 0; c < kProbeChains; ++c) x[c] = hs::ex2(-x[c]);  // (0, 1]
#pragma unroll
        for (int c = 0; c < kProbeChains; ++c) x[c] = -hs::lg2(x[c]);  // back to >= 0
    }
    float acc = 0.0f;
#pragma unroll
    for (int c = 0; c < kProbeChains; ++c) acc += x[c];
    if (acc == 123456.0f) sink[threadIdx.x] = acc;  // never true in practice
}

}  // namespace

// =============================================================================================
extern "C" {

hs_status heinsen_scan_probe_mufu(int iterations, double* results, double* seconds) {
    if (iterations <= 0 || !results || !seconds) return HS_ERR_INVALID_ARG;
    DeviceInfo dev;
    hs_status st = device_info(dev);
    if (st != HS_OK) return st;
    if (dev.cc_major != 10) return HS_ERR_UNSUPPORTED_DEVICE;
    void* scratch = nullptr;
    st = static_scratch_address(&scratch);
    if (st != HS_OK) return st;
    const int threads = 256, blocks = dev.sm_count * 8;  // 64 warps per SM: every MUFU unit has work queued
    cudaEvent_t e0, e1;
    cudaError_t e;
    if ((e = cudaEventCreate(&e0)) != cudaSuccess) return cuda_fail("cudaEventCreate", e);
    if ((e = cudaEventCreate(&e1)) != cudaSuccess) { cudaEventDestroy(e0); return cuda_fail("cudaEventCreate", e); }
    // the sink is never written (see the kernel); the library's fixed array only gives it a valid address
    float* sink = static_cast<float*>(scratch);
    mufu_probe_kernel<<<blocks, threads>>>(16, 0.5f, sink);  // warm-up
    cudaEventRecord(e0);
    mufu_probe_kernel<<<blocks, threads>>>(iterations, 0.5f, sink);
    cudaEventRecord(e1);
    e = cudaEventSynchronize(e1);
    float ms = 0.0f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (e != cudaSuccess) return cuda_fail("mufu probe", e);
    g_launches.fetch_add(2);
    *results = (double)blocks * threads * (double)iterations * kProbeChains * 2.0;
    *seconds = (double)ms * 1e-3;
    return HS_OK;
}

hs_status heinsen_scan_linear(const void* a, const void* b, const void* x0, void* x, int64_t rows, int64_t n,
                              hs_dtype dtype, void* workspace, size_t workspace_bytes, void* stream) {
    hs_status st = validate_common(a, b, x0, x, rows, n);
    if (st != HS_OK || rows == 0 || n == 0) return st;
    if (dtype != HS_F32) return HS_ERR_INVALID_ARG;
    Problem pr;
    std::memset(&pr, 0, sizeof pr);
    pr.mode = kLinear;
    pr.din = pr.dout = dtype;
    pr.p.in_a = a; pr.p.in_b = b; pr.p.x0 = x0; pr.p.out = x;
    pr.p.rows = rows; pr.p.n = n;
    return run(pr, workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
}

hs_status heinsen_scan_linear_pairs(const void* a, const void* b, const void* x0, void* x, int64_t rows, int64_t n,
                                    hs_dtype dtype, void* workspace, size_t workspace_bytes, void* stream) {
    hs_status st = validate_common(a, b, x0, x, rows, n);
    if (st != HS_OK || rows == 0 || n == 0) return st;
    if (dtype != HS_F32) return HS_ERR_INVALID_ARG;
    Problem pr;
    std::memset(&pr, 0, sizeof pr);
    pr.mode = kPairs;
    pr.din = pr.dout = dtype;
    pr.p.in_a = a; pr.p.in_b = b; pr.p.x0 = x0; pr.p.out = x;
    pr.p.rows = rows; pr.p.n = n;
    return run(pr, workspace, workspace_bytes, static_cast<cudaStream_t>(stream), HS_PATH_BATCHED);
}

hs_status heinsen_scan_log(const void* log_a, const void* log_b, const void* log_x0, void* log_x,
                           const uint8_t* sign_a, const uint8_t* sign_b, const uint8_t* sign_x0, uint8_t* sign_x,
                           int64_t rows, int64_t n, hs_dtype dtype_in, hs_dtype dtype_out, void* workspace,
                           size_t workspace_bytes, void* stream) {
    hs_status st = validate_common(log_a, log_b, log_x0, log_x, rows, n);
    if (st != HS_OK || rows == 0 || n == 0) return st;
    if ((dtype_in != HS_F32 && dtype_in != HS_BF16) || (dtype_out != HS_F32 && dtype_out != HS_BF16))
        return HS_ERR_INVALID_ARG;
    if (dtype_in == HS_BF16 && dtype_out == HS_F32) return HS_ERR_INVALID_ARG;
    const bool is_signed = sign_a || sign_b || sign_x0;
    if (is_signed && !sign_x) return HS_ERR_INVALID_ARG;
    Problem pr;
    std::memset(&pr, 0, sizeof pr);
    pr.mode = is_signed ? kLogSigned : kLogUnsigned;
    pr.din = dtype_in; pr.dout = dtype_out;
    pr.p.in_a = log_a; pr.p.in_b = log_b; pr.p.x0 = log_x0; pr.p.out = log_x;
    if (is_signed) { pr.p.sign_a = sign_a; pr.p.sign_b = sign_b; pr.p.sign_x0 = sign_x0; pr.p.sign_x = sign_x; }
    pr.p.rows = rows; pr.p.n = n;
    return run(pr, workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
}

hs_status heinsen_scan_log_static(const void* log_a, const void* log_b, const void* log_x0, void* log_x, int64_t rows,
                                  int64_t n, void* stream) {
    hs_status st = validate_common(log_a, log_b, log_x0, log_x, rows, n);
    if (st != HS_OK || rows == 0 || n == 0) return st;
    // the descriptors of every tile of the problem must fit the fixed array
    if (workspace_bytes_for(rows, n) > kStaticScratchBytes) return HS_ERR_WORKSPACE_TOO_SMALL;
    void* scratch = nullptr;
    st = static_scratch_address(&scratch);
    if (st != HS_OK) return st;
    Problem pr;
    std::memset(&pr, 0, sizeof pr);
    pr.mode = kLogUnsigned;
    pr.din = pr.dout = HS_F32;
    pr.p.in_a = log_a; pr.p.in_b = log_b; pr.p.x0 = log_x0; pr.p.out = log_x;
    pr.p.rows = rows; pr.p.n = n;
    // every descriptor the kernel reads carries the call's id, so what the previous call left in the
    // array does not matter
    return run(pr, scratch, kStaticScratchBytes, static_cast<cudaStream_t>(stream), HS_PATH_LOOKBACK);
}

// Complex-logarithm interface (Summary, last paragraph: the logarithm of a negative value is complex,
// log r + i*pi on the principal branch).  Values arrive and leave as complex64; the kernels read the
// magnitude from the real part and one sign bit from the imaginary part of every element as it comes out of
// shared memory, and write (log|x|, 0 or pi): 24 bytes per element of traffic, the representation's own.
size_t heinsen_scan_complex_workspace_bytes(int64_t rows, int64_t n) {
    if (rows <= 0 || n <= 0 || rows > 0x7fffffffll || n > kMaxN || rows > (1ll << 62) / n) return 0;
    return workspace_bytes_for(rows, n, kComplexChunk);
}

hs_status heinsen_scan_log_complex(const void* log_a, const void* log_b, const void* log_x0, void* log_x, int64_t rows,
                                   int64_t n, void* workspace, size_t workspace_bytes, void* stream) {
    hs_status st = validate_common(log_a, log_b, log_x0, log_x, rows, n);
    if (st != HS_OK || rows == 0 || n == 0) return st;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return HS_ERR_INVALID_ARG;
    if (workspace_bytes < workspace_bytes_for(rows, n, kComplexChunk)) return HS_ERR_WORKSPACE_TOO_SMALL;
    if (n > kMaxN / 2) return HS_ERR_INVALID_ARG;  // a row of 2n floats must still fit the 32-bit column indices
    Problem pr;
    std::memset(&pr, 0, sizeof pr);
    pr.mode = kLogSigned;
    pr.din = pr.dout = kC64;
    pr.p.in_a = log_a; pr.p.in_b = log_b; pr.p.x0 = log_x0; pr.p.out = log_x;
    pr.p.rows = rows; pr.p.n = n;
    return run(pr, workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
}

hs_status scan_linear(const void* a, const void* b, const void* x0, void* x, int64_t rows, int64_t n) {
    hs_status st = validate_common(a, b, x0, x, rows, n);
    if (st != HS_OK || rows == 0 || n == 0) return st;
    void* scratch = nullptr;
    st = static_scratch_address(&scratch);
    if (st != HS_OK) return st;
    return heinsen_scan_linear(a, b, x0, x, rows, n, HS_F32, scratch, kStaticScratchBytes, nullptr);
}

hs_status scan_log(const void* log_a, const void* log_b, const void* log_x0, void* log_x, const uint8_t* sign_a,
                   const uint8_t* sign_b, const uint8_t* sign_x0, uint8_t* sign_x, int64_t rows, int64_t n) {
    hs_status st = validate_common(log_a, log_b, log_x0, log_x, rows, n);
    if (st != HS_OK || rows == 0 || n == 0) return st;
    if ((sign_a || sign_b || sign_x0) && !sign_x) return HS_ERR_INVALID_ARG;
    void* scratch = nullptr;
    st = static_scratch_address(&scratch);
    if (st != HS_OK) return st;
    return heinsen_scan_log(log_a, log_b, log_x0, log_x, sign_a, sign_b, sign_x0, sign_x, rows, n, HS_F32, HS_F32, scratch,
                            kStaticScratchBytes, nullptr);
}

hs_status heinsen_scan_check_static(void* stream) {
    void* scratch = nullptr;
    hs_status st = static_scratch_address(&scratch);
    if (st != HS_OK) return st;
    return heinsen_scan_check(scratch, stream);
}

size_t heinsen_scan_static_max_elements(void) {
    // workspace_bytes_for() grows with rows * ceil(n / 4096); this is the single-row capacity
    size_t lo = 0, hi = (size_t)1 << 31;
    while (hi - lo > 1) {
        const size_t mid = lo + (hi - lo) / 2;
        if (mid <= (size_t)kMaxN && workspace_bytes_for(1, (long long)mid) <= kStaticScratchBytes) lo = mid;
        else hi = mid;
    }
    return lo;
}

size_t heinsen_scan_workspace_bytes(int64_t rows, int64_t n) {
    if (rows <= 0 || n <= 0) return 0;
    if (rows > 0x7fffffffll || n > kMaxN || rows > (1ll << 62) / n) return 0;
    return workspace_bytes_for(rows, n);
}

hs_status heinsen_scan_check(const void* workspace, void* stream) {
    if (!workspace) return HS_ERR_INVALID_ARG;
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail("cudaStreamSynchronize", e);
    Header h;
    e = cudaMemcpy(&h, workspace, sizeof h, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail("cudaMemcpy", e);
    if (h.error_id == h.started_id && h.started_id != 0 &&
        (h.error_code == HS_ERR_LOOKBACK_TIMEOUT || h.error_code == HS_ERR_COPY_TIMEOUT))
        return static_cast<hs_status>(h.error_code);
    return HS_OK;
}

hs_status heinsen_scan_set_path(hs_path path) {
    if (path != HS_PATH_AUTO && path != HS_PATH_BATCHED && path != HS_PATH_LOOKBACK) return HS_ERR_INVALID_ARG;
    g_path.store(path);
    return HS_OK;
}
hs_status heinsen_scan_debug_config(uint32_t lookback_spin_limit, int64_t mute_tile) {
    g_spin_limit.store(lookback_spin_limit ? lookback_spin_limit : hs::kLookbackSpinLimit);
    g_mute_tile.store(mute_tile);
    return HS_OK;
}
int heinsen_scan_debug_faults(uint64_t out[4]) {
    if (out) out[0] = out[1] = out[2] = out[3] = 0;
#ifdef HEINSEN_DEBUG
    unsigned long long f[4] = {0, 0, 0, 0};
    if (cudaDeviceSynchronize() != cudaSuccess) return -1;
    if (cudaMemcpyFromSymbol(f, hs::g_debug_fault, sizeof f) != cudaSuccess) return -1;
    if (f[0] != 0) {
        const unsigned long long zero[4] = {0, 0, 0, 0};
        if (cudaMemcpyToSymbol(hs::g_debug_fault, zero, sizeof zero) != cudaSuccess) return -1;
    }
    if (out) for (int i = 0; i < 4; ++i) out[i] = f[i];
    return f[0] != 0 ? 1 : 0;
#else
    return 0;
#endif
}
int heinsen_scan_debug_build(void) {
#ifdef HEINSEN_DEBUG
    return 1;
#else
    return 0;
#endif
}
int heinsen_scan_debug_window_ok(uint64_t addr, uint64_t bytes, uint64_t base, uint64_t size, uint64_t align) {
    if (align == 0) return 0;
    return hs::debug_window_ok(addr, bytes, base, size, align) ? 1 : 0;
}

hs_status heinsen_scan_tune(const char* name, int value) {
    if (!name) return HS_ERR_INVALID_ARG;
    std::call_once(g_knobs_once, load_knobs_from_env);
    for (int k = 0; k < kKnobCount; ++k) {
        if (std::strcmp(name, kKnobNames[k]) == 0) {
            g_knobs[k].store(value < 0 ? kKnobUnset : value);
            return HS_OK;
        }
    }
    return HS_ERR_INVALID_ARG;
}
int heinsen_scan_last_path(void) { return g_last_path.load(); }
int64_t heinsen_scan_launch_count(void) { return g_launches.load(); }

const char* heinsen_scan_strerror(hs_status status) {
    switch (status) {
        case HS_OK: return "ok";
        case HS_ERR_INVALID_ARG: return "invalid argument (null pointer, bad size, unsupported type or misaligned workspace)";
        case HS_ERR_UNSUPPORTED_DEVICE: return "unsupported device: this library runs on sm_100 (B200) only";
        case HS_ERR_WORKSPACE_TOO_SMALL: return "workspace too small: see heinsen_scan_workspace_bytes()";
        case HS_ERR_CUDA: return g_cuda_msg[0] ? g_cuda_msg : "CUDA runtime error";
        case HS_ERR_LOOKBACK_TIMEOUT: return "device: a tile's bounded wait for its predecessors ran out";
        case HS_ERR_COPY_TIMEOUT: return "device: a bounded wait for an asynchronous chunk copy ran out";
    }
    return "unknown status";
}

// ---------------------------------------------------------------------------------------------
// Host-buffer variants: copy in, run, copy out, on `stream`; synchronise before returning.
constexpr int kHostBlocks = 8;  // row blocks of the host-buffer entry points (copy/compute overlap)

static int host_blocks(int64_t rows) { return rows < kHostBlocks ? (int)rows : kHostBlocks; }
static size_t up256(size_t v) { return (v + 255) & ~size_t(255); }

size_t heinsen_scan_host_scratch_bytes(int64_t rows, int64_t n, hs_dtype dtype_in, hs_dtype dtype_out, int with_signs) {
    if (rows <= 0 || n <= 0) return 0;
    const size_t es_in = dtype_in == HS_F32 ? 4 : 2, es_out = dtype_out == HS_F32 ? 4 : 2;
    const size_t cnt = (size_t)rows * (size_t)n;
    const int nblk = host_blocks(rows);
    const int64_t rows_blk = (rows + nblk - 1) / nblk;
    size_t total = (size_t)nblk * up256(workspace_bytes_for(rows_blk, n));
    total += 2 * up256(cnt * es_in) + up256((size_t)rows * es_in) + up256(cnt * es_out);
    if (with_signs) total += 3 * up256(cnt) + up256((size_t)rows);
    return total;
}

namespace {
// Two side streams per device so that the host->device copy of one row block overlaps the
// device->host copy of the previous one (PCIe is full duplex) and the kernels in between.
struct HostLanes {
    cudaStream_t side[2] = {nullptr, nullptr};
    cudaEvent_t start = nullptr, done[2] = {nullptr, nullptr};
    bool ok = false;
    std::mutex busy;  // host-buffer calls on one device share the side streams and events: one at a time
};
hs_status host_lanes(HostLanes** out) {
    static std::mutex mu;
    static HostLanes lanes[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail("cudaGetDevice", e);
    if (dev < 0 || dev >= 64) return HS_ERR_UNSUPPORTED_DEVICE;
    std::lock_guard<std::mutex> lk(mu);
    HostLanes& h = lanes[dev];
    if (!h.ok) {
        for (int i = 0; i < 2; ++i) {
            if ((e = cudaStreamCreateWithFlags(&h.side[i], cudaStreamNonBlocking)) != cudaSuccess)
                return cuda_fail("cudaStreamCreateWithFlags", e);
            if ((e = cudaEventCreateWithFlags(&h.done[i], cudaEventDisableTiming)) != cudaSuccess)
                return cuda_fail("cudaEventCreateWithFlags", e);
        }
        if ((e = cudaEventCreateWithFlags(&h.start, cudaEventDisableTiming)) != cudaSuccess)
            return cuda_fail("cudaEventCreateWithFlags", e);
        h.ok = true;
    }
    *out = &h;
    return HS_OK;
}
}  // namespace

static hs_status host_run(int linear, const void* a, const void* b, const void* x0, void* x, const uint8_t* sa,
                          const uint8_t* sb, const uint8_t* sx0, uint8_t* sx, int64_t rows, int64_t n, hs_dtype din,
                          hs_dtype dout, void* scratch, size_t scratch_bytes, cudaStream_t stream) {
    hs_status st = validate_common(a, b, x0, x, rows, n);
    if (st != HS_OK || rows == 0 || n == 0) return st;
    const bool with_signs = sa || sb || sx0;
    if (with_signs && !sx) return HS_ERR_INVALID_ARG;
    if (!scratch || (reinterpret_cast<uintptr_t>(scratch) & 255u)) return HS_ERR_INVALID_ARG;
    if (scratch_bytes < heinsen_scan_host_scratch_bytes(rows, n, din, dout, with_signs)) return HS_ERR_WORKSPACE_TOO_SMALL;
    const size_t es_in = din == HS_F32 ? 4 : 2, es_out = dout == HS_F32 ? 4 : 2;
    const size_t cnt = (size_t)rows * (size_t)n;
    const int nblk = host_blocks(rows);
    const int64_t rows_blk = (rows + nblk - 1) / nblk;
    const size_t ws_bytes = workspace_bytes_for(rows_blk, n);

    uint8_t* w = static_cast<uint8_t*>(scratch);
    uint8_t* ws0 = w;             w += (size_t)nblk * up256(ws_bytes);
    uint8_t* d_a = w;             w += up256(cnt * es_in);
    uint8_t* d_b = w;             w += up256(cnt * es_in);
    uint8_t* d_x0 = w;            w += up256((size_t)rows * es_in);
    uint8_t* d_x = w;             w += up256(cnt * es_out);
    uint8_t *d_sa = nullptr, *d_sb = nullptr, *d_sx0 = nullptr, *d_sx = nullptr;
    if (with_signs) {
        d_sa = w; w += up256(cnt);
        d_sb = w; w += up256(cnt);
        d_sx = w; w += up256(cnt);
        d_sx0 = w; w += up256((size_t)rows);
    }
    HostLanes* hl = nullptr;
    st = host_lanes(&hl);
    if (st != HS_OK) return st;
    std::lock_guard<std::mutex> one_at_a_time(hl->busy);
    cudaError_t e;
#define HS_TRY(call)                                          \
    do {                                                      \
        e = (call);                                           \
        if (e != cudaSuccess) return cuda_fail(#call, e);     \
    } while (0)
    // x_0 of all rows goes first, in one copy, on the caller's stream
    HS_TRY(cudaMemcpyAsync(d_x0, x0, (size_t)rows * es_in, cudaMemcpyHostToDevice, stream));
    if (sx0) HS_TRY(cudaMemcpyAsync(d_sx0, sx0, (size_t)rows, cudaMemcpyHostToDevice, stream));
    // the side streams start after everything already queued on the caller's stream
    HS_TRY(cudaEventRecord(hl->start, stream));
    HS_TRY(cudaStreamWaitEvent(hl->side[0], hl->start, 0));
    HS_TRY(cudaStreamWaitEvent(hl->side[1], hl->start, 0));
    const uint8_t *ha = static_cast<const uint8_t*>(a), *hb = static_cast<const uint8_t*>(b);
    uint8_t* hx = static_cast<uint8_t*>(x);
    // On an error return nothing may stay in flight to or from the caller's host buffers.
    auto quiesce = [&]() {
        cudaStreamSynchronize(hl->side[0]);
        cudaStreamSynchronize(hl->side[1]);
        cudaStreamSynchronize(stream);
    };
#define HS_TRY_Q(call)                                        \
    do {                                                      \
        e = (call);                                           \
        if (e != cudaSuccess) {                               \
            quiesce();                                        \
            return cuda_fail(#call, e);                       \
        }                                                     \
    } while (0)
    int launched = 0;  // row blocks actually launched (the last ones may be empty)
    for (int k = 0; k < nblk; ++k) {
        const int64_t r0 = (int64_t)k * rows_blk;
        const int64_t rb = rows - r0 < rows_blk ? rows - r0 : rows_blk;
        if (rb <= 0) break;
        cudaStream_t s = hl->side[k & 1];
        const size_t e0 = (size_t)r0 * (size_t)n, ec = (size_t)rb * (size_t)n;
        HS_TRY_Q(cudaMemcpyAsync(d_a + e0 * es_in, ha + e0 * es_in, ec * es_in, cudaMemcpyHostToDevice, s));
        HS_TRY_Q(cudaMemcpyAsync(d_b + e0 * es_in, hb + e0 * es_in, ec * es_in, cudaMemcpyHostToDevice, s));
        if (sa) HS_TRY_Q(cudaMemcpyAsync(d_sa + e0, sa + e0, ec, cudaMemcpyHostToDevice, s));
        if (sb) HS_TRY_Q(cudaMemcpyAsync(d_sb + e0, sb + e0, ec, cudaMemcpyHostToDevice, s));
        void* ws = ws0 + (size_t)k * up256(ws_bytes);
        if (linear)
            st = heinsen_scan_linear(d_a + e0 * es_in, d_b + e0 * es_in, d_x0 + (size_t)r0 * es_in, d_x + e0 * es_out, rb, n,
                                     din, ws, ws_bytes, s);
        else
            st = heinsen_scan_log(d_a + e0 * es_in, d_b + e0 * es_in, d_x0 + (size_t)r0 * es_in, d_x + e0 * es_out,
                                  sa ? d_sa + e0 : nullptr, sb ? d_sb + e0 : nullptr, sx0 ? d_sx0 + r0 : nullptr,
                                  with_signs ? d_sx + e0 : nullptr, rb, n, din, dout, ws, ws_bytes, s);
        if (st != HS_OK) {
            quiesce();
            return st;
        }
        ++launched;
        HS_TRY_Q(cudaMemcpyAsync(hx + e0 * es_out, d_x + e0 * es_out, ec * es_out, cudaMemcpyDeviceToHost, s));
        if (with_signs) HS_TRY_Q(cudaMemcpyAsync(sx + e0, d_sx + e0, ec, cudaMemcpyDeviceToHost, s));
    }
    for (int i = 0; i < 2; ++i) {
        HS_TRY_Q(cudaEventRecord(hl->done[i], hl->side[i]));
        HS_TRY_Q(cudaStreamWaitEvent(stream, hl->done[i], 0));
    }
#undef HS_TRY_Q
#undef HS_TRY
    // one synchronisation and one strided read-back of the status words of the row blocks that ran
    e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return cuda_fail("cudaStreamSynchronize", e);
    Header heads[kHostBlocks];
    e = cudaMemcpy2D(heads, sizeof(Header), ws0, up256(ws_bytes), sizeof(Header), (size_t)launched, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail("cudaMemcpy2D", e);
    for (int k = 0; k < launched; ++k) {
        const Header& h = heads[k];
        if (h.error_id == h.started_id && h.started_id != 0 &&
            (h.error_code == HS_ERR_LOOKBACK_TIMEOUT || h.error_code == HS_ERR_COPY_TIMEOUT))
            return static_cast<hs_status>(h.error_code);
    }
    return HS_OK;
}

hs_status heinsen_scan_linear_host(const void* a, const void* b, const void* x0, void* x, int64_t rows, int64_t n,
                                   hs_dtype dtype, void* device_scratch, size_t device_scratch_bytes, void* stream) {
    if (dtype != HS_F32) return (rows == 0 || n == 0) ? HS_OK : HS_ERR_INVALID_ARG;
    return host_run(1, a, b, x0, x, nullptr, nullptr, nullptr, nullptr, rows, n, dtype, dtype, device_scratch,
                    device_scratch_bytes, static_cast<cudaStream_t>(stream));
}

hs_status heinsen_scan_log_host(const void* log_a, const void* log_b, const void* log_x0, void* log_x,
                                const uint8_t* sign_a, const uint8_t* sign_b, const uint8_t* sign_x0, uint8_t* sign_x,
                                int64_t rows, int64_t n, hs_dtype dtype_in, hs_dtype dtype_out, void* device_scratch,
                                size_t device_scratch_bytes, void* stream) {
    if ((dtype_in != HS_F32 && dtype_in != HS_BF16) || (dtype_out != HS_F32 && dtype_out != HS_BF16) ||
        (dtype_in == HS_BF16 && dtype_out == HS_F32))
        return (rows == 0 || n == 0) ? HS_OK : HS_ERR_INVALID_ARG;
    return host_run(0, log_a, log_b, log_x0, log_x, sign_a, sign_b, sign_x0, sign_x, rows, n, dtype_in, dtype_out,
                    device_scratch, device_scratch_bytes, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
