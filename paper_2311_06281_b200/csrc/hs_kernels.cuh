// Kernels of libheinsen_scan (sm_100a only).
//
//   batched_scan_kernel  : one warp walks one row chunk by chunk, the value of x carried in
//                          registers from chunk to chunk (rows >= a few per SM).
//   lookback_scan_kernel : rows are cut into tiles of WARPS chunks; one CTA per tile, single
//                          pass, the carry between tiles found by decoupled look-back over
//                          per-tile descriptors in the caller's workspace (few, long rows).
//
// Both read every input element once and write every output element once.  Chunks travel
// HBM -> shared memory by TMA (per-warp mbarrier pipelines, 128-byte swizzle) and back by TMA
// stores; the scans themselves run in registers (hs_device.cuh).
#pragma once
#include <cuda.h>

#include "hs_device.cuh"

namespace hs {

constexpr int kMaxStages = 4;
constexpr uint32_t kCopySpinLimit = 1u << 22;      // try_wait polls (each up to ~1 us in hardware)
constexpr uint32_t kLookbackSpinLimit = 1u << 20;  // polls of predecessor flags (each an L2 round trip)

// Status codes written to the workspace header (mirrors hs_status).
constexpr int kErrLookbackTimeout = 5;
constexpr int kErrCopyTimeout = 6;

// First 256 bytes of the caller's workspace.
struct Header {
    unsigned long long started_id;  // id of the call that last started on this workspace
    unsigned long long error_id;    // id of the call that recorded `error_code`
    int error_code;
    int error_where;                // tile or row index, for diagnosis
    unsigned long long reserved[29];
};
static_assert(sizeof(Header) == 256, "workspace header is 256 bytes");

struct Params {
    const void* in_a;
    const void* in_b;
    const void* x0;
    void* out;
    const uint8_t* sign_a;
    const uint8_t* sign_b;
    const uint8_t* sign_x0;
    uint8_t* sign_x;
    long long rows;
    long long n;
    int nchunks;        // chunks per row
    int stages;         // input stages per warp (2..kMaxStages)
    int sign_vec_ok;    // sign tensors may be accessed with 16-byte vectors
    unsigned long long call_id;
    Header* ws;
    // look-back kernel only
    int tiles_per_row;
    long long num_tiles;
    unsigned long long* flags;  // [num_tiles] (call_id << 2) | state
    float4* agg;                // [num_tiles] tile aggregate (A, m, s, p)
    float4* inc;                // [num_tiles] value of x after the tile (m, s, -, -)
    unsigned int spin_limit;    // bound on polls of predecessor flags
    long long mute_tile;        // test hook: this tile never publishes (-1: none)
};

// The first thread to report an error in this call records it; heinsen_scan_check() reports it
// when error_id equals started_id.
__device__ __forceinline__ void record_error(const Params& p, int code, long long where) {
    Header* h = p.ws;
    if (atomicExch(&h->error_id, p.call_id) != p.call_id) {
        h->error_code = code;
        h->error_where = (int)where;
    }
}

// Neutral padding of a ragged row tail: a = 1 (log a = 0), b = 0 (log b = -inf).
template <int MODE>
__device__ __forceinline__ float neutral_a() { return MODE == kLinear ? 1.0f : 0.0f; }
template <int MODE>
__device__ __forceinline__ float neutral_b() { return MODE == kLinear ? 0.0f : neg_inf(); }

// ------------------------------------------------------------------------------------------
// Per-warp chunk engine shared by both kernels: everything between "the chunk's inputs are in
// shared memory" and "the chunk's outputs are in shared memory".
template <int MODE, typename TIn, typename TOut, int K>
struct ChunkEngine {
    using R = Run<MODE, TIn, TOut, K>;
    static constexpr bool SIGNED = R::SIGNED;
    using E = Elem<SIGNED>;

    // sign masks of the lane's K elements from a uint8 tensor (0/1 per element)
    __device__ static __forceinline__ void load_signs(const uint8_t* g, long long base, long long col0, long long n,
                                                      bool vec, uint32_t* mask) {
        if (g == nullptr) {
#pragma unroll
            for (int t = 0; t < K; ++t) mask[t] = 0u;
            return;
        }
        if (vec && col0 + K <= n) {
#pragma unroll
            for (int j = 0; j < K / 16; ++j) {
                const uint4 v = __ldg(reinterpret_cast<const uint4*>(g + base + col0 + 16 * j));
                const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int t = 0; t < 16; ++t) mask[16 * j + t] = (w[t >> 2] << (31 - 8 * (t & 3))) & kSignBit;
            }
        } else {
#pragma unroll
            for (int t = 0; t < K; ++t) mask[t] = (col0 + t < n) ? (((uint32_t)g[base + col0 + t] & 1u) << 31) : 0u;
        }
    }
    __device__ static __forceinline__ void store_signs(uint8_t* g, long long base, long long col0, long long n,
                                                       bool vec, const uint32_t* mask) {
        if (vec && col0 + K <= n) {
#pragma unroll
            for (int j = 0; j < K / 16; ++j) {
                uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
                for (int t = 0; t < 16; ++t) w[t >> 2] |= (mask[16 * j + t] >> 31) << (8 * (t & 3));
                *reinterpret_cast<uint4*>(g + base + col0 + 16 * j) = make_uint4(w[0], w[1], w[2], w[3]);
            }
        } else {
#pragma unroll
            for (int t = 0; t < K; ++t)
                if (col0 + t < n) g[base + col0 + t] = (uint8_t)(mask[t] >> 31);
        }
    }

    // Tracked form, pass 1: the lane's run as one part, every step with its own reference.
    __device__ static __noinline__ E slow_pass1(const uint8_t* sm_a, const uint8_t* sm_b, int lane, const uint8_t* gsa,
                                                const uint8_t* gsb, long long gbase, int valid) {
        E e = identity_elem<SIGNED>();
        for (int t = 0; t < K; ++t) {
            const int i = lane * K + t;
            if (i < valid) {
                const uint32_t sa = gsa ? (((uint32_t)gsa[gbase + i] & 1u) << 31) : 0u;
                const uint32_t sb = gsb ? (((uint32_t)gsb[gbase + i] & 1u) << 31) : 0u;
                e = compose(e, Leaf<MODE, TIn>::get(sm_a, sm_b, (uint32_t)i, sa, sb));
            }
        }
        return e;
    }
    // Tracked form, pass 2: step the value through the lane's run and write each output.
    __device__ static __noinline__ void slow_apply(E st, const uint8_t* sm_a, const uint8_t* sm_b, uint8_t* sm_out,
                                                   int lane, const uint8_t* gsa, const uint8_t* gsb, uint8_t* gsx,
                                                   long long gbase, int valid) {
        for (int t = 0; t < K; ++t) {
            const int i = lane * K + t;
            if (i < valid) {
                const uint32_t sa = gsa ? (((uint32_t)gsa[gbase + i] & 1u) << 31) : 0u;
                const uint32_t sb = gsb ? (((uint32_t)gsb[gbase + i] & 1u) << 31) : 0u;
                st = compose(st, Leaf<MODE, TIn>::get(sm_a, sm_b, (uint32_t)i, sa, sb));
                renormalise(st);
                float v;
                if (MODE == kLinear) {
                    const float h = ex2(st.m * (0.5f * kLog2e));
                    v = (st.s * h) * h;
                    if (st.s == 0.0f) v = 0.0f;
                } else {
                    v = fmaf(lg2(fabsf(st.s)), kLn2, st.m);
                    if (st.s == 0.0f) v = neg_inf();
                }
                Storage<TOut>::to_smem(sm_out, (uint32_t)i, v);
                if (MODE == kLogSigned && gsx) gsx[gbase + i] = (st.s < 0.0f) ? 1 : 0;
            }
        }
    }

    // Runs the chunk.  `entering_chunk` is the value of x entering the chunk when `known` is
    // true (batched kernel).  Returns the chunk's aggregate through `total`; writes outputs to
    // sm_out.  The look-back kernel calls the two halves separately (see below).
    struct Pending {  // what phase 2 needs from phase 1
        R run;
        E excl;       // parts of this chunk before the lane's run
        bool slow;
    };

    __device__ static __forceinline__ void phase1(const Params& p, const uint8_t* sm_a, const uint8_t* sm_b, int lane,
                                                  long long row, int chunk, Pending& pd, E& total) {
        float va[K], vb[K];
        uint32_t sa[SIGNED ? K : 1], sb[SIGNED ? K : 1];
        R::load(sm_a, sm_b, lane, va, vb);
        const long long col0 = (long long)chunk * R::CHUNK + lane * K;
        const long long gbase = row * p.n;
        if ((long long)(chunk + 1) * R::CHUNK > p.n) {
#pragma unroll
            for (int t = 0; t < K; ++t) {
                if (col0 + t >= p.n) { va[t] = neutral_a<MODE>(); vb[t] = neutral_b<MODE>(); }
            }
        }
        if (MODE == kLogSigned) {
            load_signs(p.sign_a, gbase, col0, p.n, p.sign_vec_ok != 0, sa);
            load_signs(p.sign_b, gbase, col0, p.n, p.sign_vec_ok != 0, sb);
        }
        E agg = pd.run.pass1(va, vb, sa, sb);
        pd.slow = __any_sync(0xffffffffu, pd.run.bad);
        if (pd.slow) {
            const long long rem = p.n - (long long)chunk * R::CHUNK;
            const int valid = rem < R::CHUNK ? (int)rem : R::CHUNK;
            agg = slow_pass1(sm_a, sm_b, lane, MODE == kLogSigned ? p.sign_a : nullptr,
                             MODE == kLogSigned ? p.sign_b : nullptr, gbase + (long long)chunk * R::CHUNK, valid);
        }
        warp_scan(agg, lane, pd.excl, total);
    }

    // `entering_chunk`: value of x entering the chunk.
    __device__ static __forceinline__ void phase2(const Params& p, const uint8_t* sm_a, const uint8_t* sm_b,
                                                  uint8_t* sm_out, int lane, long long row, int chunk,
                                                  const Pending& pd, const E& entering_chunk) {
        const E entering = compose(entering_chunk, pd.excl);
        const long long col0 = (long long)chunk * R::CHUNK + lane * K;
        const long long gbase = row * p.n;
        float out_mag[K];
        uint32_t out_sign[MODE == kLogSigned ? K : 1];
        bool ok = false;
        if (!pd.slow) ok = pd.run.apply(entering, out_mag, out_sign);
        ok = __all_sync(0xffffffffu, ok);
        if (ok) {
            const uint32_t ob = smem_u32(sm_out);
#pragma unroll
            for (int j = 0; j < R::OUT_UNITS; ++j) {
                sts128(ob + swz_unit((uint32_t)(lane * R::OUT_UNITS + j)),
                       Storage<TOut>::pack(out_mag + j * Storage<TOut>::kPerUnit));
            }
            if (MODE == kLogSigned) store_signs(p.sign_x, gbase, col0, p.n, p.sign_vec_ok != 0, out_sign);
        } else {
            const long long rem = p.n - (long long)chunk * R::CHUNK;
            const int valid = rem < R::CHUNK ? (int)rem : R::CHUNK;
            slow_apply(entering, sm_a, sm_b, sm_out, lane, MODE == kLogSigned ? p.sign_a : nullptr,
                       MODE == kLogSigned ? p.sign_b : nullptr, MODE == kLogSigned ? p.sign_x : nullptr,
                       gbase + (long long)chunk * R::CHUNK, valid);
        }
    }

    // Value of x_0 of a row as the element that starts the second scan (Eq. 7's cat(log x_0, .)).
    __device__ static __forceinline__ E row_start(const Params& p, long long row) {
        const float v = Storage<TIn>::load(p.x0, row);
        if (MODE == kLinear) return state_elem<SIGNED>(log_abs_accurate(v), __float_as_uint(v) & kSignBit);
        uint32_t sg = 0u;
        if (MODE == kLogSigned && p.sign_x0) sg = ((uint32_t)p.sign_x0[row] & 1u) << 31;
        return state_elem<SIGNED>(v, sg);
    }

    // Plain-load staging for rows that TMA cannot address (unaligned base or row pitch).
    __device__ static __forceinline__ void generic_load(const Params& p, uint8_t* sm_a, uint8_t* sm_b, int lane,
                                                        long long row, int chunk) {
        const long long gbase = row * p.n;
        for (int i = lane; i < R::CHUNK; i += 32) {
            const long long col = (long long)chunk * R::CHUNK + i;
            const bool in = col < p.n;
            Storage<TIn>::to_smem(sm_a, (uint32_t)i, in ? Storage<TIn>::load(p.in_a, gbase + col) : neutral_a<MODE>());
            Storage<TIn>::to_smem(sm_b, (uint32_t)i, in ? Storage<TIn>::load(p.in_b, gbase + col) : neutral_b<MODE>());
        }
    }
    __device__ static __forceinline__ void generic_store(const Params& p, const uint8_t* sm_out, int lane, long long row,
                                                         int chunk) {
        const long long gbase = row * p.n;
        for (int i = lane; i < R::CHUNK; i += 32) {
            const long long col = (long long)chunk * R::CHUNK + i;
            if (col < p.n) Storage<TOut>::store(p.out, gbase + col, Storage<TOut>::from_smem(sm_out, (uint32_t)i));
        }
    }
};

__device__ __forceinline__ uint8_t* align_1024(uint8_t* p) {
    return reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(p) + 1023) & ~uintptr_t(1023));
}

// Per-warp shared-memory footprint (bytes): `stages` input stages of two tensors + two output buffers.
template <int MODE, typename TIn, typename TOut, int K>
__host__ __device__ constexpr int warp_smem_bytes(int stages) {
    return stages * 2 * (32 * K * (int)sizeof(TIn)) + 2 * (32 * K * (int)sizeof(TOut));
}

// Per-warp asynchronous chunk pipeline: TMA loads into a ring of input stages, TMA stores from
// two output buffers.  Lane r moves the r-th 128-byte row of a chunk.
template <typename TIn, typename TOut, int K>
struct WarpPipe {
    static constexpr int IN_BYTES = 32 * K * (int)sizeof(TIn);
    static constexpr int OUT_BYTES = 32 * K * (int)sizeof(TOut);
    static constexpr int IN_ROWS = IN_BYTES / 128;
    static constexpr int OUT_ROWS = OUT_BYTES / 128;
    static constexpr int IN_PER_ROW = 128 / (int)sizeof(TIn);
    static constexpr int OUT_PER_ROW = 128 / (int)sizeof(TOut);
    uint8_t* base;   // this warp's shared memory
    uint32_t bars;   // shared address of this warp's mbarriers
    int stages;
    int lane;

    __device__ __forceinline__ uint8_t* in_a(int s) const { return base + s * 2 * IN_BYTES; }
    __device__ __forceinline__ uint8_t* in_b(int s) const { return base + s * 2 * IN_BYTES + IN_BYTES; }
    __device__ __forceinline__ uint8_t* out(int o) const { return base + stages * 2 * IN_BYTES + o * OUT_BYTES; }

    __device__ __forceinline__ void init() {
        if (lane == 0) {
            for (int s = 0; s < stages; ++s) mbar_init(bars + 8 * s, 1);
            fence_mbar_init();
        }
        __syncwarp();
    }
    __device__ __forceinline__ void issue(const CUtensorMap* tm_a, const CUtensorMap* tm_b, long long row, int chunk, int s) {
        const uint32_t bar = bars + 8 * s;
        if (lane == 0) mbar_expect_tx(bar, 2 * IN_BYTES);
        __syncwarp();
        if (lane < IN_ROWS) {
            const int x = chunk * (32 * K) + lane * IN_PER_ROW;
            tma_load_2d(smem_u32(in_a(s)) + lane * 128, tm_a, x, (int)row, bar);
            tma_load_2d(smem_u32(in_b(s)) + lane * 128, tm_b, x, (int)row, bar);
        }
    }
    __device__ __forceinline__ bool wait(int s, uint32_t parity) const {
        return mbar_wait_bounded(bars + 8 * s, parity, kCopySpinLimit);
    }
    // before writing output buffer o: the store issued from it two chunks ago has been read
    __device__ __forceinline__ void acquire_out() const {
        if (lane < OUT_ROWS) bulk_wait_read<1>();
        __syncwarp();
    }
    __device__ __forceinline__ void store(const CUtensorMap* tm_o, long long row, int chunk, int o) const {
        fence_async_smem();
        __syncwarp();
        if (lane < OUT_ROWS) {
            const int x = chunk * (32 * K) + lane * OUT_PER_ROW;
            tma_store_2d(tm_o, x, (int)row, smem_u32(out(o)) + lane * 128);
            bulk_commit();
        }
    }
    __device__ __forceinline__ void drain() const {
        if (lane < OUT_ROWS) bulk_wait_all();
        __syncwarp();
    }
    // Error exit: loads `consumed`..`issued`-1 are still in flight into this warp's stages; give
    // each a bounded wait so that none lands after the CTA has gone.
    __device__ __forceinline__ void drain_loads(long long consumed, long long issued) const {
        for (long long c = consumed; c < issued; ++c) (void)wait((int)(c % stages), (uint32_t)((c / stages) & 1));
    }
};

// ------------------------------------------------------------------------------------------
// (a) Row-batched kernel.  Persistent: warp g of G handles rows g, g+G, g+2G, ...
template <int MODE, typename TIn, typename TOut, int K, bool TMA>
__global__ void __launch_bounds__(512, 1)
batched_scan_kernel(const Params p, const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                    const __grid_constant__ CUtensorMap tm_o) {
    using CE = ChunkEngine<MODE, TIn, TOut, K>;
    using E = typename CE::E;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align_1024(smem_raw);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int S = TMA ? p.stages : 1;
    const int per_warp = warp_smem_bytes<MODE, TIn, TOut, K>(S);

    WarpPipe<TIn, TOut, K> pipe;
    pipe.base = smem + warp * per_warp;
    pipe.bars = smem_u32(smem + nwarps * per_warp) + warp * (8 * kMaxStages);
    pipe.stages = S;
    pipe.lane = lane;
    if (TMA) pipe.init();

    if (blockIdx.x == 0 && threadIdx.x == 0) p.ws->started_id = p.call_id;

    const long long gw = (long long)blockIdx.x * nwarps + warp;
    const long long GW = (long long)gridDim.x * nwarps;
    if (gw >= p.rows) return;
    const long long my_rows = (p.rows - gw + GW - 1) / GW;
    const long long items = my_rows * p.nchunks;

    // producer cursor
    long long prow = gw;
    int pchunk = 0;
    long long issued = 0;
    if (TMA) {
        for (; issued < S - 1 && issued < items; ++issued) {
            pipe.issue(&tm_a, &tm_b, prow, pchunk, (int)(issued % S));
            if (++pchunk == p.nchunks) { pchunk = 0; prow += GW; }
        }
    }

    long long row = gw;
    int chunk = 0;
    E state = CE::row_start(p, row);
    int stage = 0;
    uint32_t parity = 0;
    for (long long q = 0; q < items; ++q) {
        if (TMA) {
            if (issued < items) {
                pipe.issue(&tm_a, &tm_b, prow, pchunk, (int)(issued % S));
                ++issued;
                if (++pchunk == p.nchunks) { pchunk = 0; prow += GW; }
            }
            if (!pipe.wait(stage, parity)) {
                if (lane == 0) record_error(p, kErrCopyTimeout, row);
                pipe.drain_loads(q + 1, issued);
                break;
            }
        } else {
            CE::generic_load(p, pipe.in_a(0), pipe.in_b(0), lane, row, chunk);
            __syncwarp();
        }
        const uint8_t* sm_a = pipe.in_a(stage);
        const uint8_t* sm_b = pipe.in_b(stage);
        uint8_t* sm_out = pipe.out((int)(q & 1));

        typename CE::Pending pd;
        E total;
        CE::phase1(p, sm_a, sm_b, lane, row, chunk, pd, total);
        if (TMA) pipe.acquire_out();
        CE::phase2(p, sm_a, sm_b, sm_out, lane, row, chunk, pd, state);
        state = compose(state, total);
        renormalise(state);

        if (TMA) {
            pipe.store(&tm_o, row, chunk, (int)(q & 1));
        } else {
            __syncwarp();
            CE::generic_store(p, sm_out, lane, row, chunk);
        }
        __syncwarp();  // every lane is done with this input stage

        if (++chunk == p.nchunks) {
            chunk = 0;
            row += GW;
            if (row < p.rows) state = CE::row_start(p, row);
        }
        if (++stage == S) { stage = 0; parity ^= 1u; }
    }
    if (TMA) pipe.drain();
}

// ------------------------------------------------------------------------------------------
// (b) Single-pass kernel with decoupled look-back, for few long rows.
//
// A row is cut into tiles of WARPS chunks.  CTA c handles tiles c, c+G, c+2G, ... (all CTAs are
// resident: cooperative launch), warp w the w-th chunk of each tile.  After the chunks' first
// phase the tile's aggregate is published; the value of x entering the tile is then assembled
// from the descriptors of the preceding tiles of the same row (aggregates until a tile whose
// value of x is already known), which is the "by parts" evaluation that the associativity of
// prefix sums allows, done in one pass.  Descriptor states carry the id of the call, so the
// workspace never has to be cleared.
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

constexpr int kLookPerLane = 4;                     // predecessors polled by each lane per round
constexpr int kLookWindow = 32 * kLookPerLane;      // tiles covered by one round

template <int MODE, typename TIn, typename TOut, int K>
struct Lookback {
    using CE = ChunkEngine<MODE, TIn, TOut, K>;
    static constexpr bool SIGNED = CE::SIGNED;
    using E = Elem<SIGNED>;
    enum : int { kNotReady = 0, kAgg = 1, kInc = 2, kSkip = 3 };

    __device__ static __forceinline__ void publish_agg(const Params& p, long long T, const E& e) {
        p.agg[T] = make_float4(e.A, e.m, e.s, __uint_as_float(e.p));
        st_release_u64(p.flags + T, (p.call_id << 2) | 1ull);
    }
    __device__ static __forceinline__ void publish_inc(const Params& p, long long T, const E& e) {
        p.inc[T] = make_float4(e.m, e.s, 0.0f, 0.0f);
        st_release_u64(p.flags + T, (p.call_id << 2) | 2ull);
    }

    // Warp-collective.  Returns the value of x entering tile T (tile j of `row`), j >= 1.
    __device__ static __forceinline__ E run(const Params& p, long long T, int j, long long row, int lane, bool& failed) {
        E acc = identity_elem<SIGNED>();
        failed = false;
        const unsigned long long id_agg = (p.call_id << 2) | 1ull, id_inc = (p.call_id << 2) | 2ull;
        for (int base = 1;; base += kLookWindow) {
            int st[kLookPerLane];
            bool complete = false, has_inc = false;
            uint32_t inc_mask = 0u;
            unsigned int polls = 0;
            while (true) {
                complete = true;
                has_inc = false;
#pragma unroll
                for (int q = 0; q < kLookPerLane; ++q) {
                    const int dist = base + kLookPerLane * lane + q;
                    const int jj = j - dist;
                    int s;
                    if (jj < -1) s = kSkip;
                    else if (jj == -1) s = kInc;
                    else {
                        const unsigned long long f = ld_acquire_u64(p.flags + (T - dist));
                        s = (f == id_inc) ? kInc : (f == id_agg) ? kAgg : kNotReady;
                    }
                    st[q] = s;
                }
                // ready prefix of this lane, nearest first, up to its first known value
#pragma unroll
                for (int q = 0; q < kLookPerLane; ++q) {
                    if (!has_inc && complete) {
                        if (st[q] == kNotReady) complete = false;
                        else if (st[q] == kInc) has_inc = true;
                    }
                }
                inc_mask = __ballot_sync(0xffffffffu, complete && has_inc);
                const uint32_t ok_mask = __ballot_sync(0xffffffffu, complete);
                const uint32_t need = inc_mask ? ((2u << (__ffs(inc_mask) - 1)) - 1u) : 0xffffffffu;
                if ((ok_mask & need) == need) break;
                if (++polls >= p.spin_limit || ((polls & 255u) == 0u && *(volatile unsigned long long*)&p.ws->error_id == p.call_id)) {
                    failed = true;
                    return acc;
                }
            }
            const int lstar = inc_mask ? (__ffs(inc_mask) - 1) : 31;
            E part = identity_elem<SIGNED>();
            if (lane <= lstar) {
                bool stop = false;
#pragma unroll
                for (int q = 0; q < kLookPerLane; ++q) {
                    if (!stop && st[q] != kSkip) {
                        const int dist = base + kLookPerLane * lane + q;
                        E e;
                        if (st[q] == kInc) {
                            if (j - dist == -1) {
                                e = CE::row_start(p, row);
                            } else {
                                const float4 v = __ldcg(p.inc + (T - dist));
                                e.A = neg_inf(); e.m = v.x; e.s = v.y; e.p = 0u;
                            }
                            stop = true;
                        } else {
                            const float4 v = __ldcg(p.agg + (T - dist));
                            e.A = v.x; e.m = v.y; e.s = v.z; e.p = __float_as_uint(v.w);
                        }
                        part = compose(e, part);  // e is older than everything folded so far
                    } else {
                        stop = true;
                    }
                }
            }
            // ordered reduction: lane 0 holds the newest tiles, higher lanes older ones
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                E other = shfl_down_elem(part, d);
                E c = compose(other, part);
                if (lane + d < 32) part = c;
            }
            const E window = shfl_elem(part, 0);
            acc = compose(window, acc);
            if (inc_mask) return acc;
        }
    }
};

struct alignas(16) Exchange {
    float4 agg[16];    // per-warp aggregates of the current tile
    float4 wexcl[16];  // per-warp exclusive prefixes within the tile
    float4 carry;      // value of x entering the tile (m, s)
    int abort;
    int pad[3];
};

template <bool SIGNED>
__device__ __forceinline__ float4 pack_elem(const Elem<SIGNED>& e) {
    return make_float4(e.A, e.m, e.s, __uint_as_float(e.p));
}
template <bool SIGNED>
__device__ __forceinline__ Elem<SIGNED> unpack_elem(const float4 v) {
    Elem<SIGNED> e;
    e.A = v.x; e.m = v.y; e.s = v.z; e.p = SIGNED ? __float_as_uint(v.w) : 0u;
    return e;
}

template <int MODE, typename TIn, typename TOut, int K, bool TMA>
__global__ void __launch_bounds__(256, 2)
lookback_scan_kernel(const Params p, const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                     const __grid_constant__ CUtensorMap tm_o) {
    using CE = ChunkEngine<MODE, TIn, TOut, K>;
    using LB = Lookback<MODE, TIn, TOut, K>;
    using E = typename CE::E;
    constexpr bool SIGNED = CE::SIGNED;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align_1024(smem_raw);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int S = TMA ? p.stages : 1;
    const int per_warp = warp_smem_bytes<MODE, TIn, TOut, K>(S);

    WarpPipe<TIn, TOut, K> pipe;
    pipe.base = smem + warp * per_warp;
    pipe.bars = smem_u32(smem + nwarps * per_warp) + warp * (8 * kMaxStages);
    pipe.stages = S;
    pipe.lane = lane;
    Exchange* xc = reinterpret_cast<Exchange*>(smem + nwarps * per_warp + nwarps * 8 * kMaxStages);
    if (TMA) pipe.init();
    if (blockIdx.x == 0 && threadIdx.x == 0) p.ws->started_id = p.call_id;
    if (threadIdx.x == 0) xc->abort = 0;
    __syncthreads();

    const long long G = gridDim.x;
    const int tpr = p.tiles_per_row;

    long long issued_tile = blockIdx.x;
    int issued = 0;
    auto issue_next = [&]() {
        if (issued_tile < p.num_tiles) {
            const long long r = issued_tile / tpr;
            const int jj = (int)(issued_tile - r * tpr);
            pipe.issue(&tm_a, &tm_b, r, jj * nwarps + warp, issued % S);
            issued_tile += G;
            ++issued;
        }
    };
    if (TMA) {
        for (int s = 0; s < S - 1; ++s) issue_next();
    }

    int stage = 0;
    uint32_t parity = 0;
    int q = 0;
    for (long long T = blockIdx.x; T < p.num_tiles; T += G, ++q) {
        const long long row = T / tpr;
        const int j = (int)(T - row * tpr);
        const int chunk = j * nwarps + warp;
        bool copy_failed = false;
        if (TMA) {
            issue_next();
            copy_failed = !pipe.wait(stage, parity);
        } else {
            CE::generic_load(p, pipe.in_a(0), pipe.in_b(0), lane, row, chunk);
            __syncwarp();
        }
        const uint8_t* sm_a = pipe.in_a(stage);
        const uint8_t* sm_b = pipe.in_b(stage);
        uint8_t* sm_out = pipe.out(q & 1);

        typename CE::Pending pd;
        E total;
        CE::phase1(p, sm_a, sm_b, lane, row, chunk, pd, total);
        if (lane == 0) xc->agg[warp] = pack_elem<SIGNED>(total);
        if (copy_failed && lane == 0) {
            record_error(p, kErrCopyTimeout, T);
            xc->abort = 1;
        }
        __syncthreads();  // (A) all chunk aggregates of the tile are in shared memory

        if (warp == 0) {
            E mine = (lane < nwarps) ? unpack_elem<SIGNED>(xc->agg[lane]) : identity_elem<SIGNED>();
            E wex, tile_total;
            warp_scan(mine, lane, wex, tile_total);
            if (lane < nwarps) xc->wexcl[lane] = pack_elem<SIGNED>(wex);
            const bool muted = (T == p.mute_tile);
            E carry;
            bool failed = false;
            if (j == 0) {
                carry = CE::row_start(p, row);
            } else {
                if (lane == 0 && !muted) LB::publish_agg(p, T, tile_total);
                carry = LB::run(p, T, j, row, lane, failed);
            }
            E incl = compose(carry, tile_total);
            renormalise(incl);
            if (lane == 0) {
                if (failed) {
                    record_error(p, kErrLookbackTimeout, T);
                    xc->abort = 1;
                } else if (!muted) {
                    LB::publish_inc(p, T, incl);
                }
                xc->carry = make_float4(carry.m, carry.s, 0.0f, 0.0f);
            }
        }
        __syncthreads();  // (B) the value entering the tile is known
        if (xc->abort) {
            if (TMA) pipe.drain_loads(copy_failed ? q + 2 : q + 1, issued);
            break;
        }

        E carry;
        carry.A = neg_inf(); carry.m = xc->carry.x; carry.s = xc->carry.y; carry.p = 0u;
        const E entering_chunk = compose(carry, unpack_elem<SIGNED>(xc->wexcl[warp]));
        if (TMA) pipe.acquire_out();
        CE::phase2(p, sm_a, sm_b, sm_out, lane, row, chunk, pd, entering_chunk);
        if (TMA) {
            pipe.store(&tm_o, row, chunk, q & 1);
        } else {
            __syncwarp();
            CE::generic_store(p, sm_out, lane, row, chunk);
        }
        __syncwarp();
        if (++stage == S) { stage = 0; parity ^= 1u; }
    }
    if (TMA) pipe.drain();
}

}  // namespace hs
