// Kernels of libheinsen_scan (sm_100a only).
//
//   batched_scan_kernel  : a warp walks one row (or 2-16 rows shorter than a chunk) chunk by chunk,
//                          the value of x carried in registers from chunk to chunk (rows >= a few
//                          per SM); rows are handed out to the warps by slot or by ticket.
//   lookback_scan_kernel : rows are cut into tiles of WARPS chunks; one CTA per tile, single
//                          pass, the carry between tiles propagated by one CTA of the grid (the
//                          carry server) through per-tile descriptors in the caller's workspace
//                          (few, long rows).
//
// Both read every input element once and write every output element once.  Chunks travel
// HBM -> shared memory by TMA (per-warp mbarrier pipelines, 128-byte swizzle) and back by TMA
// stores -- or, for rows that TMA cannot address, by asynchronous 4-byte copies and plain stores --;
// the scans themselves run in registers (hs_device.cuh).
#pragma once
#include <cuda.h>

#include <cstddef>

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
    unsigned long long pad;
    // batched kernel, one 16-byte word handled with 128-bit accesses: the next row group to hand out and the
    // id of the call it counts for
    unsigned long long ticket_next;
    unsigned long long ticket_call;
    unsigned long long reserved[26];
};
static_assert(offsetof(Header, ticket_next) % 16 == 0, "the ticket word is accessed as 16 bytes");
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
    int rows_per_warp;  // R: rows held by one warp of the batched kernel (1, 2, 4, 8, 16); look-back: 1
    int flat_boxes;     // R == 1: the tensor maps show a matrix as (element in 128-byte line, whole line of the row,
                        // row), and a chunk moves as ONE box of consecutive lines instead of one box per line;
                        // the last n % line elements of a row, if any, move by plain loads and stores
    unsigned long long call_id;
    Header* ws;
    // look-back kernel only
    int tiles_per_row;
    long long num_tiles;
    uint4* desc;                // [2 * num_tiles] the tiles' aggregates, two words each (look-back kernel)
    uint4* edesc;               // [num_tiles] values entering the tiles
    int lb_server;              // rows of several tiles: the grid's last CTA propagates the carries
    int lb_warps;               // look-back warps per CTA
    unsigned int lb_sleep_idle;   // ns between the carry server's polls of a batch of tile aggregates
    unsigned int lb_sleep_ready;  // ns between a tile's polls of the value entering it
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

// One 16-byte word of global memory, read / written / exchanged as a whole.
struct Desc { unsigned long long lo, hi; };
__device__ __forceinline__ Desc ld_desc(const void* p) {
    Desc d;
    asm volatile("{\n\t.reg .b128 q;\n\tld.relaxed.gpu.global.b128 q, [%2];\n\tmov.b128 {%0, %1}, q;\n\t}"
                 : "=l"(d.lo), "=l"(d.hi) : "l"(p) : "memory");
    return d;
}
__device__ __forceinline__ void st_desc(void* p, Desc d) {
    asm volatile("{\n\t.reg .b128 q;\n\tmov.b128 q, {%1, %2};\n\tst.relaxed.gpu.global.b128 [%0], q;\n\t}"
                 ::"l"(p), "l"(d.lo), "l"(d.hi) : "memory");
}
// Compare-and-swap of a whole 16-byte word; returns what was there.
__device__ __forceinline__ Desc cas_desc(void* p, Desc expected, Desc desired) {
    Desc old;
    asm volatile(
        "{\n\t.reg .b128 c, d, r;\n\t"
        "mov.b128 c, {%3, %4};\n\t"
        "mov.b128 d, {%5, %6};\n\t"
        "atom.relaxed.gpu.global.cas.b128 r, [%2], c, d;\n\t"
        "mov.b128 {%0, %1}, r;\n\t}"
        : "=l"(old.lo), "=l"(old.hi)
        : "l"(p), "l"(expected.lo), "l"(expected.hi), "l"(desired.lo), "l"(desired.hi)
        : "memory");
    return old;
}

// Neutral padding of a ragged row tail: a = 1 (log a = 0), b = 0 (log b = -inf).
template <int MODE>
__device__ __forceinline__ float neutral_a() { return MODE == kLinear ? 1.0f : 0.0f; }
template <int MODE>
__device__ __forceinline__ float neutral_b() { return MODE == kLinear ? 0.0f : neg_inf(); }

// Where a lane sits in its warp's chunk: the warp holds R rows, lane = i*R + g is segment i
// (K consecutive elements) of row g; a row's piece of the chunk is W = (32/R)*K elements wide.
struct LaneMap {
    int R;     // rows per warp: 1, 2, 4, 8 or 16
    int g;     // row within the warp's group
    int i;     // segment within the row's piece
    int W;     // elements per row per chunk
};

// ------------------------------------------------------------------------------------------
// Per-warp chunk engine shared by both kernels: everything between "the chunk's inputs are in
// shared memory" and "the chunk's outputs are in shared memory".
template <int MODE, typename TIn, typename TOut, int K>
struct ChunkEngine {
    using R_ = Run<MODE, TIn, TOut, K>;
    static constexpr bool SIGNED = R_::SIGNED;
    using E = Elem<SIGNED>;
    static constexpr int IN_UNITS = R_::IN_UNITS;
    static constexpr int OUT_UNITS = R_::OUT_UNITS;

    struct Offsets {
        uint32_t in[IN_UNITS + 1];    // the lane's 16-byte input units inside a stage, and the unit after them
        uint32_t out[OUT_UNITS + 1];  // the lane's 16-byte output units inside an output buffer, and the one after
    };
    __device__ static __forceinline__ Offsets offsets(const LaneMap& lm) {
        Offsets o;
#pragma unroll
        for (int j = 0; j <= IN_UNITS; ++j) o.in[j] = chunk_off(lm.R, lm.g, (uint32_t)((lm.i * IN_UNITS + j) * 16));
#pragma unroll
        for (int j = 0; j <= OUT_UNITS; ++j) o.out[j] = chunk_off(lm.R, lm.g, (uint32_t)((lm.i * OUT_UNITS + j) * 16));
        return o;
    }

    // Rows that TMA cannot address, one row per warp ("wide" staging): the 16-byte units of global memory that
    // hold a chunk are copied as they are, so the chunk's first element sits phi bytes into its buffer, phi =
    // address of the row's first element modulo 16 (the same for every chunk of the row: a chunk is a whole
    // number of units wide).  Each tensor has its own phi.  Buffers of these kernels are one 128-byte line longer.
    struct Wide {
        bool on;
        uint32_t phi_a, phi_b, phi_o;
    };
    __device__ static __forceinline__ Wide wide_of(const Params& p, long long row, bool on) {
        Wide w;
        w.on = on;
        const size_t e0 = (size_t)row * (size_t)p.n;
        w.phi_a = on ? (uint32_t)((reinterpret_cast<uintptr_t>(p.in_a) + e0 * sizeof(TIn)) & 15u) : 0u;
        w.phi_b = on ? (uint32_t)((reinterpret_cast<uintptr_t>(p.in_b) + e0 * sizeof(TIn)) & 15u) : 0u;
        w.phi_o = on ? (uint32_t)((reinterpret_cast<uintptr_t>(p.out) + e0 * sizeof(TOut)) & 15u) : 0u;
        return w;
    }
    static constexpr int WIDE_PAD = 128;  // bytes added to every chunk buffer of the kernels without TMA
    // Copy the units that hold columns [colbase, colbase + W) of the row, as far as the row goes (one group of
    // asynchronous copies per call, committed by the caller).  The first and the last unit may reach a few bytes
    // beyond the row: they are units that also hold bytes of the row, so they lie in mapped memory.
    template <typename T>
    __device__ static __forceinline__ void wide_copy_in(const void* tensor, long long total, uint32_t sm, int lane, long long elem0,
                                                        long long left, int W) {
        const uintptr_t g0 = reinterpret_cast<uintptr_t>(tensor) + (size_t)elem0 * sizeof(T);
        const uint32_t phi = (uint32_t)(g0 & 15u);
        const long long valid = left < W ? left : W;
        const int nunits = valid > 0 ? (int)((phi + (uint32_t)valid * (uint32_t)sizeof(T) + 15u) >> 4) : 0;
        const char* src = reinterpret_cast<const char*>(g0 - phi);
        constexpr int ROUNDS = (32 * K * (int)sizeof(T) / 16 + 1 + 31) / 32;
#pragma unroll
        for (int q = 0; q < ROUNDS; ++q) {
            const int u = q * 32 + lane;
            if (u < nunits) {
                HS_DBG_CHECK(reinterpret_cast<uintptr_t>(src) + 16u * (unsigned)u + 16u > reinterpret_cast<uintptr_t>(tensor) &&
                                 reinterpret_cast<uintptr_t>(src) + 16u * (unsigned)u <
                                     reinterpret_cast<uintptr_t>(tensor) + (size_t)total * sizeof(T),
                             kDbgUnits, elem0, continue);
                cp_async16(sm + chunk_off(1, 0, (uint32_t)(u * 16)), src + 16 * u);
            }
        }
    }
    __device__ static __forceinline__ void wide_load_async(const Params& p, uint32_t sm_a, uint32_t sm_b, int lane, long long row,
                                                           long long colbase, int W) {
        const long long left = row < p.rows ? p.n - colbase : 0;
        wide_copy_in<TIn>(p.in_a, p.rows * p.n, sm_a, lane, row * p.n + colbase, left, W);
        wide_copy_in<TIn>(p.in_b, p.rows * p.n, sm_b, lane, row * p.n + colbase, left, W);
        cp_async_commit();
    }
    // The chunk's outputs, written by the lanes phi_o bytes into the buffer, go out as whole 16-byte units
    // where they fill one, element by element at the two ends.
    __device__ static __forceinline__ void wide_store(const Params& p, uint32_t sm_out, int lane, long long row, long long colbase,
                                                      int W) {
        const long long left = row < p.rows ? p.n - colbase : 0;
        const long long valid = left < W ? left : W;
        if (valid <= 0) return;
        const uintptr_t g0 = reinterpret_cast<uintptr_t>(p.out) + (size_t)(row * p.n + colbase) * sizeof(TOut);
        const uint32_t phi = (uint32_t)(g0 & 15u);
        const uint32_t nbytes = (uint32_t)valid * (uint32_t)sizeof(TOut);
        const uint32_t head = phi ? ((16u - phi) < nbytes ? (16u - phi) : nbytes) : 0u;  // bytes of the first, partial unit
        const uint32_t body = (nbytes - head) >> 4;                                     // whole units
        const uint32_t tail = nbytes - head - (body << 4);                              // bytes of the last, partial unit
        char* const dst = reinterpret_cast<char*>(g0 - phi);
        const uint32_t u0 = phi ? 1u : 0u;
        for (uint32_t u = (uint32_t)lane; u < body; u += 32u) {
            HS_DBG_CHECK(dst + 16u * (u0 + u) >= reinterpret_cast<char*>(p.out) &&
                             dst + 16u * (u0 + u) + 16u <= reinterpret_cast<char*>(p.out) + (size_t)(p.rows * p.n) * sizeof(TOut),
                         kDbgUnits, row * p.n + colbase, continue);
            *reinterpret_cast<uint4*>(dst + 16u * (u0 + u)) = lds128(sm_out + chunk_off(1, 0, 16u * (u0 + u)));
        }
        const uint32_t head_n = head / (uint32_t)sizeof(TOut), tail_n = tail / (uint32_t)sizeof(TOut);
        if ((uint32_t)lane < head_n) {
            const uint32_t b = phi + (uint32_t)lane * (uint32_t)sizeof(TOut);
            Storage<TOut>::copy_out(dst + b, 0, sm_out + chunk_off(1, 0, b));
        }
        if ((uint32_t)lane < tail_n) {
            const uint32_t b = phi + nbytes - tail + (uint32_t)lane * (uint32_t)sizeof(TOut);
            Storage<TOut>::copy_out(dst + b, 0, sm_out + chunk_off(1, 0, b));
        }
    }
    // The lane's inputs from a stage, whichever way the chunk got there (sa, sb: filled only by storage types that
    // carry the sign in the element).
    template <bool PLAIN>
    __device__ static __forceinline__ void read_inputs(uint32_t sm_a, uint32_t sm_b, const Offsets& off, const Wide& wd,
                                                       float* va, float* vb, uint32_t* sa, uint32_t* sb) {
        if (PLAIN && wd.on) {
            Shifted<TIn, K>::read_signed(sm_a, off.in, wd.phi_a, va, sa);
            Shifted<TIn, K>::read_signed(sm_b, off.in, wd.phi_b, vb, sb);
        } else {
            R_::load_signed(sm_a, sm_b, off.in, va, vb, sa, sb);
        }
    }
    template <bool PLAIN>
    __device__ static __forceinline__ void write_outputs(uint32_t sm_out, const Offsets& off, const Wide& wd, const float* v,
                                                         const uint32_t* sg) {
        if (PLAIN && wd.on) {
            Shifted<TOut, K>::write_signed(sm_out, off.out, wd.phi_o, v, sg);
        } else {
            constexpr int PER = Storage<TOut>::kPerUnit;
#pragma unroll
            for (int j = 0; j < OUT_UNITS; ++j)
                sts128(sm_out + off.out[j], Storage<TOut>::pack_signed(v + j * PER, sg + (Storage<TOut>::kCarriesSign ? j * PER : 0)));
        }
    }
    // whether the sign tensors of the call exist (signed mode with a storage type that does not carry the sign)
    static constexpr bool SIGN_TENSORS = (MODE == kLogSigned) && !Storage<TIn>::kCarriesSign;

    // The outputs of a run whose fast form holds, into the output buffer (and the signs to global memory): unit
    // by unit, so that no more than one unit's worth of outputs is live at a time.
    template <bool PLAIN, int J = 0, bool G = false>
    __device__ static __forceinline__ void emit_units(const R_& run, const typename R_::Applied& ap, uint32_t sm_out,
                                                      const Offsets& off) {
        if constexpr (J < OUT_UNITS) {
            constexpr int PER = Storage<TOut>::kPerUnit;
            float o[PER];
            uint32_t sg[MODE == kLogSigned ? PER : 1];
            run.template outputs<J * PER, PER, G>(ap, o, sg);
            sts128(sm_out + off.out[J], Storage<TOut>::pack_signed(o, sg));
            emit_units<PLAIN, J + 1, G>(run, ap, sm_out, off);
        }
    }
    // (G: the run holds g_t instead of A_t, see Run::outputs)
    template <bool PLAIN, bool G = false>
    __device__ static __forceinline__ void emit_outputs(const Params& p, const R_& run, const typename R_::Applied& ap,
                                                        uint32_t sm_out, const Offsets& off, const Wide& wd, long long idx0,
                                                        long long left) {
        if (SIGN_TENSORS || (PLAIN && wd.on)) {
            float out_mag[K];
            uint32_t out_sign[MODE == kLogSigned ? K : 1];
            run.template outputs<0, K, G>(ap, out_mag, out_sign);
            write_outputs<PLAIN>(sm_out, off, wd, out_mag, out_sign);
            if (SIGN_TENSORS) store_signs(p.sign_x, idx0, left, p.sign_vec_ok != 0, out_sign);
        } else {
            emit_units<PLAIN, 0, G>(run, ap, sm_out, off);
        }
    }

    // sign masks of the lane's K elements from a uint8 tensor (0/1 per element); idx0 = index of
    // the lane's first element, `left` = elements of the row from there on (may be <= 0).
    __device__ static __forceinline__ void load_signs(const uint8_t* g, long long idx0, long long left, bool vec,
                                                      uint32_t* mask) {
        if (g == nullptr) {
#pragma unroll
            for (int t = 0; t < K; ++t) mask[t] = 0u;
            return;
        }
        if (vec && left >= K) {
            HS_DBG_CHECK(idx0 >= 0 && (idx0 & 15) == 0, kDbgElement, idx0, return);
#pragma unroll
            for (int j = 0; j < K / 16; ++j) {
                const uint4 v = __ldg(reinterpret_cast<const uint4*>(g + idx0 + 16 * j));
                const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int t = 0; t < 16; ++t) mask[16 * j + t] = (w[t >> 2] << (31 - 8 * (t & 3))) & kSignBit;
            }
        } else {
#pragma unroll
            for (int t = 0; t < K; ++t) mask[t] = (t < left) ? (((uint32_t)g[idx0 + t] & 1u) << 31) : 0u;
        }
    }
    __device__ static __forceinline__ void store_signs(uint8_t* g, long long idx0, long long left, bool vec,
                                                       const uint32_t* mask) {
        if (vec && left >= K) {
            HS_DBG_CHECK(idx0 >= 0 && (idx0 & 15) == 0, kDbgElement, idx0, return);
#pragma unroll
            for (int j = 0; j < K / 16; ++j) {
                uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
                for (int t = 0; t < 16; ++t) w[t >> 2] |= (mask[16 * j + t] >> 31) << (8 * (t & 3));
                *reinterpret_cast<uint4*>(g + idx0 + 16 * j) = make_uint4(w[0], w[1], w[2], w[3]);
            }
        } else {
#pragma unroll
            for (int t = 0; t < K; ++t)
                if (t < left) g[idx0 + t] = (uint8_t)(mask[t] >> 31);
        }
    }

    // Tracked form, pass 1: the lane's run as one part, every step with its own reference.
    // idx0/left as above (`left` <= 0: the run lies wholly beyond the row).
    // (phi_a, phi_b: where the chunks start in their buffers -- 0 unless staged wide)
    __device__ static __noinline__ E slow_pass1(uint32_t sm_a, uint32_t sm_b, LaneMap lm, const uint8_t* gsa,
                                                const uint8_t* gsb, long long idx0, long long left, uint32_t phi_a,
                                                uint32_t phi_b) {
        E e = identity_elem<SIGNED>();
        for (int t = 0; t < K; ++t) {
            if (t < left) {
                const uint32_t byte = (uint32_t)((lm.i * K + t) * sizeof(TIn));
                const uint32_t at_a = sm_a + chunk_off(lm.R, lm.g, phi_a + byte), at_b = sm_b + chunk_off(lm.R, lm.g, phi_b + byte);
                const uint32_t sa = gsa ? (((uint32_t)gsa[idx0 + t] & 1u) << 31) : Storage<TIn>::sign_from_smem(at_a);
                const uint32_t sb = gsb ? (((uint32_t)gsb[idx0 + t] & 1u) << 31) : Storage<TIn>::sign_from_smem(at_b);
                e = compose(e, Leaf<MODE, TIn>::get(Storage<TIn>::from_smem(at_a), Storage<TIn>::from_smem(at_b), sa, sb));
            }
        }
        return e;
    }
    struct SlowOut {
        float vals[K];
        uint32_t sgn[MODE == kLogSigned ? K : 1];
    };
    // Tracked form, pass 2: step the value through the lane's run; returns outputs (and signs).
    __device__ static __noinline__ SlowOut slow_apply(E st, uint32_t sm_a, uint32_t sm_b, LaneMap lm,
                                                      const uint8_t* gsa, const uint8_t* gsb, long long idx0,
                                                      long long left, uint32_t phi_a, uint32_t phi_b) {
        SlowOut so;
        for (int t = 0; t < K; ++t) {
            float v = 0.0f;
            uint32_t sg = 0u;
            if (t < left) {
                const uint32_t byte = (uint32_t)((lm.i * K + t) * sizeof(TIn));
                const uint32_t at_a = sm_a + chunk_off(lm.R, lm.g, phi_a + byte), at_b = sm_b + chunk_off(lm.R, lm.g, phi_b + byte);
                const uint32_t sa = gsa ? (((uint32_t)gsa[idx0 + t] & 1u) << 31) : Storage<TIn>::sign_from_smem(at_a);
                const uint32_t sb = gsb ? (((uint32_t)gsb[idx0 + t] & 1u) << 31) : Storage<TIn>::sign_from_smem(at_b);
                st = compose(st, Leaf<MODE, TIn>::get(Storage<TIn>::from_smem(at_a), Storage<TIn>::from_smem(at_b), sa, sb));
                renormalise(st);
                if (MODE == kLinear) {
                    const float h = ex2(st.m * (0.5f * kLog2e));
                    v = (st.s == 0.0f) ? 0.0f : (st.s * h) * h;
                } else {
                    v = (st.s == 0.0f) ? neg_inf() : fmaf(lg2(fabsf(st.s)), kLn2, st.m);
                    sg = (st.s < 0.0f) ? kSignBit : 0u;
                }
            }
            so.vals[t] = v;
            if (MODE == kLogSigned) so.sgn[t] = sg;
        }
        return so;
    }

    struct Pending {  // what phase 2 needs from phase 1
        R_ run;
        E excl;       // parts of this row's chunk before the lane's run
        bool slow;
    };

    // Phase 1: inputs from shared memory, the lane's run, the scan over the lanes of the row.
    // `row` is the lane's row (may be >= rows for a padded group), col0 its first column.
    // `ragged` (warp-uniform): the chunk reaches beyond the row end or the warp's group beyond the
    // last row, so some lanes must pad their run with neutral elements.
    template <bool PLAIN>
    __device__ static __forceinline__ void phase1(const Params& p, uint32_t sm_a, uint32_t sm_b,
                                                  const Offsets& off, const LaneMap& lm, int lane, long long row,
                                                  long long col0, bool ragged, const Wide& wd, Pending& pd, E& total) {
        float va[K], vb[K];
        uint32_t sa[MODE == kLogSigned ? K : 1], sb[MODE == kLogSigned ? K : 1];
        read_inputs<PLAIN>(sm_a, sm_b, off, wd, va, vb, sa, sb);
        const long long left = (row < p.rows) ? p.n - col0 : 0;
        if (ragged) {
#pragma unroll
            for (int t = 0; t < K; ++t) {
                if (t >= left) {
                    va[t] = neutral_a<MODE>();
                    vb[t] = neutral_b<MODE>();
                    if (MODE == kLogSigned) { sa[t] = 0u; sb[t] = 0u; }
                }
            }
        }
        if (SIGN_TENSORS) {
            load_signs(p.sign_a, row * p.n + col0, left, p.sign_vec_ok != 0, sa);
            load_signs(p.sign_b, row * p.n + col0, left, p.sign_vec_ok != 0, sb);
        }
        E agg = pd.run.pass1(va, vb, sa, sb);
        pd.slow = __any_sync(0xffffffffu, pd.run.bad);
        if (pd.slow) {
            agg = slow_pass1(sm_a, sm_b, lm, SIGN_TENSORS ? p.sign_a : nullptr,
                             SIGN_TENSORS ? p.sign_b : nullptr, row * p.n + col0, left, PLAIN ? wd.phi_a : 0u,
                             PLAIN ? wd.phi_b : 0u);
        }
        row_scan(agg, lane, lm.R, pd.excl, total);
    }

    // Phase 2: `entering_row` is the value of x entering this row's piece of the chunk.
    template <bool PLAIN>
    __device__ static __forceinline__ void phase2(const Params& p, uint32_t sm_a, uint32_t sm_b,
                                                  uint32_t sm_out, const Offsets& off, const LaneMap& lm, long long row,
                                                  long long col0, const Wide& wd, const Pending& pd, const E& entering_row) {
        const E entering = compose(entering_row, pd.excl);
        const long long left = (row < p.rows) ? p.n - col0 : 0;
        const uint32_t ob = sm_out;
        const typename R_::Applied ap = pd.run.prepare(entering);
        const bool ok = __all_sync(0xffffffffu, !pd.slow && ap.ok);
        if (ok) {
            emit_outputs<PLAIN>(p, pd.run, ap, ob, off, wd, row * p.n + col0, left);
        } else {
            const SlowOut so = slow_apply(entering, sm_a, sm_b, lm, SIGN_TENSORS ? p.sign_a : nullptr,
                                          SIGN_TENSORS ? p.sign_b : nullptr, row * p.n + col0, left,
                                          PLAIN ? wd.phi_a : 0u, PLAIN ? wd.phi_b : 0u);
            write_outputs<PLAIN>(ob, off, wd, so.vals, so.sgn);
            if (SIGN_TENSORS) store_signs(p.sign_x, row * p.n + col0, left, p.sign_vec_ok != 0, so.sgn);
        }
    }

    // x_0 of a row as stored (value, sign mask); rows beyond the last one are empty (x_0 = 0).
    struct RawX0 { float v; uint32_t sg; };
    __device__ static __forceinline__ RawX0 load_x0(const Params& p, long long row) {
        RawX0 r;
        r.v = MODE == kLinear ? 0.0f : neg_inf();
        r.sg = 0u;
        if (row < p.rows) {
            r.v = Storage<TIn>::load(p.x0, row);
            if (SIGN_TENSORS && p.sign_x0) r.sg = ((uint32_t)p.sign_x0[row] & 1u) << 31;
            if (Storage<TIn>::kCarriesSign) r.sg = Storage<TIn>::load_sign(p.x0, row);
        }
        return r;
    }
    // ... and as the element that starts the second scan (Eq. 7's cat(log x_0, .)).
    __device__ static __forceinline__ E x0_elem(const RawX0& r) {
        if (MODE == kLinear) return state_elem<SIGNED>(log_abs_accurate(r.v), __float_as_uint(r.v) & kSignBit);
        return state_elem<SIGNED>(r.v, r.sg);
    }
    __device__ static __forceinline__ E row_start(const Params& p, long long row) { return x0_elem(load_x0(p, row)); }

    // Plain-load staging for rows that TMA cannot address (unaligned base or row pitch).
    // row0: first row of the warp's group, colbase: first column of the chunk.  Row by row of the group,
    // 32 consecutive columns per step (one coalesced access), so that the row's base address and bounds
    // are formed once per row and no division is left in the loop.
    __device__ static __forceinline__ void generic_load(const Params& p, uint32_t sm_a, uint32_t sm_b, const LaneMap& lm,
                                                        int lane, long long row0, long long colbase) {
#pragma unroll 1
        for (int rg = 0; rg < lm.R; ++rg) {
            const long long row = row0 + rg;
            const long long base = row * p.n + colbase;
            const long long left = row < p.rows ? p.n - colbase : 0;  // columns of the row from colbase on
#pragma unroll 4
            for (int c = lane; c < lm.W; c += 32) {
                const bool in = c < left;
                const uint32_t off = chunk_off(lm.R, rg, (uint32_t)(c * sizeof(TIn)));
                HS_DBG_CHECK(!in || (base + c >= 0 && base + c < p.rows * p.n), kDbgElement, base + c, continue);
                if (in) {
                    Storage<TIn>::copy_in(sm_a + off, p.in_a, base + c);
                    Storage<TIn>::copy_in(sm_b + off, p.in_b, base + c);
                } else {
                    Storage<TIn>::to_smem(sm_a + off, neutral_a<MODE>());
                    Storage<TIn>::to_smem(sm_b + off, neutral_b<MODE>());
                }
            }
        }
    }
    // The same as one group of asynchronous 4-byte copies, so that it can run a chunk ahead of the arithmetic
    // like the TMA loads do (4-byte element types only).
    static constexpr bool ASYNC_PLAIN = sizeof(TIn) == 4;
    __device__ static __forceinline__ void generic_load_async(const Params& p, uint32_t sm_a, uint32_t sm_b,
                                                              const LaneMap& lm, int lane, long long row0, long long colbase) {
#pragma unroll 1
        for (int rg = 0; rg < lm.R; ++rg) {
            const long long row = row0 + rg;
            const TIn* const pa = static_cast<const TIn*>(p.in_a) + (row * p.n + colbase);
            const TIn* const pb = static_cast<const TIn*>(p.in_b) + (row * p.n + colbase);
            const long long left = row < p.rows ? p.n - colbase : 0;
#pragma unroll 4
            for (int c = lane; c < lm.W; c += 32) {
                const uint32_t off = chunk_off(lm.R, rg, (uint32_t)(c * sizeof(TIn)));
                if (c < left) {
                    HS_DBG_CHECK(row >= 0 && row < p.rows && colbase + c < p.n, kDbgElement, row * p.n + colbase + c, continue);
                    cp_async4(sm_a + off, pa + c);
                    cp_async4(sm_b + off, pb + c);
                } else {
                    Storage<TIn>::to_smem(sm_a + off, neutral_a<MODE>());
                    Storage<TIn>::to_smem(sm_b + off, neutral_b<MODE>());
                }
            }
        }
        cp_async_commit();
    }
    __device__ static __forceinline__ void generic_store(const Params& p, uint32_t sm_out, const LaneMap& lm, int lane,
                                                         long long row0, long long colbase) {
#pragma unroll 1
        for (int rg = 0; rg < lm.R; ++rg) {
            const long long row = row0 + rg;
            const long long base = row * p.n + colbase;
            const long long left = row < p.rows ? p.n - colbase : 0;
#pragma unroll 4
            for (int c = lane; c < lm.W; c += 32) {
                if (c < left) {
                    const uint32_t off = chunk_off(lm.R, rg, (uint32_t)(c * sizeof(TOut)));
                    HS_DBG_CHECK(base + c >= 0 && base + c < p.rows * p.n, kDbgElement, base + c, continue);
                    Storage<TOut>::copy_out(p.out, base + c, sm_out + off);
                }
            }
        }
    }

    // Flat boxes move whole 128-byte lines of a row; the last n % line elements of the row travel by
    // plain loads and stores, into and out of the places they have in the chunk that holds them
    // (one row per warp; colbase: first column of that chunk).
    static constexpr int IN_LINE = 128 / (int)sizeof(TIn), OUT_LINE = 128 / (int)sizeof(TOut);
    // (out of line: rare, and the chunk loop should stay small)
    __device__ static __noinline__ void tail_load_impl(const void* in_a, const void* in_b, long long n, long long rows,
                                                       uint32_t sm_a, uint32_t sm_b, int lane, long long row, int colbase) {
        for (int col = (int)(n / IN_LINE) * IN_LINE + lane; col < n; col += 32) {
            const uint32_t off = chunk_off(1, 0, (uint32_t)((col - colbase) * sizeof(TIn)));
            HS_DBG_CHECK(row >= 0 && row < rows && col >= colbase, kDbgElement, row * n + col, continue);
            Storage<TIn>::copy_in(sm_a + off, in_a, row * n + col);
            Storage<TIn>::copy_in(sm_b + off, in_b, row * n + col);
        }
    }
    __device__ static __noinline__ void tail_store_impl(void* out, long long n, long long rows, uint32_t sm_out, int lane,
                                                        long long row, int colbase) {
        for (int col = (int)(n / OUT_LINE) * OUT_LINE + lane; col < n; col += 32) {
            const uint32_t off = chunk_off(1, 0, (uint32_t)((col - colbase) * sizeof(TOut)));
            HS_DBG_CHECK(row >= 0 && row < rows && col >= colbase, kDbgElement, row * n + col, continue);
            Storage<TOut>::copy_out(out, row * n + col, sm_out + off);
        }
    }
    __device__ static __forceinline__ void tail_load(const Params& p, uint32_t sm_a, uint32_t sm_b, int lane, long long row,
                                                     int colbase) {
        tail_load_impl(p.in_a, p.in_b, p.n, p.rows, sm_a, sm_b, lane, row, colbase);
    }
    __device__ static __forceinline__ void tail_store(const Params& p, uint32_t sm_out, int lane, long long row, int colbase) {
        tail_store_impl(p.out, p.n, p.rows, sm_out, lane, row, colbase);
    }
};

}  // namespace hs
#include "hs_pairs.cuh"
namespace hs {

__device__ __forceinline__ uint8_t* align_1024(uint8_t* p) {
    return reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(p) + 1023) & ~uintptr_t(1023));
}

// Per-warp shared-memory footprint (bytes): `stages` input stages of two tensors + two output buffers.
// (pad: bytes added to every chunk buffer -- 0 with TMA, one 128-byte line without, see ChunkEngine::Wide)
template <int MODE, typename TIn, typename TOut, int K>
__host__ __device__ constexpr int warp_smem_bytes(int stages, int pad) {
    return stages * 2 * (32 * K * (int)sizeof(TIn) + pad) + 2 * (32 * K * (int)sizeof(TOut) + pad);
}

// Per-warp asynchronous chunk pipeline: TMA loads into a ring of input stages, TMA stores from
// two output buffers.  A chunk is moved as boxes of {128 bytes, R rows}; lane b moves box b.
template <typename TIn, typename TOut, int K, int PAD>
struct WarpPipe {
    static constexpr int IN_BYTES = 32 * K * (int)sizeof(TIn);
    static constexpr int OUT_BYTES = 32 * K * (int)sizeof(TOut);
    static constexpr int IN_BUF = IN_BYTES + PAD;    // one tensor's chunk buffer
    static constexpr int OUT_BUF = OUT_BYTES + PAD;
    static constexpr int IN_PER_BOX = 128 / (int)sizeof(TIn);    // elements of a row in one box
    static constexpr int OUT_PER_BOX = 128 / (int)sizeof(TOut);
    uint32_t base;   // this warp's shared memory (32-bit shared address)
    uint32_t bars;   // shared address of this warp's mbarriers
    int stages;
    int lane;
    int R;           // rows per box
    int in_boxes;    // boxes per tensor per chunk, input / output
    int out_boxes;
    bool flat;       // one box per chunk (see Params::flat_boxes)

    __device__ __forceinline__ void setup(int rows_per_warp, bool flat_boxes = false) {
        R = rows_per_warp;
        flat = flat_boxes;
        in_boxes = flat ? 1 : IN_BYTES / (128 * R);
        out_boxes = flat ? 1 : OUT_BYTES / (128 * R);  // lanes that issue stores
    }
    __device__ __forceinline__ uint32_t in_a(int s) const { return base + s * 2 * IN_BUF; }
    __device__ __forceinline__ uint32_t in_b(int s) const { return base + s * 2 * IN_BUF + IN_BUF; }
    __device__ __forceinline__ uint32_t out(int o) const { return base + stages * 2 * IN_BUF + o * OUT_BUF; }

    __device__ __forceinline__ void init() {
        if (lane == 0) {
            for (int s = 0; s < stages; ++s) mbar_init(bars + 8 * s, 1);
            fence_mbar_init();
        }
        __syncwarp();
    }
    // colbase: first column of the chunk, row0: first row of the group.  Flat boxes: the tensor maps
    // show a matrix as (element in line, whole line of the row, row); a chunk is the box of IN_LINES
    // lines from line colbase / IN_PER_BOX of row row0, clipped by the hardware at the row's last whole line.
    __device__ __forceinline__ void issue(const CUtensorMap* tm_a, const CUtensorMap* tm_b, int row0, int colbase, int s) {
        const uint32_t bar = bars + 8 * s;
        if (lane == 0) mbar_expect_tx(bar, 2 * IN_BYTES);
        __syncwarp();
        if (flat) {
            if (lane == 0) {
                tma_load_3d(in_a(s), tm_a, 0, colbase / IN_PER_BOX, row0, bar);
                tma_load_3d(in_b(s), tm_b, 0, colbase / IN_PER_BOX, row0, bar);
            }
        } else if (lane < in_boxes) {
            const int x = (colbase + lane * IN_PER_BOX) * Storage<TIn>::kTmaScale;
            const uint32_t dst = (uint32_t)(lane * R * 128);
            tma_load_2d(in_a(s) + dst, tm_a, x, row0, bar);
            tma_load_2d(in_b(s) + dst, tm_b, x, row0, bar);
        }
    }
    __device__ __forceinline__ bool wait(int s, uint32_t parity) const {
        return mbar_wait_bounded(bars + 8 * s, parity, kCopySpinLimit);
    }
    // before writing output buffer o: the store issued from it two chunks ago has been read
    __device__ __forceinline__ void acquire_out() const {
        if (lane < out_boxes) bulk_wait_read<1>();
        __syncwarp();
    }
    // store the chunk held in shared memory at `src` (flat boxes: its whole lines; see issue())
    __device__ __forceinline__ void store_from(const CUtensorMap* tm_o, int row0, int colbase, uint32_t src) const {
        fence_async_smem();
        __syncwarp();
        if (flat) {
            if (lane == 0) {
                tma_store_3d(tm_o, 0, colbase / OUT_PER_BOX, row0, src);
                bulk_commit();
            }
        } else if (lane < out_boxes) {
            const int x = (colbase + lane * OUT_PER_BOX) * Storage<TOut>::kTmaScale;
            tma_store_2d(tm_o, x, row0, src + (uint32_t)(lane * R * 128));
            bulk_commit();
        }
    }
    __device__ __forceinline__ void drain() const {
        if (lane < out_boxes) bulk_wait_all();
        __syncwarp();
    }
    // Error exit: loads `consumed`..`issued`-1 are still in flight into this warp's stages; give
    // each a bounded wait so that none lands after the CTA has gone.
    __device__ __forceinline__ void drain_loads(long long consumed, long long issued) const {
        for (long long c = consumed; c < issued; ++c) (void)wait((int)(c % stages), (uint32_t)((c / stages) & 1));
    }
    static constexpr int IN_LINES = IN_BYTES / 128;    // 128-byte lines of one tensor's chunk
    static constexpr int OUT_LINES = OUT_BYTES / 128;
};

// ------------------------------------------------------------------------------------------
// (a) Row-batched kernel.  Persistent: every warp walks row groups one after the other -- the first
// by its slot, the following ones drawn from a ticket counter --; a group is R consecutive rows
// (p.rows_per_warp), each walked chunk by chunk by 32/R lanes with the value of x carried in
// registers.
template <int MODE, typename TIn, typename TOut, int K, bool TMA, bool TICKETS>
__global__ void __launch_bounds__(512, 1)
batched_scan_kernel(const Params p, const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                    const __grid_constant__ CUtensorMap tm_o) {
    using CE = ChunkEngine<MODE, TIn, TOut, K>;
    using E = typename CE::E;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align_1024(smem_raw);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    // loads run ahead of the arithmetic: TMA boxes, or groups of asynchronous 4-byte copies
    const int R = p.rows_per_warp;
    constexpr bool PLAIN = !TMA;
    constexpr int PAD = PLAIN ? CE::WIDE_PAD : 0;
    const bool wide = PLAIN && R == 1;  // one row per warp that TMA cannot address: staged as whole 16-byte units
    const bool AHEAD = TMA || CE::ASYNC_PLAIN || wide;
    const int S = AHEAD ? p.stages : 1;
    const int per_warp = warp_smem_bytes<MODE, TIn, TOut, K>(S, PAD);

    LaneMap lm;
    lm.R = R;
    lm.g = lane & (R - 1);
    lm.i = lane / R;
    lm.W = (32 / R) * K;
    const typename CE::Offsets off = CE::offsets(lm);

    using Pipe = WarpPipe<TIn, TOut, K, PAD>;
    Pipe pipe;
    pipe.base = smem_u32(smem) + warp * per_warp;
    pipe.bars = smem_u32(smem + nwarps * per_warp) + warp * (8 * kMaxStages);
    pipe.stages = S;
    pipe.lane = lane;
    pipe.setup(R, p.flat_boxes != 0);
    if (TMA) pipe.init();
    // Programmatic dependent launch: the next kernel of the stream may be set up while this one runs
    // (it waits below before it touches memory), and this kernel touches global memory only after
    // everything before it in the stream has completed.  Both are no-ops for an ordinary launch.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // With many row groups per warp slot (TICKETS; the host decides) the groups are handed out by tickets: every warp
    // starts with the group of its slot and draws the next one from a counter in the workspace, so that
    // an SM that streams faster than another (their shares of the memory system differ by several
    // percent) simply takes more rows.  With few groups per slot greedy hand-out would pile the last
    // round on the SMs that are ahead, and the groups stay with their slots: slot, slot + GW, ...
    // The counter shares a 16-byte word with the id of the call it counts for: the first CTA to find another
    // call's id there replaces the whole word by {first ticket = number of warp slots, this call} in one
    // 128-bit compare-and-swap (a CTA that loses the race finds the word already right); the workspace needs
    // no initialisation and no host-side reset.
    unsigned long long* const ticket_word = &p.ws->ticket_next;
    const int GW = gridDim.x * nwarps;
    if (threadIdx.x == 0) {
        if (blockIdx.x == 0) p.ws->started_id = p.call_id;
        if (TICKETS) {
            const Desc seen = ld_desc(ticket_word);
            if (seen.hi != p.call_id) {
                Desc fresh;
                fresh.lo = (unsigned long long)GW;
                fresh.hi = p.call_id;
                (void)cas_desc(ticket_word, seen, fresh);
            }
        }
    }
    if (TICKETS) __syncthreads();  // from here on the word belongs to this call

    // All hot-loop indices are 32-bit and advance incrementally (rows < 2^31; with TMA also n < 2^31);
    // 64-bit products appear once per row only.
    // Warp slots are numbered CTA-fastest, so that few row groups spread over all SMs.
    const int gw = warp * (int)gridDim.x + (int)blockIdx.x;
    const int groups = (int)((p.rows + R - 1) / R);
    if (gw >= groups) return;
    const int nchunks = p.nchunks;
    const bool tail_ragged = (p.n % lm.W) != 0;  // the last chunk of a row is partial
    // flat boxes: the chunk of a row that holds its last n % line elements, if there are any (-1: none)
    const int tail_chunk_in = (pipe.flat && p.n % CE::IN_LINE) ? (int)(p.n / CE::IN_LINE) * CE::IN_LINE / lm.W : -1;
    const int tail_chunk_out = sizeof(TIn) == sizeof(TOut) ? tail_chunk_in  // same lines: one variable
                               : (pipe.flat && p.n % CE::OUT_LINE) ? (int)(p.n / CE::OUT_LINE) * CE::OUT_LINE / lm.W : -1;
    // A ticket is drawn a few chunks before the end of the current group -- late, so that the groups go
    // to the warps that get there first, but early enough for the atomic's latency to stay off the path --
    // and stays in lane 0 until the warp needs it.  Without tickets a warp walks slot, slot + GW, ...
    constexpr bool by_ticket = TICKETS;  // two instantiations: the hand-over code of one does not burden the other
    auto draw = [&]() -> unsigned int {
        unsigned int t = 0u;
        if (lane == 0) t = (unsigned int)atomicAdd(ticket_word, 1ull);
        return t;
    };
    auto take = [&](unsigned int t) -> int {
        const unsigned int v = __shfl_sync(0xffffffffu, t, 0);
        return v >= (unsigned int)groups ? groups : (int)v;
    };
    unsigned int drawn = 0u;
    const int draw_at = nchunks > 3 ? nchunks - 3 : 0;  // index of the chunk with which the next ticket is drawn
    // without tickets the warp's share is known: groups gw, gw + GW, ... and so many chunks
    const long long items = TICKETS ? 0 : (long long)((groups - gw + GW - 1) / GW) * nchunks;

    // x_0 of the lane's row in the next group, in flight while the current group is worked on.  With
    // tickets: the group the loads have entered and the arithmetic has not (the loads run one chunk ahead:
    // p.stages == 2; -1: none), x_0 fetched when the group is entered.  Without: the group after this one.
    int qa_group = -1;
    typename CE::RawX0 qa_x0 = CE::load_x0(p, TICKETS ? p.rows : ((long long)gw + GW) * R + lm.g);
    auto enter_group = [&](int g) {
        qa_x0 = CE::load_x0(p, (long long)g * R + lm.g);
        qa_group = g;
    };

    // producer cursor (the loads run S-1 chunks ahead)
    int pgroup = gw, pchunk = 0, pstage = 0;
    bool loading = true;  // the producer still has a row group
    long long issued = 0, consumed = 0;
    auto issue_chunk = [&]() {
        HS_DBG_CHECK(!TMA || ((long long)pgroup * R < p.rows && (long long)pchunk * lm.W < p.n &&
                              ((pchunk * lm.W * (int)sizeof(TIn)) & 15) == 0 && pstage < S),
                     kDbgTmaCoord, ((unsigned long long)pgroup << 32) | (unsigned)pchunk, return);
        if (TMA) pipe.issue(&tm_a, &tm_b, pgroup * R, pchunk * lm.W, pstage);
        else if (wide) CE::wide_load_async(p, pipe.in_a(pstage), pipe.in_b(pstage), lane, pgroup, (long long)pchunk * lm.W, lm.W);
        else CE::generic_load_async(p, pipe.in_a(pstage), pipe.in_b(pstage), lm, lane, (long long)pgroup * R, pchunk * lm.W);
    };
    auto issue_next = [&]() {
        if (TICKETS) {
            if (pchunk == 0 && issued != 0) {  // the previous group is complete: enter the next one
                pgroup = take(drawn);
                if (pgroup >= groups) {
                    loading = false;
                    return;
                }
                enter_group(pgroup);
            }
            issue_chunk();
            if (pchunk == draw_at) drawn = draw();
            ++issued;
            if (++pstage == S) pstage = 0;
            if (++pchunk == nchunks) pchunk = 0;
        } else {
            issue_chunk();
            ++issued;
            if (++pstage == S) pstage = 0;
            if (++pchunk == nchunks) {
                pchunk = 0;
                pgroup += GW;
            }
            loading = issued < items;
        }
    };
    if (AHEAD) {
        for (int s = 0; s < S - 1 && loading; ++s) issue_next();
    }

    int group = gw, chunk = 0, colbase = 0;
    long long row = (long long)group * R + lm.g;
    bool group_ragged = (group + 1) * (long long)R > p.rows;
    E state = CE::row_start(p, row);
    typename CE::Wide wd = CE::wide_of(p, row, wide);
    int stage = 0;
    uint32_t parity = 0;
    while (TICKETS ? group < groups : consumed < items) {
        if (TMA) {
            if (loading) issue_next();
            if (!pipe.wait(stage, parity)) {
                if (lane == 0) record_error(p, kErrCopyTimeout, row);
                pipe.drain_loads(consumed + 1, issued);
                break;
            }
        } else if (AHEAD) {
            if (loading) issue_next();
            // this chunk's group of copies is the oldest one pending; at most one newer group is in flight
            if (issued - consumed > 1) cp_async_wait<1>();
            else cp_async_wait<0>();
            __syncwarp();
        } else {
            CE::generic_load(p, pipe.in_a(0), pipe.in_b(0), lm, lane, (long long)group * R, colbase);
            __syncwarp();
        }
        const uint32_t sm_a = pipe.in_a(stage);
        const uint32_t sm_b = pipe.in_b(stage);
        const uint32_t sm_out = pipe.out((int)(consumed & 1));
        if (TMA && chunk == tail_chunk_in) {  // the box brought the row's whole lines; fetch the rest
            CE::tail_load(p, sm_a, sm_b, lane, row, colbase);
            __syncwarp();
        }
        const int col0 = colbase + lm.i * K;
        const bool ragged = group_ragged || (tail_ragged && chunk == nchunks - 1);

        typename CE::Pending pd;
        E total;
        CE::template phase1<PLAIN>(p, sm_a, sm_b, off, lm, lane, row, col0, ragged, wd, pd, total);
        if (TMA) pipe.acquire_out();
        CE::template phase2<PLAIN>(p, sm_a, sm_b, sm_out, off, lm, row, col0, wd, pd, state);
        state = compose(state, total);
        renormalise(state);

        HS_DBG_CHECK(!TMA || ((long long)group * R < p.rows && colbase < p.n && ((colbase * (int)sizeof(TOut)) & 15) == 0),
                     kDbgTmaCoord, ((unsigned long long)group << 32) | (unsigned)colbase, break);
        if (TMA) {
            pipe.store_from(&tm_o, group * R, colbase, sm_out);
            if (chunk == tail_chunk_out) CE::tail_store(p, sm_out, lane, row, colbase);
        } else {
            __syncwarp();
            if (wide) CE::wide_store(p, sm_out, lane, row, colbase, lm.W);
            else CE::generic_store(p, sm_out, lm, lane, (long long)group * R, colbase);
        }
        __syncwarp();  // every lane is done with this input stage
        ++consumed;
        if (!AHEAD && by_ticket && chunk == draw_at) drawn = draw();

        colbase += lm.W;
        if (++chunk == nchunks) {
            chunk = 0;
            colbase = 0;
            if (by_ticket) {
                if (!AHEAD) {  // no loads ahead: the arithmetic enters the next group itself
                    const int g = take(drawn);
                    if (g < groups) enter_group(g);
                }
                if (qa_group < 0) break;  // no group left for this warp
                group = qa_group;
                state = CE::x0_elem(qa_x0);
                qa_group = -1;
            } else {
                group += GW;  // beyond the last group only when the loop is about to end
                state = CE::x0_elem(qa_x0);
                qa_x0 = CE::load_x0(p, ((long long)group + GW) * R + lm.g);
            }
            row = (long long)group * R + lm.g;
            group_ragged = (group + 1) * (long long)R > p.rows;
            wd = CE::wide_of(p, row, wide);
        }
        if (++stage == S) { stage = 0; parity ^= 1u; }
    }
    if (TMA) pipe.drain();
}

// ------------------------------------------------------------------------------------------
// (a') Row-batched kernel with the rows cut to measure: for a number of rows between one and a few per warp slot,
// whole rows per slot leave the last round of slots partly idle (4096 rows on 2368 slots: 1.73 rounds, which costs
// nothing while the kernel is bound by HBM and 13 % once it is bound by the SM clock under the board's power cap).
// Here the rows' chunks form one sequence, (row 0, chunk 0), (row 0, chunk 1), ..., and every slot takes an equal
// share of it.  With at least one row per slot a share is
//     [the rest of a row that the slot before began] [whole rows] [the beginning of a row that the next slot ends],
// and the slot walks it in the order beginning - whole rows - rest: the beginning of a row needs nothing but x_0,
// and the value of x after it goes to the next slot through a 16-byte word in the workspace, {m, s, call id},
// long before that slot, which walks its own beginning and whole rows first, asks for it (bounded wait).
// One row per warp, any staging (TMA boxes or whole 16-byte units); the arithmetic is the batched kernel's.
template <int MODE, typename TIn, typename TOut, int K, bool TMA>
__global__ void __launch_bounds__(512, 1)
batched_span_kernel(const Params p, const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                    const __grid_constant__ CUtensorMap tm_o) {
    using CE = ChunkEngine<MODE, TIn, TOut, K>;
    using E = typename CE::E;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align_1024(smem_raw);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    constexpr bool PLAIN = !TMA;
    constexpr int PAD = PLAIN ? CE::WIDE_PAD : 0;
    constexpr int S = 2;  // input stages per warp: one chunk being worked on, one in flight
    const int per_warp = warp_smem_bytes<MODE, TIn, TOut, K>(S, PAD);

    LaneMap lm;
    lm.R = 1; lm.g = 0; lm.i = lane; lm.W = 32 * K;
    const typename CE::Offsets off = CE::offsets(lm);
    using Pipe = WarpPipe<TIn, TOut, K, PAD>;
    Pipe pipe;
    pipe.base = smem_u32(smem) + warp * per_warp;
    pipe.bars = smem_u32(smem + nwarps * per_warp) + warp * (8 * kMaxStages);
    pipe.stages = S;
    pipe.lane = lane;
    pipe.setup(1, p.flat_boxes != 0);
    if (TMA) pipe.init();
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (threadIdx.x == 0 && blockIdx.x == 0) p.ws->started_id = p.call_id;

    // the slot's share of the chunk sequence (slots numbered CTA-fastest, as in the batched kernel)
    const int GW = gridDim.x * nwarps;
    const int gw = warp * (int)gridDim.x + (int)blockIdx.x;
    const int nchunks = p.nchunks;
    const long long total = p.rows * (long long)nchunks;
    const long long q0 = total / GW, rem = total % GW;
    const long long lo = gw * q0 + (gw < rem ? gw : rem), hi = lo + q0 + (gw < rem ? 1 : 0);
    const int len = (int)(hi - lo);  // (the host sends shapes with at least one row per slot: q0 >= nchunks)
    if (len <= 0) return;
    const int row_lo = (int)(lo / nchunks), c_lo = (int)(lo % nchunks);
    const int row_hi = (int)(hi / nchunks), c_hi = (int)(hi % nchunks);
    const int n_head = c_hi;                         // chunks [0, c_hi) of row_hi, walked first
    const int n_rest = c_lo ? nchunks - c_lo : 0;    // chunks [c_lo, nchunks) of row_lo, walked last
    const int first_whole = row_lo + (c_lo ? 1 : 0);
    // position q of the walk -> (row, chunk)
    struct Cursor {
        int q, row, chunk;
    };
    auto start = [&]() {
        Cursor c;
        c.q = 0;
        if (n_head) { c.row = row_hi; c.chunk = 0; }
        else if (len > n_rest) { c.row = first_whole; c.chunk = 0; }
        else { c.row = row_lo; c.chunk = c_lo; }
        return c;
    };
    auto advance = [&](Cursor& c) {
        ++c.q;
        ++c.chunk;
        if (c.q == n_head) {                       // the beginning is done: on to the whole rows, or to the rest
            if (len - n_rest > n_head) { c.row = first_whole; c.chunk = 0; }
            else { c.row = row_lo; c.chunk = c_lo; }
        } else if (c.q == len - n_rest) {          // the whole rows are done: the rest of the first row
            c.row = row_lo; c.chunk = c_lo;
        } else if (c.chunk == nchunks) {
            c.chunk = 0; ++c.row;
        }
    };
    const bool tail_ragged = (p.n % lm.W) != 0;
    const int tail_chunk_in = (pipe.flat && p.n % CE::IN_LINE) ? (int)(p.n / CE::IN_LINE) * CE::IN_LINE / lm.W : -1;
    const int tail_chunk_out = sizeof(TIn) == sizeof(TOut) ? tail_chunk_in
                               : (pipe.flat && p.n % CE::OUT_LINE) ? (int)(p.n / CE::OUT_LINE) * CE::OUT_LINE / lm.W : -1;

    // Loads run one chunk ahead of the arithmetic (two stages): the chunk after the one being worked on is issued
    // at the top of every step, from the same cursor.
    auto issue = [&](const Cursor& c, int stg) {
        HS_DBG_CHECK(c.row >= 0 && c.row < p.rows && c.chunk >= 0 && c.chunk < nchunks && stg < S, kDbgTmaCoord,
                     ((unsigned long long)c.row << 32) | (unsigned)c.chunk, return);
        if (TMA) pipe.issue(&tm_a, &tm_b, c.row, c.chunk * lm.W, stg);
        else CE::wide_load_async(p, pipe.in_a(stg), pipe.in_b(stg), lane, c.row, (long long)c.chunk * lm.W, lm.W);
    };

    uint4* const handoff = p.desc;  // [GW]: the value of x after a slot's beginning of a row
    // x_0 of the next row that starts in the walk, in flight while the current row is worked on
    auto row_start_after = [&](int r) {
        if (n_head && r == row_hi) return (len - n_rest > n_head) ? first_whole : -1;
        return (r + 1 < row_hi) ? r + 1 : -1;
    };
    int x0_row = n_head ? row_hi : (len > n_rest ? first_whole : -1);
    typename CE::RawX0 x0_next = CE::load_x0(p, x0_row >= 0 ? (long long)x0_row : p.rows);
    Cursor cur = start();
    issue(cur, 0);
    Desc early;  // the previous slot's hand-over word, read ahead of its use
    early.lo = 0ull; early.hi = 0ull;
    if (n_rest && len - n_rest <= 1) early = ld_desc(handoff + (gw - 1));
    typename CE::Wide wd = CE::wide_of(p, cur.row, PLAIN);
    E state = identity_elem<CE::SIGNED>();
    bool fresh = true;          // the next chunk starts a segment (a row from x_0, or the rest of a row)
    int stage = 0;
    uint32_t parity = 0;
    for (int consumed = 0; consumed < len; ++consumed) {
        const int row = cur.row, chunk = cur.chunk, colbase = chunk * lm.W;
        Cursor nxt = cur;
        advance(nxt);
        const bool more = consumed + 1 < len;
        if (more) issue(nxt, stage ^ 1);
        if (TMA) {
            if (!pipe.wait(stage, parity)) {
                if (lane == 0) record_error(p, kErrCopyTimeout, row);
                if (more) (void)pipe.wait(stage ^ 1, stage ? parity ^ 1u : parity);
                break;
            }
        } else {
            if (more) cp_async_wait<1>();
            else cp_async_wait<0>();
            __syncwarp();
        }
        if (fresh) {
            wd = CE::wide_of(p, row, PLAIN);
            if (chunk == 0) {
                state = CE::x0_elem(x0_next);   // (x0_row == row here)
                x0_row = row_start_after(row);
                x0_next = CE::load_x0(p, x0_row >= 0 ? (long long)x0_row : p.rows);
            } else {
                // the rest of a row: its beginning is the previous slot's, walked first there (the word was asked
                // for a chunk ago, so that its way through L2 is not waited for here)
                Desc d = early;
                bool got = d.hi == p.call_id;
                for (unsigned int polls = 0; !got && polls < p.spin_limit; ++polls) {
                    __nanosleep(200);
                    d = ld_desc(handoff + (gw - 1));
                    got = d.hi == p.call_id;
                }
                if (!got) {
                    if (lane == 0) record_error(p, kErrLookbackTimeout, row);
                    if (TMA && more) (void)pipe.wait(stage ^ 1, stage ? parity ^ 1u : parity);
                    break;
                }
                state.A = neg_inf();
                state.m = __uint_as_float((uint32_t)d.lo);
                state.s = __uint_as_float((uint32_t)(d.lo >> 32));
                state.p = 0u;
            }
        }
        const uint32_t sm_a = pipe.in_a(stage), sm_b = pipe.in_b(stage), sm_out = pipe.out(stage);
        if (TMA && chunk == tail_chunk_in) {
            CE::tail_load(p, sm_a, sm_b, lane, row, colbase);
            __syncwarp();
        }
        const int col0 = colbase + lane * K;
        const bool ragged = tail_ragged && chunk == nchunks - 1;
        typename CE::Pending pd;
        E total_e;
        CE::template phase1<PLAIN>(p, sm_a, sm_b, off, lm, lane, row, col0, ragged, wd, pd, total_e);
        if (TMA) pipe.acquire_out();
        CE::template phase2<PLAIN>(p, sm_a, sm_b, sm_out, off, lm, row, col0, wd, pd, state);
        state = compose(state, total_e);
        renormalise(state);
        if (TMA) {
            pipe.store_from(&tm_o, row, colbase, sm_out);
            if (chunk == tail_chunk_out) CE::tail_store(p, sm_out, lane, row, colbase);
        } else {
            __syncwarp();
            CE::wide_store(p, sm_out, lane, row, colbase, lm.W);
        }
        __syncwarp();
        fresh = nxt.chunk == 0;           // the next chunk starts a row ...
        if (consumed + 1 == n_head) {
            // the beginning of the last row of the share is done: hand the value of x to the slot that has the rest
            if (lane == 0) {
                Desc d;
                d.lo = (unsigned long long)__float_as_uint(state.m) | ((unsigned long long)__float_as_uint(state.s) << 32);
                d.hi = p.call_id;
                st_desc(handoff + gw, d);
            }
            fresh = true;
        }
        if (consumed + 1 == len - n_rest) fresh = true;   // ... or the rest of the share's first row
        if (n_rest && consumed + 2 == len - n_rest) early = ld_desc(handoff + (gw - 1));
        cur = nxt;
        stage ^= 1;
        if (stage == 0) parity ^= 1u;
    }
    if (TMA) pipe.drain();
}

// ------------------------------------------------------------------------------------------
// (b) Single-pass kernel for few long rows, the carry between tiles decoupled from the tiles' arithmetic.
//
// A row is cut into tiles of W chunks (W = compute warps per CTA).  CTA c handles tiles c, c+G,
// c+2G, ... (all CTAs are resident: cooperative launch); compute warp w owns the w-th chunk of
// each tile, and two more warps do nothing but carry propagation.  The kernel is software
// pipelined so that the latency of the carry never stalls the arithmetic:
//
//   compute warp, iteration i :  phase 1 of tile i   (inputs -> partial sums s_t parked in shared
//                                                     memory, chunk aggregate handed to the
//                                                     publisher warp)
//                                phase 2 of tile i-D (whose entering value has arrived meanwhile:
//                                                     outputs, TMA store), D = stages - 2
//   publisher warp, tile i    :  scan of the W chunk aggregates, publish the tile's aggregate
//   carry server (last CTA)   :  prefix over the tiles' aggregates in tile order, 32 tiles per
//                                warp at a time: the value of x entering each tile
//   look-back warp, tile i    :  wait for that value, hand it to the compute warps.
//
// This is the "by parts" evaluation that the associativity of prefix sums allows, done in one
// pass over HBM.  Every wait is bounded; when one runs out the CTA records an error and leaves.
// Descriptors are 16-byte words, each read and written with a single 128-bit access and tagged
// with the call's id (see Lookback below).
// Bounded wait that also gives up when `*abort` becomes non-zero: the flag is looked at between the polls,
// each of which the hardware suspends for a bounded time of its own.
__device__ __forceinline__ bool mbar_wait_abortable(uint32_t bar, uint32_t parity, uint32_t limit, const int* abort) {
#pragma unroll 1
    for (uint32_t i = 0; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*(const volatile int*)abort) return false;
    }
    return false;
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

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

constexpr int kLbMaxWarps = 16;                     // compute warps per CTA, at most
constexpr int kSrvRing = 32;                        // hand-over slots between the batches of the carry server

// The carry between tiles goes through two arrays of 16-byte words in the workspace:
//   desc[2T], desc[2T+1] = aggregate of tile T, written by the tile's CTA right after its phase 1;
//   edesc[T]             = value of x entering tile T, written by the carry server.
// Each word is read and written with one 128-bit access and carries the call's 62-bit id in its upper half: a
// word counts only if the id is this call's, so the workspace needs no clearing between calls (nor before the
// first one), and payload and tag cannot be torn apart.
// The carry server is the last CTA of the grid; it computes no tile.  Its warps take batches of 32 consecutive
// tiles in turn (lane l <-> tile 32q + l): wait for the 32 aggregates, scan them, take the value entering the
// batch from the batch before (through the server's shared memory: the only sequential step, a compose and a
// flag per 32 tiles), write the 32 entering values.  A tile's CTA then waits for ONE word that only it reads.
// Against a look-back in which every tile reads its predecessors' descriptors and composes them itself:
// each descriptor is read once instead of by every tile of its round (no lines of L2 that all SMs poll at
// once), a tile's warp has nothing to reduce (the look-back warp's reductions, ~4400 cycles per tile, paced
// the whole kernel), and nothing a tile waits for depends on what a tile of the same round publishes after
// a look-back of its own.
template <int MODE, typename TIn, typename TOut, int K>
struct Lookback {
    using CE = ChunkEngine<MODE, TIn, TOut, K>;
    static constexpr bool SIGNED = CE::SIGNED;
    using E = Elem<SIGNED>;
    // A tile's aggregate as two words {A, m, id} and {s, parity, id}, the value entering a tile as one word
    // {m, s, id}: a word belongs to this call exactly if its upper half is the call's id.
    __device__ static __forceinline__ void publish_agg(const Params& p, long long T, const E& e) {
        HS_DBG_CHECK(T >= 0 && T < p.num_tiles, kDbgTile, T, return);
        Desc d1, d2;
        d1.lo = (unsigned long long)__float_as_uint(e.A) | ((unsigned long long)__float_as_uint(e.m) << 32);
        d2.lo = (unsigned long long)__float_as_uint(e.s) | ((unsigned long long)(e.p >> 31) << 32);
        d1.hi = d2.hi = p.call_id;
        st_desc(p.desc + 2 * T, d1);
        st_desc(p.desc + 2 * T + 1, d2);
    }
    __device__ static __forceinline__ E unpack_agg(const Desc& d1, const Desc& d2) {
        E e;
        e.A = __uint_as_float((uint32_t)d1.lo);
        e.m = __uint_as_float((uint32_t)(d1.lo >> 32));
        e.s = __uint_as_float((uint32_t)d2.lo);
        e.p = SIGNED ? ((uint32_t)(d2.lo >> 32) & 1u) << 31 : 0u;
        return e;
    }
    __device__ static __forceinline__ Desc pack_value(const Params& p, const E& e) {
        Desc d;
        d.lo = (unsigned long long)__float_as_uint(e.m) | ((unsigned long long)__float_as_uint(e.s) << 32);
        d.hi = p.call_id;
        return d;
    }
    __device__ static __forceinline__ E unpack_value(const Desc& d) {
        E e;
        e.A = neg_inf();
        e.m = __uint_as_float((uint32_t)d.lo);
        e.s = __uint_as_float((uint32_t)(d.lo >> 32));
        e.p = 0u;
        return e;
    }

    __device__ static __forceinline__ bool give_up(const Params& p, unsigned int& polls) {
        return ++polls >= p.spin_limit ||
               ((polls & 255u) == 0u && *(volatile unsigned long long*)&p.ws->error_id == p.call_id);
    }

    // Warp-collective, in a tile's CTA: waits for the value of x entering tile T (every lane reads the same word).
    __device__ static __forceinline__ E await_entering(const Params& p, long long T, const volatile int* abort_flag,
                                                       bool& failed, unsigned int& total_polls) {
        failed = false;
        unsigned int polls = 0;
        HS_DBG_CHECK(T >= 0 && T < p.num_tiles, kDbgTile, T, failed = true);
        Desc d;
        d.lo = 0ull; d.hi = 0ull;
        while (!failed) {
            d = ld_desc(p.edesc + T);
            ++total_polls;
            d.lo = __shfl_sync(0xffffffffu, d.lo, 0);
            d.hi = __shfl_sync(0xffffffffu, d.hi, 0);
            if (d.hi == p.call_id) break;
            if (__any_sync(0xffffffffu, *abort_flag || give_up(p, polls))) { failed = true; break; }
            __nanosleep(p.lb_sleep_ready);
        }
        return unpack_value(d);
    }

    // The carry server (all warps of the grid's last CTA).  `ring` is kSrvRing hand-over slots in its shared memory.
    struct ServerRing {
        float2 value[kSrvRing];             // (m, s) of x after batch q, in slot q % kSrvRing
        unsigned long long done[kSrvRing];  // q + 1 once it is there
        int abort;
    };
    __device__ static __forceinline__ void serve(const Params& p, ServerRing* ring, int lane, int warp, int nwarps) {
        if (threadIdx.x < kSrvRing) ring->done[threadIdx.x] = 0ull;
        if (threadIdx.x == 0) ring->abort = 0;
        __syncthreads();
        const long long nb = (p.num_tiles + 31) / 32;
        for (long long q = warp; q < nb; q += nwarps) {
            const long long T = q * 32 + lane;
            const bool active = T < p.num_tiles;
            long long row = 0;
            int j = 0;
            if (active) {
                row = T / p.tiles_per_row;
                j = (int)(T - row * p.tiles_per_row);
            }
            HS_DBG_CHECK(!active || (row >= 0 && row < p.rows), kDbgTile, T, (void)0);
            const bool starts_row = active && j == 0;
            E x0e = identity_elem<SIGNED>();
            if (starts_row) x0e = CE::row_start(p, row);
            // the batch's aggregates
            Desc d1, d2;
            d1.lo = 0ull; d1.hi = 0ull;
            d2 = d1;
            unsigned int polls = 0;
            bool ok = true;
            while (true) {
                if (active && !(d1.hi == p.call_id && d2.hi == p.call_id)) {
                    d1 = ld_desc(p.desc + 2 * T);
                    d2 = ld_desc(p.desc + 2 * T + 1);
                }
                if (__all_sync(0xffffffffu, !active || (d1.hi == p.call_id && d2.hi == p.call_id))) break;
                if (__any_sync(0xffffffffu, *(volatile int*)&ring->abort || give_up(p, polls))) { ok = false; break; }
                __nanosleep(p.lb_sleep_idle);
            }
            E part = identity_elem<SIGNED>();
            if (ok) {
                if (active) part = unpack_agg(d1, d2);
                if (starts_row) part = compose(x0e, part);  // a value (A = -inf): forgets what came before the row
            }
            E wex, total;
            warp_scan(part, lane, wex, total);
            // the value entering the batch: from the batch before
            E cin = identity_elem<SIGNED>();
            if (ok && q > 0) {
                const int slot = (int)((q - 1) % kSrvRing);
                polls = 0;
                while (!__all_sync(0xffffffffu, *(volatile unsigned long long*)&ring->done[slot] == (unsigned long long)q)) {
                    if (__any_sync(0xffffffffu, *(volatile int*)&ring->abort || give_up(p, polls))) { ok = false; break; }
                }
                if (ok) {
                    __threadfence_block();
                    cin.A = neg_inf();
                    cin.m = *(volatile float*)&ring->value[slot].x;
                    cin.s = *(volatile float*)&ring->value[slot].y;
                    cin.p = 0u;
                }
            }
            if (!ok) {
                if (lane == 0 && !*(volatile int*)&ring->abort) {
                    record_error(p, kErrLookbackTimeout, q * 32);
                    ring->abort = 1;
                }
                break;
            }
            E after = compose(cin, total);
            renormalise(after);
            if (lane == 0) {
                const int slot = (int)(q % kSrvRing);
                *(volatile float*)&ring->value[slot].x = after.m;
                *(volatile float*)&ring->value[slot].y = after.s;
                __threadfence_block();
                *(volatile unsigned long long*)&ring->done[slot] = (unsigned long long)(q + 1);
            }
            if (active) {
                E ent = starts_row ? x0e : compose(cin, wex);
                renormalise(ent);
                st_desc(p.edesc + T, pack_value(p, ent));
            }
        }
    }
};

// CTA-level exchange between the compute warps and the look-back warps (a ring of tiles in flight).
constexpr int kLbRing = 4;      // ring slots: tiles between "aggregate delivered" and "carry consumed"
constexpr int kLbMaxStages = 5; // input stages per compute warp, at most
struct alignas(16) Exchange {
    float4 agg[kLbRing][kLbMaxWarps];    // per-warp aggregates of a tile; the publisher warp replaces them in
                                         // place by the per-warp exclusive prefixes within the tile
    float4 carry[kLbRing];               // value of x entering the tile (m, s)
    unsigned long long total_ready[kLbRing];  // mbarrier: the publisher warp has written wexcl and published the tile
    unsigned long long agg_ready[kLbRing];    // mbarrier: all compute warps have delivered their aggregate
    unsigned long long carry_ready[kLbRing];  // mbarrier: a look-back warp has delivered the carry
    int abort;
    int pad[3];
};

// Per-lane state carried from phase 1 to phase 2 of a chunk.  It stays in registers: the compute
// warps keep the records of the last four tiles and shift them by one every iteration.
template <bool SIGNED>
struct LanePark {
    float r;              // reference of the lane's run
    Elem<SIGNED> excl;    // parts of the chunk before the lane's run
    bool slow;            // the chunk took the tracked form in phase 1 (warp-uniform)
};

// One input stage of a compute warp: [a-tensor chunk][b-tensor chunk][park].  The partial sums
// s_t (fp32) of phase 1 are parked over the b-tensor chunk when the input type is 4 bytes wide
// (in place), else in a region of their own; the outputs of phase 2 are written over the parked
// sums and stored from there.
// (PAD: bytes added to every chunk buffer -- 0 with TMA, one 128-byte line without, see ChunkEngine::Wide)
template <typename TIn, int K, int PAD>
struct LbStage {
    static constexpr int IN_BYTES = 32 * K * (int)sizeof(TIn);
    static constexpr int IN_BUF = IN_BYTES + PAD;
    static constexpr bool IN_PLACE = sizeof(TIn) >= 4;  // the parked fp32 sums fit over the b-tensor chunk
    static constexpr int PARK_OFF = IN_PLACE ? IN_BUF : 2 * IN_BUF;
    static constexpr int BYTES = IN_PLACE ? 2 * IN_BUF : 2 * IN_BUF + 32 * K * 4 + PAD;
    static_assert(PAD != 0 || (BYTES % 1024 == 0 && PARK_OFF % 1024 == 0), "swizzled TMA buffers need 1024-byte alignment");
    static_assert(BYTES % 128 == 0 && PARK_OFF % 128 == 0, "chunk buffers are made of 128-byte lines");
};
// total dynamic shared memory of the look-back kernel for W compute warps and S stages (without alignment slack)
template <typename TIn, int K, int PAD>
__host__ __device__ constexpr int lb_total_smem_bytes(int W, int S) {
    return W * S * LbStage<TIn, K, PAD>::BYTES + (int)sizeof(Exchange) + W * kLbMaxStages * 8;
}

// Position of a CTA's tile sequence: tile T = tile j of row `row`; advances by a fixed stride
// without divisions (the stride is split once into whole rows and a remainder).
struct TileCursor {
    long long T;
    int row, j;
    __device__ __forceinline__ void init(long long t, int tiles_per_row) {
        T = t;
        row = (int)(t / tiles_per_row);
        j = (int)(t - (long long)row * tiles_per_row);
    }
    __device__ __forceinline__ void advance(int stride, int stride_rows, int stride_rem, int tiles_per_row) {
        T += stride;
        row += stride_rows;
        j += stride_rem;
        if (j >= tiles_per_row) { j -= tiles_per_row; ++row; }
    }
};

template <int MODE, typename TIn, typename TOut, int K, bool TMA>
__global__ void __launch_bounds__(512, 1)
lookback_scan_kernel(const Params p, const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                     const __grid_constant__ CUtensorMap tm_o) {
    using CE = ChunkEngine<MODE, TIn, TOut, K>;
    using LB = Lookback<MODE, TIn, TOut, K>;
    using R_ = Run<MODE, TIn, TOut, K>;
    constexpr bool PLAIN = !TMA;
    using ST = LbStage<TIn, K, PLAIN ? CE::WIDE_PAD : 0>;
    using E = typename CE::E;
    constexpr bool SIGNED = CE::SIGNED;
    constexpr int CHUNK = 32 * K;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align_1024(smem_raw);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int NLB = p.lb_warps;                 // look-back warps; after them comes one publisher warp
    const int W = (blockDim.x >> 5) - NLB - 1;  // compute warps
    const int S = p.stages;                     // input stages per compute warp
    const int D = S - 2;                        // phase 2 of a tile runs D iterations after its phase 1

    uint8_t* tail = smem + (size_t)W * S * ST::BYTES;
    Exchange* xc = reinterpret_cast<Exchange*>(tail);
    const uint32_t warp_bars = smem_u32(reinterpret_cast<uint8_t*>(xc) + sizeof(Exchange));  // [W][kLbMaxStages]
    const uint32_t agg_bar = smem_u32(&xc->agg_ready[0]), carry_bar = smem_u32(&xc->carry_ready[0]);
    const uint32_t total_bar = smem_u32(&xc->total_ready[0]);

    // (every compute warp initialises its own mbarriers, thread 0 those of the exchange: one thread initialising
    // all of them takes more than a microsecond, which a short launch feels)
    if (lane == 0) {
        if (warp < W) {
            for (int i = 0; i < kLbMaxStages; ++i) mbar_init(warp_bars + 8 * (warp * kLbMaxStages + i), 1);
        }
        if (warp == 0) {
            xc->abort = 0;
            for (int b = 0; b < kLbRing; ++b) {
                mbar_init(agg_bar + 8 * b, W);
                mbar_init(total_bar + 8 * b, 1);
                mbar_init(carry_bar + 8 * b, 1);
            }
        }
        fence_mbar_init();
    }
    // Programmatic dependent launch, as in the batched kernel: when the host launches the single-tile form with
    // programmatic stream serialisation, everything above overlaps the end of the previous kernel of the stream
    // and global memory is touched only from here on; for the cooperative launch both are no-ops.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (threadIdx.x == 0 && blockIdx.x == 0) p.ws->started_id = p.call_id;
    __syncthreads();

    // rows of several tiles: the grid's last CTA is the carry server, the others take the tiles
    const bool served = p.lb_server != 0;
    if (served && blockIdx.x == gridDim.x - 1) {
        LB::serve(p, reinterpret_cast<typename LB::ServerRing*>(smem), lane, warp, (int)(blockDim.x >> 5));
        return;
    }
    const long long G = gridDim.x - (served ? 1 : 0);
    const int tpr = p.tiles_per_row;
    const long long first = blockIdx.x;
    const long long my_tiles = first < p.num_tiles ? (p.num_tiles - first + G - 1) / G : 0;

    if (warp == W + NLB) {
        // ------------------------------------------------------------------ publisher warp
        // Blocks on each tile's chunk aggregates in turn, folds them (per-warp exclusive prefixes
        // for phase 2, the tile's aggregate for everyone else) and publishes the tile's descriptor
        // at once: the tiles after this one are waiting for it.
        TileCursor cur;
        cur.init(first, tpr);
        const int g_rows_p = (int)G / tpr, g_rem_p = (int)G % tpr;
        for (long long i = 0; i < my_tiles; ++i, cur.advance((int)G, g_rows_p, g_rem_p, tpr)) {
            const int b = (int)(i % kLbRing);
            // (the wait watches the CTA's abort flag: once the compute warps have given up, nobody arrives
            // on this barrier any more, and the publisher must leave at once rather than poll to the limit)
            const bool arrived = mbar_wait_abortable(agg_bar + 8 * b, (uint32_t)((i / kLbRing) & 1), kCopySpinLimit, &xc->abort);
            if (!arrived || *(volatile int*)&xc->abort) {
                if (lane == 0 && !*(volatile int*)&xc->abort) { record_error(p, kErrCopyTimeout, cur.T); xc->abort = 1; }
                __syncwarp();
                if (lane == 0) mbar_arrive(total_bar + 8 * b);
                break;
            }
            E mine = (lane < W) ? unpack_elem<SIGNED>(xc->agg[b][lane]) : identity_elem<SIGNED>();
            E wex, tile_total;
            warp_scan(mine, lane, wex, tile_total);
            if (lane < W) xc->agg[b][lane] = pack_elem<SIGNED>(wex);  // every lane has read its aggregate by now
            if (lane == 0 && cur.T != p.mute_tile) LB::publish_agg(p, cur.T, tile_total);
            __syncwarp();
            if (lane == 0) mbar_arrive(total_bar + 8 * b);
        }
        return;
    }
    if (warp >= W) {
        // ------------------------------------------------------------------ look-back warps
        TileCursor cur;
        cur.init(first + (long long)(warp - W) * G, tpr);
        const int lb_stride = NLB * (int)G;
        const int lb_rows = lb_stride / tpr, lb_rem = lb_stride % tpr;
        for (long long i = warp - W; i < my_tiles; i += NLB, cur.advance(lb_stride, lb_rows, lb_rem, tpr)) {
            const long long T = cur.T;
            const int b = (int)(i % kLbRing);
            bool failed = false;
            unsigned int npolls = 0;
            // (the tile's own aggregate first: the warp must not run ahead of the ring slots the compute warps hold)
            if (!mbar_wait_abortable(total_bar + 8 * b, (uint32_t)((i / kLbRing) & 1), kCopySpinLimit, &xc->abort)) {
                if (lane == 0) mbar_arrive(carry_bar + 8 * b);  // (the compute warps look at the abort flag next)
                break;
            }
            E carry;
            if (served) carry = LB::await_entering(p, T, &xc->abort, failed, npolls);
            else carry = CE::row_start(p, cur.row);  // every row is a single tile
            if (lane == 0) {
                if (failed) {
                    record_error(p, kErrLookbackTimeout, T);
                    xc->abort = 1;
                }
                xc->carry[b] = make_float4(carry.m, carry.s, 0.0f, 0.0f);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(carry_bar + 8 * b);  // releases wexcl, carry and abort to the CTA
            if (failed) break;
        }
        return;
    }

    // ---------------------------------------------------------------------- compute warps
    LaneMap lm;
    lm.R = 1; lm.g = 0; lm.i = lane; lm.W = CHUNK;
    const typename CE::Offsets off = CE::offsets(lm);
    uint32_t park_off[K / 4];  // the lane's K partial sums as fp32 units
#pragma unroll
    for (int jx = 0; jx < K / 4; ++jx) park_off[jx] = chunk_off(1, 0, (uint32_t)((lane * (K / 4) + jx) * 16));

    const uint32_t wb = smem_u32(smem) + (uint32_t)(warp * S * ST::BYTES);
    auto st_a = [&](int st) { return wb + st * ST::BYTES; };
    auto st_b = [&](int st) { return wb + st * ST::BYTES + ST::IN_BUF; };
    auto st_park = [&](int st) { return wb + st * ST::BYTES + ST::PARK_OFF; };
    LanePark<SIGNED> lp[4];  // lp[d]: the tile that went through phase 1 d iterations ago
#pragma unroll
    for (int d = 0; d < 4; ++d) { lp[d].r = neg_inf(); lp[d].excl = identity_elem<SIGNED>(); lp[d].slow = false; }
    const uint32_t bars = warp_bars + warp * (8 * kLbMaxStages);

    // TMA helpers (same box geometry as WarpPipe, buffers laid out per stage here)
    const bool flat = p.flat_boxes != 0;
    constexpr int IN_PER_BOX = 128 / (int)sizeof(TIn), OUT_PER_BOX = 128 / (int)sizeof(TOut);
    const int in_boxes = flat ? 1 : ST::IN_BYTES / 128;
    constexpr int OUT_LINES = (CHUNK * (int)sizeof(TOut)) / 128;
    const int out_boxes = flat ? 1 : OUT_LINES;  // lanes that issue stores
    // flat boxes: first column of the chunk that holds the row's last n % line elements, if there are any
    const int tail_colbase_in = (flat && p.n % CE::IN_LINE) ? (int)(p.n / CE::IN_LINE) * CE::IN_LINE / CHUNK * CHUNK : -1;
    const int tail_colbase_out = (flat && p.n % CE::OUT_LINE) ? (int)(p.n / CE::OUT_LINE) * CE::OUT_LINE / CHUNK * CHUNK : -1;

    const int g_rows = (int)G / tpr, g_rem = (int)G % tpr;
    TileCursor ci, c1, c2;  // tiles being loaded, in phase 1, in phase 2
    ci.init(first, tpr);
    c1 = ci;
    c2 = ci;
    auto colbase_of = [&](const TileCursor& c) { return (c.j * W + warp) * CHUNK; };
    long long issued = 0;
    int istage = 0;
    // loads run a tile ahead of phase 1: TMA boxes, or groups of asynchronous 4-byte copies
    // (without TMA: the chunk's 16-byte units copied asynchronously as they are -- see ChunkEngine::Wide)
    constexpr bool AHEAD = true;
    auto issue_next = [&]() {
        if (issued < my_tiles) {
            const int cb = colbase_of(ci);
            const uint32_t bar = bars + 8 * istage;
            // (a chunk of the row's last tile may lie wholly beyond the row: TMA fills it with zeros, the plain path skips it)
            HS_DBG_CHECK(ci.row >= 0 && ci.row < p.rows && ((cb * (int)sizeof(TIn)) & 15) == 0 && istage < S, kDbgTmaCoord,
                         ((unsigned long long)ci.row << 32) | (unsigned)cb, return);
            if (!TMA) {
                CE::wide_load_async(p, st_a(istage), st_b(istage), lane, ci.row, cb, CHUNK);
            } else if (flat) {
                if (lane == 0) mbar_expect_tx(bar, 2 * ST::IN_BYTES);
                __syncwarp();
                if (lane == 0) {
                    tma_load_3d(st_a(istage), &tm_a, 0, cb / IN_PER_BOX, ci.row, bar);
                    tma_load_3d(st_b(istage), &tm_b, 0, cb / IN_PER_BOX, ci.row, bar);
                }
            } else {
                if (lane == 0) mbar_expect_tx(bar, 2 * ST::IN_BYTES);
                __syncwarp();
                if (lane < in_boxes) {
                    const int x = (cb + lane * IN_PER_BOX) * Storage<TIn>::kTmaScale;
                    tma_load_2d(st_a(istage) + lane * 128, &tm_a, x, ci.row, bar);
                    tma_load_2d(st_b(istage) + lane * 128, &tm_b, x, ci.row, bar);
                }
            }
            ++issued;
            if (++istage == S) istage = 0;
            ci.advance((int)G, g_rows, g_rem, tpr);
        }
    };
    if (AHEAD) issue_next();

    bool aborted = false;
    long long consumed = 0;
    int st1 = 0, st2 = 0;          // stages of the tiles in phase 1 / phase 2
    uint32_t par1 = 0;             // parity of stage st1's mbarrier
    int b1 = 0, b2 = 0;            // ring slots of those tiles
    uint32_t parb2 = 0;            // parity of ring slot b2's carry mbarrier
    for (long long i = 0; i < my_tiles + D && !aborted; ++i) {
        lp[3] = lp[2]; lp[2] = lp[1]; lp[1] = lp[0];
        // ---- phase 1 of tile i
        if (i < my_tiles) {
            const long long row = c1.row;
            const int colbase = colbase_of(c1);
            const int st = st1, b = b1;
            if (TMA) {
                // tile i+1 goes into the stage whose tile finished phase 2 in the previous iteration;
                // the store issued from it then has been read by now
                if (lane < out_boxes) bulk_wait_read<0>();
                __syncwarp();
                issue_next();
                if (!mbar_wait_bounded(bars + 8 * st, par1, kCopySpinLimit)) {
                    if (lane == 0) { record_error(p, kErrCopyTimeout, c1.T); xc->abort = 1; }
                    aborted = true;
                } else {
                    ++consumed;
                    if (colbase == tail_colbase_in) {  // the box brought the row's whole lines; fetch the rest
                        CE::tail_load(p, st_a(st), st_b(st), lane, row, colbase);
                        __syncwarp();
                    }
                }
            } else if (AHEAD) {
                // (the tile that left this stage was stored by plain stores, which are done)
                issue_next();
                // this tile's group of copies is the oldest one pending; at most one newer group is in flight
                if (issued - consumed > 1) cp_async_wait<1>();
                else cp_async_wait<0>();
                __syncwarp();
                ++consumed;
            }
            if (!aborted) {
                const long long col0 = colbase + lane * K;
                typename CE::Pending pd;
                E total;
                const typename CE::Wide wd = CE::wide_of(p, row, PLAIN);
                CE::template phase1<PLAIN>(p, st_a(st), st_b(st), off, lm, lane, row, col0, colbase + CHUNK > p.n, wd, pd, total);
                if (MODE == kLinear && !pd.slow) {
                    // phase 2 gets g_t = +-exp(A_t / 2) instead of A_t and the parities (see Run::outputs); where that
                    // would leave fp32's range, the chunk keeps its inputs and phase 2 takes the tracked form
                    float amx = 0.0f;
#pragma unroll
                    for (int t = 0; t < K; t += 2) amx = max3(amx, fabsf(pd.run.A[t]), fabsf(pd.run.A[t + 1]));
                    if (__any_sync(0xffffffffu, !(amx <= 240.0f))) pd.slow = true;
                }
                if (!pd.slow) {  // park the partial sums (a slow chunk keeps its inputs instead)
                    const uint32_t pb = st_park(st);
                    // (wide staging: a lane's inputs reach into the unit after its own, where its neighbour parks;
                    // elements wider than the parked sums: a lane parks over other lanes' inputs)
                    if (PLAIN || sizeof(TIn) > 4) __syncwarp();
#pragma unroll
                    for (int jx = 0; jx < K / 4; ++jx) sts128(pb + park_off[jx], Storage<float>::pack(pd.run.s + 4 * jx));
                    if (MODE == kLinear) {
                        // ... and g_t over the a-tensor chunk: phase 2 would otherwise take the logarithm of every
                        // a_t a second time
                        const uint32_t ab = st_a(st);
#pragma unroll
                        for (int jx = 0; jx < K / 4; ++jx) {
                            float g[4];
#pragma unroll
                            for (int q = 0; q < 4; q += 2) {
                                const int t = 4 * jx + q;
                                const float2 h = mul2(pk(pd.run.A[t], pd.run.A[t + 1]), pk(0.5f));
                                const float2 gg = mul2(pk(ex2(h.x), ex2(h.y)), pk(pd.run.Pf[t], pd.run.Pf[t + 1]));
                                g[q] = gg.x;
                                g[q + 1] = gg.y;
                            }
                            sts128(ab + park_off[jx], Storage<float>::pack(g));
                        }
                    }
                }
                lp[0].r = pd.run.r;
                lp[0].excl = pd.excl;
                lp[0].slow = pd.slow;
                if (lane == 0) xc->agg[b][warp] = pack_elem<SIGNED>(total);
                __syncwarp();
                if (lane == 0) mbar_arrive(agg_bar + 8 * b);
            }
            c1.advance((int)G, g_rows, g_rem, tpr);
            if (++st1 == S) { st1 = 0; par1 ^= 1u; }
            if (++b1 == kLbRing) b1 = 0;
        }
        // ---- phase 2 of tile i-D
        if (i >= D && !aborted) {
            const long long row = c2.row;
            const int colbase = colbase_of(c2);
            const int st = st2, b = b2;
            const bool carry_ok = mbar_wait_bounded(carry_bar + 8 * b, parb2, kCopySpinLimit);
            if (!carry_ok) {
                if (lane == 0) { record_error(p, kErrLookbackTimeout, c2.T); xc->abort = 1; }
                aborted = true;
            } else if (*(volatile int*)&xc->abort) {
                aborted = true;
            }
            if (!aborted) {
                const long long col0 = colbase + lane * K;
                const long long left = p.n - col0;
                const typename CE::Wide wd = CE::wide_of(p, row, PLAIN);
                E carry;
                carry.A = neg_inf(); carry.m = xc->carry[b].x; carry.s = xc->carry[b].y; carry.p = 0u;
                const LanePark<SIGNED> mine = (D == 1) ? lp[1] : (D == 2) ? lp[2] : lp[3];
                const E excl = mine.excl;
                const E entering = compose(compose(carry, unpack_elem<SIGNED>(xc->agg[b][warp])), excl);
                uint32_t sm_a = st_a(st);
                uint32_t sm_b = st_b(st);
                const uint32_t pb = st_park(st);
                bool ok = false;
                const bool was_slow = mine.slow;  // (warp-uniform)
                if (!was_slow) {
                    R_ run;
                    // rebuild A_t (and the parity of a) from the inputs -- kLinear: fetch the parked A_t --,
                    // fetch the parked s_t, apply
                    float va[K];
                    uint32_t sa[MODE == kLogSigned ? K : 1];
                    if (MODE == kLinear) {
#pragma unroll
                        for (int jx = 0; jx < K / 4; ++jx) Storage<float>::unpack(lds128(sm_a + park_off[jx]), run.A + 4 * jx);
                        run.bad = false;
                    } else {
                        if (PLAIN) Shifted<TIn, K>::read_signed(sm_a, off.in, wd.phi_a, va, sa);
                        else R_::load_a_signed(sm_a, off.in, va, sa);
                        if (colbase + CHUNK > p.n) {
#pragma unroll
                            for (int t = 0; t < K; ++t)
                                if (t >= left) {
                                    va[t] = neutral_a<MODE>();
                                    if (MODE == kLogSigned) sa[t] = 0u;
                                }
                        }
                        if (CE::SIGN_TENSORS) CE::load_signs(p.sign_a, row * p.n + col0, left, p.sign_vec_ok != 0, sa);
                        run.rebuild(va, sa);
                    }
                    run.r = mine.r;
#pragma unroll
                    for (int jx = 0; jx < K / 4; ++jx) Storage<float>::unpack(lds128(pb + park_off[jx]), run.s + 4 * jx);
                    typename R_::Applied ap = run.prepare(entering);
                    ok = __all_sync(0xffffffffu, ap.ok);  // also: every lane has read its parked sums
                    if (MODE == kLinear) ap.hM = ex2(ap.M * (0.5f * kLog2e));
                    if (ok) CE::template emit_outputs<PLAIN, MODE == kLinear>(p, run, ap, pb, off, wd, row * p.n + col0, left);
                }
                if (!ok) {
                    // where the lane's inputs are now: as staged (shifted) when the chunk kept them, at the lane's
                    // own units when they are fetched again below
                    uint32_t phi_a = PLAIN ? wd.phi_a : 0u, phi_b = PLAIN ? wd.phi_b : 0u;
                    if (!was_slow && ST::IN_PLACE) {
                        // the parked sums replaced the b-tensor chunk: fetch the lane's b values again
                        __syncwarp();
#pragma unroll
                        for (int t = 0; t < K; ++t) {
                            const uint32_t at = chunk_off(1, 0, (uint32_t)((lane * K + t) * sizeof(TIn)));
                            if (t < left) Storage<TIn>::copy_in(sm_b + at, p.in_b, row * p.n + col0 + t);
                            else Storage<TIn>::to_smem(sm_b + at, neutral_b<MODE>());
                            if (MODE == kLinear) {  // A_t replaced the a-tensor chunk as well
                                if (t < left) Storage<TIn>::copy_in(sm_a + at, p.in_a, row * p.n + col0 + t);
                                else Storage<TIn>::to_smem(sm_a + at, neutral_a<MODE>());
                            }
                        }
                        phi_b = 0u;
                        if (MODE == kLinear) phi_a = 0u;
                        __syncwarp();
                    }
                    const typename CE::SlowOut so =
                        CE::slow_apply(entering, sm_a, sm_b, lm, CE::SIGN_TENSORS ? p.sign_a : nullptr,
                                       CE::SIGN_TENSORS ? p.sign_b : nullptr, row * p.n + col0, left, phi_a, phi_b);
                    __syncwarp();
                    CE::template write_outputs<PLAIN>(pb, off, wd, so.vals, so.sgn);
                    if (CE::SIGN_TENSORS) CE::store_signs(p.sign_x, row * p.n + col0, left, p.sign_vec_ok != 0, so.sgn);
                }
                if (TMA) {
                    fence_async_smem();
                    __syncwarp();
                    // a flat box holds the whole lines of the row that fall into the chunk (the hardware clips it
                    // at the row's last whole line); what is left of the row goes out by plain stores
                    if (flat) {
                        if (lane == 0 && colbase < p.n) {
                            tma_store_3d(&tm_o, 0, colbase / OUT_PER_BOX, (int)row, pb);
                            bulk_commit();
                        }
                        if (colbase == tail_colbase_out) CE::tail_store(p, pb, lane, row, colbase);
                    } else if (lane < out_boxes) {
                        tma_store_2d(&tm_o, (colbase + lane * OUT_PER_BOX) * Storage<TOut>::kTmaScale, (int)row,
                                     pb + (uint32_t)(lane * 128));
                        bulk_commit();
                    }
                } else {
                    __syncwarp();
                    CE::wide_store(p, st_park(st), lane, row, colbase, CHUNK);
                }
                __syncwarp();  // every lane is done with this tile's stage
            }
            c2.advance((int)G, g_rows, g_rem, tpr);
            if (++st2 == S) st2 = 0;
            if (++b2 == kLbRing) { b2 = 0; parb2 ^= 1u; }
        }
    }
    if (TMA) {
        if (aborted) {
            for (long long c = consumed; c < issued; ++c)
                (void)mbar_wait_bounded(bars + 8 * (int)(c % S), (uint32_t)((c / S) & 1), kCopySpinLimit);
        }
        if (lane < out_boxes) bulk_wait_all();
        __syncwarp();
    }
}

}  // namespace hs
