// Device-side building blocks of libheinsen_scan (sm_100a only).
//
// Notation follows the paper: a*_t = cumsum(log a_t) (Eq. 2), LCSE = log cumsum exp (Eq. 8),
// x_0 is prepended to the second scan as the paper's cat(log x_0, .) (Eq. 7).
//
// The associativity of prefix sums (Summary, footnote) lets both scans be computed by parts.
// A part [i..j] is summarised by the affine map x -> alpha*x + beta it applies to the value
// entering it, kept in log space:
//     alpha = (-1)^p * exp(A),   A = sum of log|a| over the part,   p = parity of negative a's
//     beta  = s * exp(m),        m = log-sum-exp reference ("max tracking"), s = signed scaled sum
// Composing two parts needs one exp of a non-positive number.  The value of x itself is the
// part that starts at x_0, for which alpha is irrelevant.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace hs {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr uint32_t kSignBit = 0x80000000u;
// Reference of an empty sum (beta == 0, s == 0).  A large finite value instead of -inf keeps
// differences of references free of inf - inf without a guard in the inner combine.
constexpr float kEmpty = -1e20f;

enum Mode : int { kLogUnsigned = 0, kLogSigned = 1, kLinear = 2, kPairs = 3 /* linear-domain comparison path */ };

__device__ __forceinline__ float neg_inf() { return __int_as_float(0xff800000); }

// MUFU wrappers: one instruction each.
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float lg2(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float rcp_approx(float x) {
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float flip(float v, uint32_t mask) { return __uint_as_float(__float_as_uint(v) ^ mask); }
// three-input maximum / minimum: one instruction on sm_100
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float min3(float a, float b, float c) {
    float d;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// Natural logarithm of |v| accurate to about one ulp also for v close to 1, where lg2.approx's
// absolute error would be a large relative error of log a_t and would bias a*_t over a long
// sequence.  v = m*2^e with m in [2/3, 4/3); log m = 2 atanh(w), w = (m-1)/(m+1), odd series.
__device__ __forceinline__ float log_abs_accurate(float v) {
    v = fabsf(v);
    const bool zero = (v == 0.0f);
    const bool tiny = (v < 1.17549435e-38f);
    const float bias = tiny ? -23.0f : 0.0f;
    v = tiny ? v * 8388608.0f : v;
    const int bits = __float_as_int(v);
    const int e = (bits - 0x3f2aaaab) >> 23;
    const float m = __int_as_float(bits - (e << 23));
    const float f = m - 1.0f;
    const float d = 2.0f + f;
    const float r = rcp_approx(d);
    float w = f * r;
    w = fmaf(fmaf(-w, d, f), r, w);  // one Newton correction of the quotient
    const float w2 = w * w;
    float poly = fmaf(w2, 1.0f / 9.0f, 1.0f / 7.0f);
    poly = fmaf(w2, poly, 1.0f / 5.0f);
    poly = fmaf(w2, poly, 1.0f / 3.0f);
    poly = poly * w2;
    const float lm = fmaf(2.0f * w, poly, 2.0f * w);
    return zero ? neg_inf() : fmaf((float)e + bias, kLn2, lm);
}

// Packed fp32 pairs (sm_100's f32x2 arithmetic): one instruction, hence one issue slot, for two
// elements.  The kernels are short of issue slots before they are short of anything else, so all
// element-wise arithmetic of a lane's run is written on pairs of neighbouring elements.
__device__ __forceinline__ float2 pk(float x, float y) { return make_float2(x, y); }
__device__ __forceinline__ float2 pk(float x) { return make_float2(x, x); }
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) { return __ffma2_rn(a, b, c); }
__device__ __forceinline__ float2 mul2(float2 a, float2 b) { return __fmul2_rn(a, b); }
__device__ __forceinline__ float2 add2(float2 a, float2 b) { return __fadd2_rn(a, b); }

// log2|v| for the hot path of the linear entry point, about half the cost of log_abs_accurate, in binary
// logarithms because that is what ex2 / lg2 work in (the linear entry point keeps the A_t of a run in these
// units): near 1 (|v| in (0.875, 1.125)) the Taylor series of log(1+f) in f = |v| - 1 (exact in fp32) to the
// sixth power, its coefficients carrying the factor log2(e), relative error <= |f|^6 / 7 <= 5.5e-7; elsewhere
// lg2.approx, whose absolute error of 2^-22 is there a relative error <= 1.4e-6 of the logarithm (inside the
// 2e-6 |a*_t| term of the tolerance even if it never cancelled).  |v| = 0 and denormals give -inf.
__device__ __forceinline__ float log2_abs_fast(float v) {
    const float av = fabsf(v);
    const float f = av - 1.0f;
    float p = fmaf(f, -kLog2e / 6.0f, kLog2e / 5.0f);
    p = fmaf(p, f, -kLog2e / 4.0f);
    p = fmaf(p, f, kLog2e / 3.0f);
    p = fmaf(p, f, -kLog2e / 2.0f);
    p = fmaf(p, f, kLog2e);
    return (fabsf(f) < 0.125f) ? p * f : lg2(av);
}
// ... on two values at once.
__device__ __forceinline__ float2 log2_abs_fast2(float2 v) {
    const float2 av = pk(fabsf(v.x), fabsf(v.y));
    const float2 f = add2(av, pk(-1.0f));
    float2 p = fma2(f, pk(-kLog2e / 6.0f), pk(kLog2e / 5.0f));
    p = fma2(p, f, pk(-kLog2e / 4.0f));
    p = fma2(p, f, pk(kLog2e / 3.0f));
    p = fma2(p, f, pk(-kLog2e / 2.0f));
    p = fma2(p, f, pk(kLog2e));
    const float2 near_one = mul2(p, f);
    return pk((fabsf(f.x) < 0.125f) ? near_one.x : lg2(av.x), (fabsf(f.y) < 0.125f) ? near_one.y : lg2(av.y));
}

// ------------------------------------------------------------------------------------------
// The associative element.
template <bool SIGNED>
struct Elem {
    float A;     // sum of log|a|
    float m;     // reference of beta = s*exp(m), always finite (>= about kEmpty); beta == 0 <=> s == 0
    float s;     // signed, scaled sum
    uint32_t p;  // sign mask (0 or 0x80000000) of alpha; unused when !SIGNED
};

template <bool SIGNED>
__device__ __forceinline__ Elem<SIGNED> identity_elem() {
    Elem<SIGNED> e;
    e.A = 0.0f; e.m = kEmpty; e.s = 0.0f; e.p = 0u;
    return e;
}

// "first" is the older part, "second" the newer one: result = second o first.
// second.m must be finite (it always is: leaves and aggregates clamp at kEmpty); first.m + second.A
// may be -inf (a_t = 0 inside the second part wipes out the first part's beta).
template <bool SIGNED>
__device__ __forceinline__ Elem<SIGNED> compose(const Elem<SIGNED>& first, const Elem<SIGNED>& second) {
    Elem<SIGNED> o;
    o.A = first.A + second.A;
    const float m1 = first.m + second.A;  // beta_1 carried through alpha_2
    const float s1 = SIGNED ? flip(first.s, second.p) : first.s;
    o.m = fmaxf(m1, second.m);
    const float d = m1 - second.m;
    const float e = ex2(-fabsf(d) * kLog2e);
    const bool first_is_ref = (d >= 0.0f);
    const float hi = first_is_ref ? s1 : second.s;
    const float lo = first_is_ref ? second.s : s1;
    o.s = fmaf(lo, e, hi);
    o.p = SIGNED ? (first.p ^ second.p) : 0u;
    return o;
}

template <bool SIGNED>
__device__ __forceinline__ Elem<SIGNED> shfl_up_elem(const Elem<SIGNED>& e, int delta) {
    Elem<SIGNED> o;
    o.A = __shfl_up_sync(0xffffffffu, e.A, delta);
    o.m = __shfl_up_sync(0xffffffffu, e.m, delta);
    o.s = __shfl_up_sync(0xffffffffu, e.s, delta);
    o.p = SIGNED ? __shfl_up_sync(0xffffffffu, e.p, delta) : 0u;
    return o;
}
template <bool SIGNED>
__device__ __forceinline__ Elem<SIGNED> shfl_elem(const Elem<SIGNED>& e, int src) {
    Elem<SIGNED> o;
    o.A = __shfl_sync(0xffffffffu, e.A, src);
    o.m = __shfl_sync(0xffffffffu, e.m, src);
    o.s = __shfl_sync(0xffffffffu, e.s, src);
    o.p = SIGNED ? __shfl_sync(0xffffffffu, e.p, src) : 0u;
    return o;
}
template <bool SIGNED>
__device__ __forceinline__ Elem<SIGNED> shfl_down_elem(const Elem<SIGNED>& e, int delta) {
    Elem<SIGNED> o;
    o.A = __shfl_down_sync(0xffffffffu, e.A, delta);
    o.m = __shfl_down_sync(0xffffffffu, e.m, delta);
    o.s = __shfl_down_sync(0xffffffffu, e.s, delta);
    o.p = SIGNED ? __shfl_down_sync(0xffffffffu, e.p, delta) : 0u;
    return o;
}

// Inclusive Kogge-Stone scan (the Hillis-Steele pattern the paper cites for O(log n) prefix sums)
// over the lanes that share a row.  A warp holds R rows (R = 1, 2, 4 or 8); lane = i*R + g is
// segment i of row g, so the lanes of one row are R apart and the scan takes log2(32/R) steps.
// Returns the exclusive prefix of each lane and the total of its row (held by every lane of the row).
template <bool SIGNED>
__device__ __forceinline__ void row_scan(const Elem<SIGNED>& mine, int lane, int R, Elem<SIGNED>& exclusive,
                                         Elem<SIGNED>& total) {
    Elem<SIGNED> inc = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        if (d >= R) {  // warp-uniform
            Elem<SIGNED> up = shfl_up_elem(inc, d);
            Elem<SIGNED> c = compose(up, inc);
            if (lane >= d) inc = c;
        }
    }
    total = shfl_elem(inc, 32 - R + (lane & (R - 1)));
    Elem<SIGNED> up = shfl_up_elem(inc, R);
    exclusive = (lane < R) ? identity_elem<SIGNED>() : up;
}

// Plain 32-lane scan (one row per warp), used for the per-warp aggregates of a look-back tile.
template <bool SIGNED>
__device__ __forceinline__ void warp_scan(const Elem<SIGNED>& mine, int lane, Elem<SIGNED>& exclusive,
                                          Elem<SIGNED>& total) {
    row_scan(mine, lane, 1, exclusive, total);
}

// The running value x = s*exp(m) as an element (alpha irrelevant: A = -inf absorbs whatever
// came before, exactly as prepending log x_0 to the second scan does in Eq. 7).
template <bool SIGNED>
__device__ __forceinline__ Elem<SIGNED> state_elem(float log_mag, uint32_t sign_mask) {
    Elem<SIGNED> e;
    e.A = neg_inf();
    e.m = fmaxf(log_mag, kEmpty);
    e.s = (log_mag == neg_inf()) ? 0.0f : (SIGNED ? flip(1.0f, sign_mask) : 1.0f);
    e.p = 0u;
    return e;
}

// Bring |s| back into [1,2) once it has drifted 20 binary orders away, so that a long signed cancellation
// cannot strand the reference far above the value (and s, in the end, below fp32's range).  Exact apart from
// one rounding of m.
template <bool SIGNED>
__device__ __forceinline__ void renormalise(Elem<SIGNED>& e) {
    if (!SIGNED) return;
    const float as = fabsf(e.s);
    if (as >= 9.5367431640625e-07f /* 2^-20 */ && as <= 1048576.0f /* 2^20 */) return;  // nowhere near fp32's limits
    if (as == 0.0f) { e.m = kEmpty; e.s = 0.0f; return; }
    if (as >= 1.17549435e-38f) {
        const int ex = ((__float_as_int(as) >> 23) & 0xff) - 127;
        e.m = fmaf((float)ex, kLn2, e.m);
        e.s = __int_as_float(__float_as_int(e.s) - (ex << 23));
    }
}

// ------------------------------------------------------------------------------------------
// Shared-memory chunk layout.  A warp's chunk is R rows x (32/R lanes x K elements): every row
// contributes one contiguous piece, fetched by TMA as boxes of {128 bytes, R rows} with the
// 128-byte swizzle.  Box b of a chunk lands at byte b*R*128; inside, row g of the box is the
// shared-memory row b*R+g, whose 16-byte units are XORed with (row & 7).  A lane reading its own
// K contiguous elements with 128-bit loads is then bank-conflict free (the 8 lanes of a
// wavefront fall on 8 different unit positions).
// byte_in_row: byte offset inside the row's piece of the chunk.
__device__ __forceinline__ uint32_t chunk_off(int R, int g, uint32_t byte_in_row) {
    const uint32_t srow = (byte_in_row >> 7) * (uint32_t)R + (uint32_t)g;
    return (srow << 7) + (((((byte_in_row >> 4) ^ srow) & 7u)) << 4) + (byte_in_row & 15u);
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ------------------------------------------------------------------------------------------
// Checked build (-DHEINSEN_DEBUG).  compute-sanitizer is not always available where this library runs, so
// the library can be built with its own index checks: every shared-memory access of the wrappers below
// verifies that its address lies inside the CTA's dynamic shared memory and is aligned to its width, and the
// kernels verify the element, row, tile and TMA coordinates they are about to use (HS_DBG_CHECK).  A check
// that fails never traps: it records {code, detail, block, thread} in g_debug_fault (the first failure of a
// process wins; heinsen_scan_debug_faults() reads and clears it) and the access is skipped.  In the normal
// build all of this compiles to nothing.
// The predicate itself is plain arithmetic, shared with the host so that it can be unit-tested without a GPU.
__host__ __device__ inline bool debug_window_ok(unsigned long long addr, unsigned long long bytes, unsigned long long base,
                                                unsigned long long size, unsigned long long align) {
    return addr >= base && bytes <= size && addr - base <= size - bytes && (addr % align) == 0;
}
enum DebugCode : int {
    kDbgSmemWindow = 1,   // shared-memory address outside the CTA's dynamic shared memory, or misaligned
    kDbgElement = 2,      // element index outside [0, rows * n)
    kDbgRow = 3,          // row index outside [0, rows)
    kDbgTile = 4,         // tile / group descriptor index outside the descriptor arrays
    kDbgTmaCoord = 5,     // TMA coordinate out of range or not on a 16-byte boundary
    kDbgUnits = 6         // 16-byte unit copy reaching beyond the units that hold the tensor
};
#ifdef HEINSEN_DEBUG
__device__ unsigned long long g_debug_fault[4];
__device__ __noinline__ void debug_record(int code, unsigned long long detail) {
    if (atomicCAS(&g_debug_fault[0], 0ull, (unsigned long long)code) == 0ull) {
        g_debug_fault[1] = detail;
        g_debug_fault[2] = blockIdx.x;
        g_debug_fault[3] = threadIdx.x;
    }
}
__device__ __forceinline__ bool debug_smem_ok(uint32_t addr, uint32_t bytes) {
    extern __shared__ uint8_t hs_debug_dynamic_smem[];
    uint32_t size;
    asm volatile("mov.u32 %0, %%dynamic_smem_size;" : "=r"(size));
    const uint32_t base = smem_u32(hs_debug_dynamic_smem);
    if (debug_window_ok(addr, bytes, base, size, bytes)) return true;
    debug_record(kDbgSmemWindow, ((unsigned long long)addr << 32) | bytes);
    return false;
}
#define HS_DBG_SMEM(addr, bytes, fail) \
    do {                               \
        if (!debug_smem_ok((addr), (bytes))) fail; \
    } while (0)
// `cond` must hold; otherwise the failure is recorded and `fail` runs (skip the access)
#define HS_DBG_CHECK(cond, code, detail, fail)                               \
    do {                                                                     \
        if (!(cond)) {                                                       \
            debug_record((code), (unsigned long long)(detail));              \
            fail;                                                            \
        }                                                                    \
    } while (0)
#else
#define HS_DBG_SMEM(addr, bytes, fail) do { } while (0)
#define HS_DBG_CHECK(cond, code, detail, fail) do { } while (0)
#endif

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    HS_DBG_SMEM(addr, 16u, return make_uint4(0u, 0u, 0u, 0u));
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint4 v) {
    HS_DBG_SMEM(addr, 16u, return);
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

template <typename T>
struct Storage;
template <>
struct Storage<float> {
    static constexpr int kPerUnit = 4;
    __device__ static __forceinline__ void unpack(uint4 u, float* o) {
        o[0] = __uint_as_float(u.x); o[1] = __uint_as_float(u.y); o[2] = __uint_as_float(u.z); o[3] = __uint_as_float(u.w);
    }
    __device__ static __forceinline__ uint4 pack(const float* v) {
        return make_uint4(__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3]));
    }
    __device__ static __forceinline__ float load(const void* p, int64_t i) { return ((const float*)p)[i]; }
    __device__ static __forceinline__ void store(void* p, int64_t i, float v) { ((float*)p)[i] = v; }
    // addr: 32-bit shared-memory address
    __device__ static __forceinline__ float from_smem(uint32_t addr) {
        float v;
        HS_DBG_SMEM(addr, 4u, return 0.0f);
        asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
        return v;
    }
    __device__ static __forceinline__ void to_smem(uint32_t addr, float v) {
        HS_DBG_SMEM(addr, 4u, return);
        asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
    }
    // A storage type may carry the sign of a value itself (complex logarithms do); these do not.
    static constexpr bool kCarriesSign = false;
    static constexpr int kTmaScale = 1;  // tensor-map elements per stored element
    __device__ static __forceinline__ void unpack_signed(uint4 u, float* o, uint32_t*) { unpack(u, o); }
    __device__ static __forceinline__ uint4 pack_signed(const float* v, const uint32_t*) { return pack(v); }
    __device__ static __forceinline__ uint32_t sign_from_smem(uint32_t) { return 0u; }
    __device__ static __forceinline__ uint32_t load_sign(const void*, int64_t) { return 0u; }
    // one element moved as it is, global -> shared / shared -> global
    __device__ static __forceinline__ void copy_in(uint32_t addr, const void* p, int64_t i) { to_smem(addr, load(p, i)); }
    __device__ static __forceinline__ void copy_out(void* p, int64_t i, uint32_t addr) { store(p, i, from_smem(addr)); }
};
template <>
struct Storage<__nv_bfloat16> {
    static constexpr int kPerUnit = 8;
    __device__ static __forceinline__ void unpack(uint4 u, float* o) {
        o[0] = __uint_as_float(u.x << 16); o[1] = __uint_as_float(u.x & 0xffff0000u);
        o[2] = __uint_as_float(u.y << 16); o[3] = __uint_as_float(u.y & 0xffff0000u);
        o[4] = __uint_as_float(u.z << 16); o[5] = __uint_as_float(u.z & 0xffff0000u);
        o[6] = __uint_as_float(u.w << 16); o[7] = __uint_as_float(u.w & 0xffff0000u);
    }
    __device__ static __forceinline__ uint32_t pack2(float lo, float hi) {
        __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&h);
    }
    __device__ static __forceinline__ uint4 pack(const float* v) {
        return make_uint4(pack2(v[0], v[1]), pack2(v[2], v[3]), pack2(v[4], v[5]), pack2(v[6], v[7]));
    }
    __device__ static __forceinline__ float load(const void* p, int64_t i) {
        return __bfloat162float(((const __nv_bfloat16*)p)[i]);
    }
    __device__ static __forceinline__ void store(void* p, int64_t i, float v) {
        ((__nv_bfloat16*)p)[i] = __float2bfloat16_rn(v);
    }
    __device__ static __forceinline__ float from_smem(uint32_t addr) {
        unsigned short h;
        HS_DBG_SMEM(addr, 2u, return 0.0f);
        asm volatile("ld.shared.u16 %0, [%1];" : "=h"(h) : "r"(addr));
        return __uint_as_float((uint32_t)h << 16);
    }
    __device__ static __forceinline__ void to_smem(uint32_t addr, float v) {
        const __nv_bfloat16 b = __float2bfloat16_rn(v);
        HS_DBG_SMEM(addr, 2u, return);
        asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"(*reinterpret_cast<const unsigned short*>(&b)) : "memory");
    }
    static constexpr bool kCarriesSign = false;
    static constexpr int kTmaScale = 1;
    __device__ static __forceinline__ void unpack_signed(uint4 u, float* o, uint32_t*) { unpack(u, o); }
    __device__ static __forceinline__ uint4 pack_signed(const float* v, const uint32_t*) { return pack(v); }
    __device__ static __forceinline__ uint32_t sign_from_smem(uint32_t) { return 0u; }
    __device__ static __forceinline__ uint32_t load_sign(const void*, int64_t) { return 0u; }
    __device__ static __forceinline__ void copy_in(uint32_t addr, const void* p, int64_t i) {
        HS_DBG_SMEM(addr, 2u, return);
        asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"(((const unsigned short*)p)[i]) : "memory");
    }
    __device__ static __forceinline__ void copy_out(void* p, int64_t i, uint32_t addr) {
        unsigned short h;
        HS_DBG_SMEM(addr, 2u, return);
        asm volatile("ld.shared.u16 %0, [%1];" : "=h"(h) : "r"(addr));
        ((unsigned short*)p)[i] = h;
    }
};

// The logarithm of a real number as the paper writes it for negative values (Summary, last paragraph): a
// complex number (log|v|, k*pi) on the principal branch, k odd for a negative v.  Stored as two floats; the
// kernels take the magnitude from the real part and one sign bit from the imaginary part, and write
// (log|x|, 0) or (log|x|, pi).
struct cplx {
    float re, im;
};
constexpr float kPi = 3.14159265358979323846f;
template <>
struct Storage<cplx> {
    static constexpr int kPerUnit = 2;
    static constexpr bool kCarriesSign = true;
    static constexpr int kTmaScale = 2;
    // parity of round(im / pi) as a sign mask: adding 1.5 * 2^23 leaves the rounded integer in the low mantissa bits
    __device__ static __forceinline__ uint32_t sign_of(uint32_t im_bits) {
        return __float_as_uint(fmaf(__uint_as_float(im_bits), 1.0f / kPi, 12582912.0f)) << 31;
    }
    __device__ static __forceinline__ uint32_t imag_of(uint32_t sign_mask) { return sign_mask ? __float_as_uint(kPi) : 0u; }
    __device__ static __forceinline__ void unpack(uint4 u, float* o) {
        o[0] = __uint_as_float(u.x); o[1] = __uint_as_float(u.z);
    }
    __device__ static __forceinline__ void unpack_signed(uint4 u, float* o, uint32_t* sg) {
        o[0] = __uint_as_float(u.x); o[1] = __uint_as_float(u.z);
        sg[0] = sign_of(u.y); sg[1] = sign_of(u.w);
    }
    __device__ static __forceinline__ uint4 pack_signed(const float* v, const uint32_t* sg) {
        return make_uint4(__float_as_uint(v[0]), imag_of(sg[0]), __float_as_uint(v[1]), imag_of(sg[1]));
    }
    __device__ static __forceinline__ uint4 pack(const float* v) {
        return make_uint4(__float_as_uint(v[0]), 0u, __float_as_uint(v[1]), 0u);
    }
    __device__ static __forceinline__ float load(const void* p, int64_t i) { return ((const cplx*)p)[i].re; }
    __device__ static __forceinline__ uint32_t load_sign(const void* p, int64_t i) {
        return sign_of(__float_as_uint(((const cplx*)p)[i].im));
    }
    __device__ static __forceinline__ float from_smem(uint32_t addr) { return Storage<float>::from_smem(addr); }
    __device__ static __forceinline__ uint32_t sign_from_smem(uint32_t addr) {
        return sign_of(__float_as_uint(Storage<float>::from_smem(addr + 4u)));
    }
    __device__ static __forceinline__ void to_smem(uint32_t addr, float v) {  // a positive value of that magnitude
        HS_DBG_SMEM(addr, 8u, return);
        asm volatile("st.shared.v2.f32 [%0], {%1, %2};" ::"r"(addr), "f"(v), "f"(0.0f) : "memory");
    }
    __device__ static __forceinline__ void copy_in(uint32_t addr, const void* p, int64_t i) {
        const float2 v = ((const float2*)p)[i];
        HS_DBG_SMEM(addr, 8u, return);
        asm volatile("st.shared.v2.f32 [%0], {%1, %2};" ::"r"(addr), "f"(v.x), "f"(v.y) : "memory");
    }
    __device__ static __forceinline__ void copy_out(void* p, int64_t i, uint32_t addr) {
        float2 v;
        HS_DBG_SMEM(addr, 8u, return);
        asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr));
        ((float2*)p)[i] = v;
    }
};

// ------------------------------------------------------------------------------------------
// A lane's K elements when the chunk sits `phi` bytes into its buffer (rows whose chunks do not start on a
// 16-byte boundary of global memory are staged unit for unit, so the misalignment travels with them).
// `off` holds the shared-memory offsets of the lane's K / kPerUnit units and of the one after them; which
// words of those units are the lane's depends on phi only, so every shift is a statically indexed variant.
__device__ __forceinline__ void sts32(uint32_t addr, uint32_t v) {
    HS_DBG_SMEM(addr, 4u, return);
    asm volatile("st.shared.b32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void sts16(uint32_t addr, uint32_t v) {
    HS_DBG_SMEM(addr, 2u, return);
    asm volatile("st.shared.b16 [%0], %1;" ::"r"(addr), "h"((unsigned short)v) : "memory");
}
template <typename T, int K>
struct Shifted;
template <int K>
struct Shifted<float, K> {
    static constexpr int UNITS = K / 4;
    template <int SH>
    __device__ static __forceinline__ void pick(const float* w, float* v) {
#pragma unroll
        for (int t = 0; t < K; ++t) v[t] = w[t + SH];
    }
    __device__ static __forceinline__ void read(uint32_t sm, const uint32_t* off, uint32_t phi, float* v) {
        float w[K + 4];
#pragma unroll
        for (int j = 0; j <= UNITS; ++j) Storage<float>::unpack(lds128(sm + off[j]), w + 4 * j);
        switch (phi >> 2) {
            case 0: pick<0>(w, v); break;
            case 1: pick<1>(w, v); break;
            case 2: pick<2>(w, v); break;
            default: pick<3>(w, v); break;
        }
    }
    template <int SH>
    __device__ static __forceinline__ void put(uint32_t sm, const uint32_t* off, const float* v) {
#pragma unroll
        for (int t = 0; t < K; ++t) sts32(sm + off[(t + SH) >> 2] + (uint32_t)(((t + SH) & 3) * 4), __float_as_uint(v[t]));
    }
    __device__ static __forceinline__ void write(uint32_t sm, const uint32_t* off, uint32_t phi, const float* v) {
        switch (phi >> 2) {
            case 0: put<0>(sm, off, v); break;
            case 1: put<1>(sm, off, v); break;
            case 2: put<2>(sm, off, v); break;
            default: put<3>(sm, off, v); break;
        }
    }
    __device__ static __forceinline__ void read_signed(uint32_t sm, const uint32_t* off, uint32_t phi, float* v, uint32_t*) {
        read(sm, off, phi, v);
    }
    __device__ static __forceinline__ void write_signed(uint32_t sm, const uint32_t* off, uint32_t phi, const float* v,
                                                        const uint32_t*) {
        write(sm, off, phi, v);
    }
};
template <int K>
struct Shifted<cplx, K> {
    static constexpr int UNITS = K / 2;
    // (the chunk starts 0 or 8 bytes into its buffer: elements are 8 bytes wide and 8-byte aligned)
    template <int SH>
    __device__ static __forceinline__ void pick(const uint32_t* w, float* v, uint32_t* sg) {
#pragma unroll
        for (int t = 0; t < K; ++t) {
            v[t] = __uint_as_float(w[2 * t + SH]);
            sg[t] = Storage<cplx>::sign_of(w[2 * t + 1 + SH]);
        }
    }
    __device__ static __forceinline__ void read_signed(uint32_t sm, const uint32_t* off, uint32_t phi, float* v, uint32_t* sg) {
        uint32_t w[2 * K + 4];
#pragma unroll
        for (int j = 0; j <= UNITS; ++j) {
            const uint4 q = lds128(sm + off[j]);
            w[4 * j] = q.x; w[4 * j + 1] = q.y; w[4 * j + 2] = q.z; w[4 * j + 3] = q.w;
        }
        if (phi) pick<2>(w, v, sg);
        else pick<0>(w, v, sg);
    }
    __device__ static __forceinline__ void write_signed(uint32_t sm, const uint32_t* off, uint32_t phi, const float* v,
                                                        const uint32_t* sg) {
        const int sh = phi ? 2 : 0;
#pragma unroll
        for (int t = 0; t < K; ++t) {
            const uint32_t addr0 = sm + off[t >> 1] + (uint32_t)((t & 1) * 8);        // phi == 0
            const uint32_t addr8 = sm + off[(t + 1) >> 1] + (uint32_t)(((t + 1) & 1) * 8);  // phi == 8
            const uint32_t addr = sh ? addr8 : addr0;
            HS_DBG_SMEM(addr, 8u, continue);
            asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(addr), "r"(__float_as_uint(v[t])),
                         "r"(Storage<cplx>::imag_of(sg[t]))
                         : "memory");
        }
    }
};
template <int K>
struct Shifted<__nv_bfloat16, K> {
    static constexpr int UNITS = K / 8;
    template <int SH>
    __device__ static __forceinline__ void pick(const uint32_t* w, float* v) {
#pragma unroll
        for (int t = 0; t < K; ++t) {
            const uint32_t word = w[(t + SH) >> 1];
            v[t] = __uint_as_float(((t + SH) & 1) ? (word & 0xffff0000u) : (word << 16));
        }
    }
    __device__ static __forceinline__ void read(uint32_t sm, const uint32_t* off, uint32_t phi, float* v) {
        uint32_t w[K / 2 + 4];
#pragma unroll
        for (int j = 0; j <= UNITS; ++j) {
            const uint4 q = lds128(sm + off[j]);
            w[4 * j] = q.x; w[4 * j + 1] = q.y; w[4 * j + 2] = q.z; w[4 * j + 3] = q.w;
        }
        switch (phi >> 1) {
            case 0: pick<0>(w, v); break;
            case 1: pick<1>(w, v); break;
            case 2: pick<2>(w, v); break;
            case 3: pick<3>(w, v); break;
            case 4: pick<4>(w, v); break;
            case 5: pick<5>(w, v); break;
            case 6: pick<6>(w, v); break;
            default: pick<7>(w, v); break;
        }
    }
    // element t goes to halfword t + SH of the lane's units
    template <int SH>
    __device__ static __forceinline__ void put(uint32_t sm, const uint32_t* off, const float* v) {
        auto addr = [&](int h) { return sm + off[h >> 3] + (uint32_t)((h & 7) * 2); };
        if (SH & 1) {
            // the first and the last element share their words with the neighbouring lanes
            sts16(addr(SH), Storage<__nv_bfloat16>::pack2(v[0], 0.0f));
#pragma unroll
            for (int t = 1; t + 1 < K; t += 2) sts32(addr(t + SH), Storage<__nv_bfloat16>::pack2(v[t], v[t + 1]));
            sts16(addr(K - 1 + SH), Storage<__nv_bfloat16>::pack2(v[K - 1], 0.0f));
        } else {
#pragma unroll
            for (int t = 0; t < K; t += 2) sts32(addr(t + SH), Storage<__nv_bfloat16>::pack2(v[t], v[t + 1]));
        }
    }
    __device__ static __forceinline__ void write(uint32_t sm, const uint32_t* off, uint32_t phi, const float* v) {
        switch (phi >> 1) {
            case 0: put<0>(sm, off, v); break;
            case 1: put<1>(sm, off, v); break;
            case 2: put<2>(sm, off, v); break;
            case 3: put<3>(sm, off, v); break;
            case 4: put<4>(sm, off, v); break;
            case 5: put<5>(sm, off, v); break;
            case 6: put<6>(sm, off, v); break;
            default: put<7>(sm, off, v); break;
        }
    }
    __device__ static __forceinline__ void read_signed(uint32_t sm, const uint32_t* off, uint32_t phi, float* v, uint32_t*) {
        read(sm, off, phi, v);
    }
    __device__ static __forceinline__ void write_signed(uint32_t sm, const uint32_t* off, uint32_t phi, const float* v,
                                                        const uint32_t*) {
        write(sm, off, phi, v);
    }
};

// ------------------------------------------------------------------------------------------
// mbarrier / TMA wrappers (raw PTX).
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
// Bounded wait: returns false when the limit ran out (the caller records an error and leaves).
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint32_t limit) {
#pragma unroll 1
    for (uint32_t i = 0; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
    }
    return false;
}
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Asynchronous 4-byte copy global -> shared (for rows that TMA cannot address), with its group bookkeeping.
__device__ __forceinline__ void cp_async4(uint32_t dst, const void* src) {
    HS_DBG_SMEM(dst, 4u, return);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
// ... and 16-byte copy (both addresses 16-byte aligned), past L1.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    HS_DBG_SMEM(dst, 16u, return);
    HS_DBG_CHECK((reinterpret_cast<uintptr_t>(src) & 15u) == 0, kDbgUnits, reinterpret_cast<uintptr_t>(src), return);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// One 2-D tiled TMA load (no multicast) of one box into shared memory.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const void* tmap, int32_t x, int32_t y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(tmap), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tma_store_2d(const void* tmap, int32_t x, int32_t y, uint32_t src) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];" ::"l"(tmap), "r"(x),
                 "r"(y), "r"(src)
                 : "memory");
}
// The same with three coordinates (x, y, z), for the view of a matrix as 128-byte lines of its rows.
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const void* tmap, int32_t x, int32_t y, int32_t z, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
        "l"(tmap), "r"(x), "r"(y), "r"(z), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tma_store_3d(const void* tmap, int32_t x, int32_t y, int32_t z, uint32_t src) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3}], [%4];" ::"l"(tmap), "r"(x),
                 "r"(y), "r"(z), "r"(src)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// ------------------------------------------------------------------------------------------
// One lane's run of K consecutive elements.
//
// Fast form (within the run the second scan is taken relative to the run start, Eq. 2 written
// for a part):  A_t = sum_{i<=t} log|a_i|,  u_t = log|b_t| - A_t,  r = max_t u_t (the
// log-sum-exp reference, Eq. 8),  s_t = sum_{i<=t} +-exp(u_i - r).  Then, for a value
// x_c = S_c exp(M_c) entering the run,
//     x_t = +-exp(A_t + M) * (S_c exp(M_c - M) + s_t exp(r - M)),   M = max(M_c, r),
// i.e. one exp per element for the scan, one log (log output) or one exp (linear output) per
// element for the result, and O(1) transcendental per run for the carry.
template <int MODE, typename TIn, typename TOut, int K>
struct Run {
    static constexpr bool SIGNED = (MODE != kLogUnsigned);
    using E = Elem<SIGNED>;
    static constexpr int IN_UNITS = K / Storage<TIn>::kPerUnit;    // 16-byte units per lane, input
    static constexpr int OUT_UNITS = K / Storage<TOut>::kPerUnit;  // 16-byte units per lane, output
    static constexpr int CHUNK = 32 * K;
    static constexpr int IN_BYTES = CHUNK * (int)sizeof(TIn);
    static constexpr int OUT_BYTES = CHUNK * (int)sizeof(TOut);

    float A[K];     // A_t (kLinear: in binary logarithms, log2 of the product of |a|)
    float s[K];     // s_t (before that: u_t)
    uint32_t P[K];  // parity mask of a_1..a_t (log modes with signs)
    float Pf[K];    // kLinear: the same parity as a factor, +1.0f or -1.0f (applied by a packed multiply)
    float r;        // reference of the run, -inf when the run has no non-zero b
    bool bad;       // the fast form does not apply to this run (a_t = 0, inf or NaN in it)

    // Load the lane's K inputs of both tensors from the swizzled chunk; `off` holds the lane's
    // IN_UNITS unit offsets (chunk_off), computed once per kernel.
    __device__ __forceinline__ static void load(uint32_t base_a, uint32_t base_b, const uint32_t* off, float* va,
                                                float* vb) {
#pragma unroll
        for (int j = 0; j < IN_UNITS; ++j) {
            Storage<TIn>::unpack(lds128(base_a + off[j]), va + j * Storage<TIn>::kPerUnit);
            Storage<TIn>::unpack(lds128(base_b + off[j]), vb + j * Storage<TIn>::kPerUnit);
        }
    }

    __device__ __forceinline__ static void load_a(uint32_t base_a, const uint32_t* off, float* va) {
#pragma unroll
        for (int j = 0; j < IN_UNITS; ++j) Storage<TIn>::unpack(lds128(base_a + off[j]), va + j * Storage<TIn>::kPerUnit);
    }
    // ... with the sign masks, for storage types that carry the sign in the element (sa, sb untouched otherwise)
    __device__ __forceinline__ static void load_signed(uint32_t base_a, uint32_t base_b, const uint32_t* off, float* va,
                                                       float* vb, uint32_t* sa, uint32_t* sb) {
        constexpr int PER = Storage<TIn>::kPerUnit;
#pragma unroll
        for (int j = 0; j < IN_UNITS; ++j) {
            Storage<TIn>::unpack_signed(lds128(base_a + off[j]), va + j * PER, sa + (Storage<TIn>::kCarriesSign ? j * PER : 0));
            Storage<TIn>::unpack_signed(lds128(base_b + off[j]), vb + j * PER, sb + (Storage<TIn>::kCarriesSign ? j * PER : 0));
        }
    }
    __device__ __forceinline__ static void load_a_signed(uint32_t base_a, const uint32_t* off, float* va, uint32_t* sa) {
        constexpr int PER = Storage<TIn>::kPerUnit;
#pragma unroll
        for (int j = 0; j < IN_UNITS; ++j)
            Storage<TIn>::unpack_signed(lds128(base_a + off[j]), va + j * PER, sa + (Storage<TIn>::kCarriesSign ? j * PER : 0));
    }

    // va, vb: the stored inputs (log a, log b for the log modes; a, b for kLinear).
    // sa, sb: per-element sign masks for kLogSigned (ignored otherwise).
    __device__ __forceinline__ E pass1(const float* va, const float* vb, const uint32_t* sa, const uint32_t* sb) {
        static_assert(K % 2 == 0, "runs are processed in pairs of elements");
        float acc = 0.0f;
        uint32_t par = 0u;
        float rr = neg_inf();
        if (MODE == kLinear) {
            // The reference of the run is taken from the largest |b_t| and the smallest A_t: it bounds
            // every u_t = log|b_t| - A_t from above, which is all a log-sum-exp reference has to do, and it
            // costs one logarithm per run instead of one per element; b_t itself enters the sum linearly.
            float bmax = 0.0f, amin = 0.0f, sgf = 1.0f;
#pragma unroll
            for (int t = 0; t < K; t += 2) {
                const float2 la = log2_abs_fast2(pk(va[t], va[t + 1]));  // A_t of this mode: binary logarithms
                sgf = flip(sgf, __float_as_uint(va[t]) & kSignBit);
                Pf[t] = sgf;
                sgf = flip(sgf, __float_as_uint(va[t + 1]) & kSignBit);
                Pf[t + 1] = sgf;
                acc += la.x;
                A[t] = acc;
                acc += la.y;
                A[t + 1] = acc;
                bmax = max3(bmax, fabsf(vb[t]), fabsf(vb[t + 1]));
                amin = min3(amin, A[t], A[t + 1]);
            }
            par = __float_as_uint(sgf) & kSignBit;
            // (2^-126 <= bmax keeps the scale factor below 2^127; smaller b_t are zero to ex2/lg2.approx.ftz anyway)
            rr = (bmax >= 1.17549435e-38f) ? (lg2(bmax) - amin) * kLn2 : neg_inf();
            bad = !(acc >= -1e30f) || !(bmax <= 3.0e38f) || !(amin >= -1e30f);
        } else {
#pragma unroll
            for (int t = 0; t < K; t += 2) {
                if (MODE == kLogSigned) {
                    par ^= sa[t];
                    P[t] = par;
                    par ^= sa[t + 1];
                    P[t + 1] = par;
                }
                acc += va[t];
                A[t] = acc;
                acc += va[t + 1];
                A[t + 1] = acc;
                const float2 u = fma2(pk(A[t], A[t + 1]), pk(-1.0f), pk(vb[t], vb[t + 1]));
                s[t] = u.x;
                s[t + 1] = u.y;
                rr = max3(rr, u.x, u.y);
            }
            bad = !(acc >= -1e30f) || !(rr <= 1e30f);
        }
        r = rr;
        const float ref = (rr == neg_inf()) ? 0.0f : rr;
        const float2 c = pk(-ref * kLog2e);
        float sum = 0.0f;
#pragma unroll
        for (int t = 0; t < K; t += 2) {
            float2 e;
            if (MODE == kLinear) {
                const float2 arg = fma2(pk(A[t], A[t + 1]), pk(-1.0f), c);  // <= 126: A_t >= amin, bmax >= 2^-126
                e = mul2(mul2(pk(vb[t], vb[t + 1]), pk(ex2(arg.x), ex2(arg.y))), pk(Pf[t], Pf[t + 1]));
            } else {
                const float2 arg = fma2(pk(s[t], s[t + 1]), pk(kLog2e), c);
                e = pk(ex2(arg.x), ex2(arg.y));
                if (MODE == kLogSigned) e = pk(flip(e.x, sb[t] ^ P[t]), flip(e.y, sb[t + 1] ^ P[t + 1]));
            }
            sum += e.x;
            s[t] = sum;
            sum += e.y;
            s[t + 1] = sum;
        }
        if (MODE == kLinear) acc *= kLn2;  // parts are composed in natural logarithms
        E agg;
        agg.A = acc;
        agg.m = fmaxf(rr + acc, kEmpty);
        agg.s = SIGNED ? flip(sum, par) : sum;  // beta = alpha * (sum relative to the run start)
        agg.p = par;
        return agg;
    }

    // Recompute A_t and the parity of a_1..a_t from the inputs (s_t and r come from elsewhere):
    // the look-back kernel parks only s_t between its two phases.
    __device__ __forceinline__ void rebuild(const float* va, const uint32_t* sa) {
        float acc = 0.0f;
        uint32_t par = 0u;
#pragma unroll
        for (int t = 0; t < K; ++t) {
            if (MODE == kLinear) {
                acc += log2_abs_fast(va[t]);
                par ^= __float_as_uint(va[t]) & kSignBit;
            } else {
                acc += va[t];
                if (MODE == kLogSigned) par ^= sa[t];
            }
            A[t] = acc;
            if (MODE == kLinear) Pf[t] = __uint_as_float(0x3f800000u | par);
            else if (SIGNED) P[t] = par;
        }
        bad = false;
    }

    // Apply the value entering the run and produce the outputs, in two steps so that a caller can store the
    // outputs piece by piece instead of holding all K of them:
    //   prepare() : the run's common factors, and whether the fast form can be trusted -- it cannot when an
    //               early prefix is too small relative to the run's reference (the caller then redoes the chunk
    //               with the tracked form);
    //   outputs() : elements T0 .. T0+N-1.  out_mag: log|x_t| (log modes) or x_t (kLinear); out_sign: sign
    //               masks (kLogSigned).
    struct Applied {
        float M, C, w;
        bool ok;
        float hM;  // (outputs<.., G = true> only) exp(M / 2), set by the caller
    };
    __device__ __forceinline__ Applied prepare(const E& entering) const {
        const float Mc = entering.m, Sc = entering.s;  // Mc is finite (>= kEmpty); r may be -inf
        Applied a;
        a.M = fmaxf(Mc, r);
        const float d = Mc - r;
        const float ed = ex2(-fabsf(d) * kLog2e);
        a.C = (d >= 0.0f) ? Sc : Sc * ed;
        a.w = (d >= 0.0f) ? ed : 1.0f;
        const float S1 = fmaf(s[0], a.w, a.C);
        a.ok = (fabsf(S1) >= 8.67361738e-19f /* 2^-60 */) || (Sc == 0.0f && r == neg_inf());
        a.hM = 0.0f;
        return a;
    }
    // G (kLinear, look-back kernel): A[t] holds g_t = +-exp(A_t / 2), the sign that of the product a_1..a_t, instead of
    // A_t, and x_t = (g_t h)|g_t h| S_t with h = exp(M / 2): no transcendental and no sign factor in this phase.
    template <int T0, int N, bool G = false>
    __device__ __forceinline__ void outputs(const Applied& a, float* out_mag, uint32_t* out_sign) const {
        static_assert(T0 % 2 == 0 && N % 2 == 0, "outputs are produced in pairs");
        const float2 w2 = pk(a.w), C2 = pk(a.C);
#pragma unroll
        for (int i = 0; i < N; i += 2) {
            const int t = T0 + i;
            const float2 S = fma2(pk(s[t], s[t + 1]), w2, C2);
            if (MODE == kLinear && G) {
                const float2 gh = mul2(pk(A[t], A[t + 1]), pk(a.hM));
                const float2 x = mul2(gh, S);
                out_mag[i] = x.x * fabsf(gh.x);
                out_mag[i + 1] = x.y * fabsf(gh.y);
            } else if (MODE == kLinear) {
                // exp(A_t + M) as the square of exp((A_t + M) / 2): the exponent range of fp32 twice over
                const float2 arg = fma2(pk(A[t], A[t + 1]), pk(0.5f), pk(a.M * (0.5f * kLog2e)));  // (A_t: binary logarithms)
                const float2 h = pk(ex2(arg.x), ex2(arg.y));
                const float2 x = mul2(mul2(mul2(S, h), h), pk(Pf[t], Pf[t + 1]));
                out_mag[i] = x.x;
                out_mag[i + 1] = x.y;
            } else {
                const float2 o = fma2(pk(lg2(fabsf(S.x)), lg2(fabsf(S.y))), pk(kLn2), add2(pk(A[t], A[t + 1]), pk(a.M)));
                out_mag[i] = o.x;
                out_mag[i + 1] = o.y;
                if (MODE == kLogSigned) {
                    const uint32_t sg0 = (__float_as_uint(S.x) ^ P[t]) & kSignBit;
                    const uint32_t sg1 = (__float_as_uint(S.y) ^ P[t + 1]) & kSignBit;
                    out_sign[i] = (S.x == 0.0f) ? 0u : sg0;
                    out_sign[i + 1] = (S.y == 0.0f) ? 0u : sg1;
                }
            }
        }
    }
    // all K at once
    __device__ __forceinline__ bool apply(const E& entering, float* out_mag, uint32_t* out_sign) const {
        const Applied a = prepare(entering);
        outputs<0, K>(a, out_mag, out_sign);
        return a.ok;
    }
};

// ------------------------------------------------------------------------------------------
// Tracked form, used for the rare chunk the fast form declines (a_t = 0 inside a run, or more
// than ~60 binary orders of magnitude between an early prefix and a later term of one run).
// Every step carries its own max reference; inputs are re-read from shared memory, so it needs
// no registers of the fast form.
template <int MODE, typename TIn>
struct Leaf {
    static constexpr bool SIGNED = (MODE != kLogUnsigned);
    // One element (stored values va, vb; sign masks sa, sb for kLogSigned) as a one-step part.
    __device__ static __forceinline__ Elem<SIGNED> get(float va, float vb, uint32_t sa, uint32_t sb) {
        Elem<SIGNED> e;
        float lb;
        uint32_t psb;
        if (MODE == kLinear) {
            e.A = log_abs_accurate(va);
            e.p = __float_as_uint(va) & kSignBit;
            lb = log_abs_accurate(vb);
            psb = __float_as_uint(vb) & kSignBit;
        } else {
            e.A = va;
            e.p = SIGNED ? sa : 0u;
            lb = vb;
            psb = SIGNED ? sb : 0u;
        }
        e.m = fmaxf(lb, kEmpty);
        e.s = (lb == neg_inf()) ? 0.0f : (SIGNED ? flip(1.0f, psb) : 1.0f);
        return e;
    }
};

}  // namespace hs
