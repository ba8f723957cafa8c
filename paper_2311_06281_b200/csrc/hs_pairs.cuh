// Linear-domain comparison path: the recurrence x_t = a_t x_{t-1} + b_t scanned directly as
// pairs (alpha, beta) meaning x -> alpha x + beta, with (alpha_2 alpha_1, alpha_2 beta_1 + beta_2)
// as the associative combine -- the general two-operator formulation the paper contrasts its
// log-space expression with (section "Compared to Blelloch's Formulation").  No logarithms and
// no exponentials: the prefix products and partial sums live in fp32's own range, so whatever
// leaves that range on the way (a product of many |a_t| > 1e38 or < 1e-45 inside one part) is
// lost, where the log-space kernels carry it.  Used by heinsen_scan_linear_pairs only; the
// chunk pipeline, the shared-memory layout and the batched kernel are the common ones.
#pragma once

namespace hs {

struct PairElem {
    float alpha;
    float beta;
};

// "first" is the older part: result = second o first.
__device__ __forceinline__ PairElem compose(const PairElem& first, const PairElem& second) {
    PairElem o;
    o.alpha = second.alpha * first.alpha;
    o.beta = fmaf(second.alpha, first.beta, second.beta);
    return o;
}
__device__ __forceinline__ void renormalise(PairElem&) {}

// Same lane layout and Kogge-Stone pattern as row_scan() of the log-space elements.
__device__ __forceinline__ void row_scan(const PairElem& mine, int lane, int R, PairElem& exclusive, PairElem& total) {
    PairElem inc = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        if (d >= R) {  // warp-uniform
            PairElem up;
            up.alpha = __shfl_up_sync(0xffffffffu, inc.alpha, d);
            up.beta = __shfl_up_sync(0xffffffffu, inc.beta, d);
            const PairElem c = compose(up, inc);
            if (lane >= d) inc = c;
        }
    }
    const int last = 32 - R + (lane & (R - 1));
    total.alpha = __shfl_sync(0xffffffffu, inc.alpha, last);
    total.beta = __shfl_sync(0xffffffffu, inc.beta, last);
    PairElem up;
    up.alpha = __shfl_up_sync(0xffffffffu, inc.alpha, R);
    up.beta = __shfl_up_sync(0xffffffffu, inc.beta, R);
    exclusive.alpha = (lane < R) ? 1.0f : up.alpha;
    exclusive.beta = (lane < R) ? 0.0f : up.beta;
}

// Chunk engine of the pair scan: same interface as the primary template, so that
// batched_scan_kernel<kPairs, ...> is the same kernel body.
template <typename TIn, typename TOut, int K>
struct ChunkEngine<kPairs, TIn, TOut, K> {
    using Base = ChunkEngine<kLinear, TIn, TOut, K>;  // staging helpers only (neutral padding a = 1, b = 0)
    using E = PairElem;
    static constexpr int IN_UNITS = Base::IN_UNITS;
    static constexpr int OUT_UNITS = Base::OUT_UNITS;
    using Offsets = typename Base::Offsets;
    __device__ static __forceinline__ Offsets offsets(const LaneMap& lm) { return Base::offsets(lm); }

    struct Pending {
        float P[K];  // prefix products of the lane's run
        float B[K];  // the run's recurrence started from 0
        E excl;
    };

    using Wide = typename Base::Wide;
    static constexpr int WIDE_PAD = Base::WIDE_PAD;
    __device__ static __forceinline__ Wide wide_of(const Params& p, long long row, bool on) { return Base::wide_of(p, row, on); }
    __device__ static __forceinline__ void wide_load_async(const Params& p, uint32_t sm_a, uint32_t sm_b, int lane, long long row,
                                                           long long colbase, int W) {
        Base::wide_load_async(p, sm_a, sm_b, lane, row, colbase, W);
    }
    __device__ static __forceinline__ void wide_store(const Params& p, uint32_t sm_out, int lane, long long row, long long colbase,
                                                      int W) {
        Base::wide_store(p, sm_out, lane, row, colbase, W);
    }

    template <bool PLAIN>
    __device__ static __forceinline__ void phase1(const Params& p, uint32_t sm_a, uint32_t sm_b, const Offsets& off,
                                                  const LaneMap&, int lane, long long row, long long col0, bool ragged,
                                                  const Wide& wd, Pending& pd, E& total) {
        float va[K], vb[K];
        uint32_t none[1];
        Base::template read_inputs<PLAIN>(sm_a, sm_b, off, wd, va, vb, none, none);
        if (ragged) {
            const long long left = (row < p.rows) ? p.n - col0 : 0;
#pragma unroll
            for (int t = 0; t < K; ++t) {
                if (t >= left) { va[t] = 1.0f; vb[t] = 0.0f; }
            }
        }
        float prod = 1.0f, acc = 0.0f;
#pragma unroll
        for (int t = 0; t < K; ++t) {
            prod *= va[t];
            acc = fmaf(va[t], acc, vb[t]);
            pd.P[t] = prod;
            pd.B[t] = acc;
        }
        E agg;
        agg.alpha = prod;
        agg.beta = acc;
        row_scan(agg, lane, p.rows_per_warp, pd.excl, total);
    }

    template <bool PLAIN>
    __device__ static __forceinline__ void phase2(const Params&, uint32_t, uint32_t, uint32_t sm_out, const Offsets& off,
                                                  const LaneMap&, long long, long long, const Wide& wd, const Pending& pd,
                                                  const E& entering_row) {
        const float x_in = fmaf(pd.excl.alpha, entering_row.beta, pd.excl.beta);
        float out[K];
#pragma unroll
        for (int t = 0; t < K; ++t) out[t] = fmaf(pd.P[t], x_in, pd.B[t]);
        const uint32_t none[1] = {0u};
        Base::template write_outputs<PLAIN>(sm_out, off, wd, out, none);
    }

    struct RawX0 { float v; };
    __device__ static __forceinline__ RawX0 load_x0(const Params& p, long long row) {
        RawX0 r;
        r.v = (row < p.rows) ? Storage<TIn>::load(p.x0, row) : 0.0f;
        return r;
    }
    // the value of x as a part: alpha = 0 forgets whatever came before
    __device__ static __forceinline__ E x0_elem(const RawX0& r) {
        E e;
        e.alpha = 0.0f;
        e.beta = r.v;
        return e;
    }
    __device__ static __forceinline__ E row_start(const Params& p, long long row) { return x0_elem(load_x0(p, row)); }

    __device__ static __forceinline__ void generic_load(const Params& p, uint32_t sm_a, uint32_t sm_b, const LaneMap& lm,
                                                        int lane, long long row0, long long colbase) {
        Base::generic_load(p, sm_a, sm_b, lm, lane, row0, colbase);
    }
    __device__ static __forceinline__ void generic_store(const Params& p, uint32_t sm_out, const LaneMap& lm, int lane,
                                                         long long row0, long long colbase) {
        Base::generic_store(p, sm_out, lm, lane, row0, colbase);
    }
    static constexpr bool ASYNC_PLAIN = Base::ASYNC_PLAIN;
    __device__ static __forceinline__ void generic_load_async(const Params& p, uint32_t sm_a, uint32_t sm_b,
                                                              const LaneMap& lm, int lane, long long row0, long long colbase) {
        Base::generic_load_async(p, sm_a, sm_b, lm, lane, row0, colbase);
    }
    static constexpr int IN_LINE = Base::IN_LINE, OUT_LINE = Base::OUT_LINE;
    __device__ static __forceinline__ void tail_load(const Params& p, uint32_t sm_a, uint32_t sm_b, int lane, long long row,
                                                     int colbase) {
        Base::tail_load(p, sm_a, sm_b, lane, row, colbase);
    }
    __device__ static __forceinline__ void tail_store(const Params& p, uint32_t sm_out, int lane, long long row, int colbase) {
        Base::tail_store(p, sm_out, lane, row, colbase);
    }
};

}  // namespace hs
