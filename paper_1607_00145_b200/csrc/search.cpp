// Candidate plans and the performance model that ranks them (Sec. 3.3 and Sec. 3.4 of the paper,
// re-parameterised for B200).  Pure host code.
//
// The paper enumerates sub-tensor shapes / blocking sizes / GEMM variants, predicts each
// candidate's time as  Time_macro + Time_A + Time_B + Time_C  (Eq. 12-14) and compiles and times
// only the best few (Sec. 7.3: four timed candidates reach ~98 % of the best).  Here a
// candidate is one set of planner overrides (tile height and width, epilogue, loaders, operand
// exchange, atom order, split-K); the same four terms are estimated from the plan the planner
// builds for it:
//   Time_macro  slabs x (tile_m x tile_n x 64 x 2 flop) at the SM's tensor (or FMA) rate,
//   Time_A/B    the operand bytes a work item pulls out of L2 at the rate of its loader
//               (TMA boxes > 16-byte gathers > scalar gathers), overlapped with Time_macro,
//   Time_C      C's bytes (read too when beta != 0 is possible) at the HBM rate, derated when the
//               stores do not run along C's stride-1 mode,
// per wave of work items over the SMs (wave quantisation is what the paper's p_F fit
// conditions become on a GPU: a candidate pays for whole waves), plus fixed costs per work
// item, per launch and for the split-K reduction.
#include <algorithm>
#include <cmath>
#include <cstring>

#include "gett_plan.h"

namespace {

// B200 rates per SM and clock, from this project's own measurements (TFLOP/s and GB/s over 148
// SMs at ~1.75 GHz): tensor 1670 TFLOP/s, fp32 73.5 TFLOP/s, TMA ~94 GB/s per SM, 16-byte
// gathers ~60 GB/s per SM, HBM 6.5 TB/s.
constexpr double CLK_GHZ = 1.75;
constexpr double TENSOR_FLOP_PER_CLK = 1670e12 / 148 / (CLK_GHZ * 1e9);
constexpr double FMA_FLOP_PER_CLK = 73.5e12 / 148 / (CLK_GHZ * 1e9);
constexpr double TMA_B_PER_CLK = 94e9 / (CLK_GHZ * 1e9);
constexpr double GATHER_B_PER_CLK = 60e9 / (CLK_GHZ * 1e9);
constexpr double SCALAR_B_PER_CLK = 6e9 / (CLK_GHZ * 1e9);
constexpr double HBM_B_PER_CLK_PER_SM = 6.5e12 / 148 / (CLK_GHZ * 1e9);
constexpr double ITEM_OVERHEAD_CLK = 2500;  // tables, first copies, pipeline fill and drain of one work item
constexpr double LAUNCH_US = 3.0;

double loader_rate(int loader)
{
    switch (loader) {
    case GETT_LOAD_TMA_FREE:
    case GETT_LOAD_TMA_K: return TMA_B_PER_CLK;
    case GETT_LOAD_VEC_FREE:
    case GETT_LOAD_VEC_K: return GATHER_B_PER_CLK;
    case GETT_LOAD_VEC_KT: return GATHER_B_PER_CLK * 0.5; // isolated 16-byte pieces, transposed in place
    default: return SCALAR_B_PER_CLK;
    }
}

} // namespace

// Predicted time of `p` in microseconds; terms[0..3] = macro, A, B, C (microseconds, whole job).
double gett_planner_model(const gett_plan* p, int sm_count, double terms[4])
{
    const gett_plan_info_t& in = p->info;
    const double sms = sm_count > 0 ? sm_count : 148;
    const bool f32 = p->dtype == GETT_F32;
    const double es = f32 ? 4.0 : 2.0;
    // the kernels' view of the loaders and sizes (info is the caller's view)
    const int la = p->swapped ? in.loader_b : in.loader_a, lb = p->swapped ? in.loader_a : in.loader_b;
    const double M = p->M.size, N = p->N.size, K = p->K.size;
    const double tm = in.tile_m, tn = in.tile_n, tk = in.tile_k;
    const double items = (double)in.tiles * in.split_k;
    const double slabs = std::ceil(std::ceil(K / tk) / in.split_k);
    double ctas_per_sm = 1.0;
    if (in.path == GETT_PATH_FFMA)
        ctas_per_sm = p->skinny ? 2.0 : (in.tile_m == 64 ? 4.0 : 2.0);
    else if (in.path == GETT_PATH_SIMT)
        ctas_per_sm = 4.0;
    const double slots = sms * ctas_per_sm;
    // (stream-K: every SM gets the same share of the tiles x slabs space, no partial last wave)
    const double waves = p->stream_k ? items / slots : std::ceil(items / slots);
    // per slab of one work item, in clocks of the SM it shares with ctas_per_sm - 1 others
    const double rate = in.path == GETT_PATH_UMMA ? TENSOR_FLOP_PER_CLK
                        : in.path == GETT_PATH_FFMA ? FMA_FLOP_PER_CLK * 0.75 // (fragment loads share the issue slots)
                                                    : FMA_FLOP_PER_CLK * 0.12;
    const double macro_clk = 2.0 * tm * tn * tk / rate * ctas_per_sm;
    const double a_clk = tm * tk * es / loader_rate(in.path == GETT_PATH_SIMT ? GETT_LOAD_SCALAR : la) * ctas_per_sm;
    const double b_clk = (p->skinny ? 0.0 : tn * tk * es / loader_rate(in.path == GETT_PATH_SIMT ? GETT_LOAD_SCALAR : lb)) *
                         ctas_per_sm;
    // C: whole job at the HBM rate; direct stores that do not run along C's stride-1 mode waste sectors
    double c_bytes = M * N * 4.0 * 2.0; // written, and read when beta != 0 (the model does not know beta)
    double c_derate = 1.0;
    const bool rows_along_c = p->M.ndig >= 1 && p->M.sY[0] == 1;
    if (p->stream_k) {
        c_bytes += 2.0 * 4.0 * (double)p->sk_pmax * std::fmod(items, slots) * tm * tn; // the left-over tiles' pieces, out and back in
    } else if (in.split_k > 1) {
        c_bytes = M * N * 4.0 * (2.0 * in.split_k + 2.0); // partial sums out and back in, then C
    } else if (in.epilogue == GETT_EPI_STAGED) {
        c_derate = 0.8; // whole runs of C, through shared memory
    } else if (rows_along_c || (in.path == GETT_PATH_FFMA && p->c_vec != 0)) {
        c_derate = 1.0; // a warp's stores cover whole lines
    } else if (p->N.ndig >= 1 && p->N.sY[0] == 1) {
        c_derate = 0.5; // each thread writes a short run of its own row: whole sectors, one row per lane
    } else {
        c_derate = 0.25; // 4-byte stores scattered over sectors
    }
    const double c_clk_total = c_bytes / (HBM_B_PER_CLK_PER_SM * sms) / c_derate;
    // (the fixed cost of an item is hidden by the SM's other resident CTAs, if there are any: not scaled)
    const double per_item = slabs * std::max(macro_clk, a_clk + b_clk) + ITEM_OVERHEAD_CLK;
    const double main_clk = waves * per_item;
    // the C traffic overlaps the main loop of other items except in the last wave
    const double total_clk = std::max(main_clk, c_clk_total) + std::min(main_clk, c_clk_total) / std::max(1.0, waves);
    const double to_us = 1.0 / (CLK_GHZ * 1e3);
    if (terms) {
        terms[0] = waves * slabs * macro_clk * to_us;
        terms[1] = waves * slabs * a_clk * to_us;
        terms[2] = waves * slabs * b_clk * to_us;
        terms[3] = c_clk_total * to_us;
    }
    return total_clk * to_us + LAUNCH_US * (in.split_k > 1 ? 2.0 : 1.0);
}

// The candidate overrides for one contraction: every combination the planner can build on top of
// `base` (fields the caller fixed are kept), de-duplicated by what the planner makes of them.
std::vector<gett_plan_opts_t> gett_planner_candidates(const gett_tensor_desc_t* A, const gett_tensor_desc_t* B,
                                                     const gett_tensor_desc_t* C, gett_dtype_t dtype,
                                                     const gett_plan_opts_t& base, int sm_count)
{
    std::vector<gett_plan_opts_t> out;
    std::vector<gett_plan_info_t> seen;
    auto same = [](const gett_plan_info_t& x, const gett_plan_info_t& y) {
        return x.path == y.path && x.loader_a == y.loader_a && x.loader_b == y.loader_b && x.epilogue == y.epilogue &&
               x.tile_m == y.tile_m && x.tile_n == y.tile_n && x.stages == y.stages && x.split_k == y.split_k &&
               x.swapped == y.swapped && x.stream_k == y.stream_k && x.digits_m == y.digits_m && x.digits_n == y.digits_n && x.digits_k == y.digits_k;
    };
    auto consider = [&](gett_plan_opts_t o) {
        gett_plan tmp;
        tmp.ws = nullptr;
        tmp.status = nullptr;
        o.search = 0;
        if (gett_planner_build(&tmp, A, B, C, dtype, &o, sm_count) != GETT_OK)
            return;
        for (const gett_plan_info_t& s : seen)
            if (same(s, tmp.info))
                return;
        seen.push_back(tmp.info);
        out.push_back(o);
    };
    consider(base); // the rule-based plan is always a candidate (and the first one)
    const int tile_ms[] = {0, 64, 128, 256};
    const int tile_ns[] = {0, 32, 64, 128, 192, 256};
    const int epis[] = {GETT_EPI_AUTO, GETT_EPI_DIRECT};
    const int flagsets[] = {0, GETT_OPT_NO_ATOMS, GETT_OPT_NO_TMA, GETT_OPT_NO_EXCHANGE, GETT_OPT_STREAMK,
                            GETT_OPT_NO_STREAMK};
    const int splits[] = {0, 1, 2, 4, 8, 16, 32};
    for (int tmv : tile_ms)
        for (int tnv : tile_ns)
            for (int ep : epis)
                for (int fl : flagsets)
                    for (int sp : splits) {
                        gett_plan_opts_t o = base;
                        if (base.tile_m == 0)
                            o.tile_m = tmv;
                        else if (tmv)
                            continue;
                        if (base.tile_n == 0)
                            o.tile_n = tnv;
                        else if (tnv)
                            continue;
                        if (base.epilogue == GETT_EPI_AUTO)
                            o.epilogue = ep;
                        else if (ep)
                            continue;
                        if (fl & base.flags)
                            continue;
                        o.flags = base.flags | fl;
                        if (base.split_k == 0)
                            o.split_k = sp;
                        else if (sp)
                            continue;
                        consider(o);
                    }
    return out;
}
