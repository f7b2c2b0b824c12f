// Host planner: from three tensor descriptors to index sets, fused dimensions,
// tile order, kernel path and blocking.  Pure host C++ (no CUDA calls), so it can
// be exercised on a machine without a GPU.
//
// Steps and where the paper describes them:
//   classify labels into I_m / I_n / I_k ............ Sec. 2.2
//   merge adjacent modes into super-indices .......... Sec. 6 (stage 1)
//   choose the sub-tensor that forms a tile, keeping
//   the stride-1 mode of each tensor inside it ....... Sec. 3.2.1
//   split a mode by factors of its extent ............ Sec. 3.2.1, Examples 1-2
//   blocking sizes, GEMM variant (here: split-K) ..... Sec. 3.3
#include <algorithm>
#include <cstring>
#include <map>

#include "gett_plan.h"

// Longest contraction (fused K) for which a C that runs along A's stride-1 mode is moved to the
// column side by exchanging the operands: beyond it the element-wise update of C hides behind the
// next tile's main loop and the direct stores keep the whole operand ring.
#ifndef GETT_EXCHANGE_MAX_K
#define GETT_EXCHANGE_MAX_K 256
#endif

namespace {

struct RawTensor {
    int n;
    int64_t ext[GETT_MAX_MODES], stride[GETT_MAX_MODES];
    int32_t label[GETT_MAX_MODES];
    int find(int32_t l) const
    {
        for (int i = 0; i < n; ++i)
            if (label[i] == l)
                return i;
        return -1;
    }
};

gett_status_t read_desc(const gett_tensor_desc_t* d, RawTensor& t)
{
    if (!d || d->nmodes < 0 || d->nmodes > GETT_MAX_MODES)
        return GETT_ERR_INVALID_ARG;
    if (d->nmodes > 0 && (!d->extent || !d->label))
        return GETT_ERR_INVALID_ARG;
    t.n = d->nmodes;
    int64_t packed = 1;
    for (int i = 0; i < t.n; ++i) {
        t.ext[i] = d->extent[i];
        t.label[i] = d->label[i];
        if (t.ext[i] < 1 || t.ext[i] >= (1ll << 31))
            return GETT_ERR_INVALID_ARG;
        t.stride[i] = d->stride ? d->stride[i] : packed;
        if (t.stride[i] < 1 || t.stride[i] >= (1ll << 46))
            return GETT_ERR_INVALID_ARG;
        packed *= t.ext[i];
        if (packed >= (1ll << 46))
            return GETT_ERR_UNSUPPORTED;
        for (int j = 0; j < i; ++j)
            if (t.label[j] == t.label[i])
                return GETT_ERR_BAD_LABELS;
    }
    return GETT_OK;
}

// C must address every element once: sorted by stride, each mode must step over
// the whole extent of the previous one.
bool c_overlaps(const RawTensor& c)
{
    std::vector<std::pair<int64_t, int64_t>> v; // (stride, extent)
    for (int i = 0; i < c.n; ++i)
        if (c.ext[i] > 1)
            v.push_back({c.stride[i], c.ext[i]});
    std::sort(v.begin(), v.end());
    for (size_t i = 1; i < v.size(); ++i)
        if (v[i].first < v[i - 1].first * v[i - 1].second)
            return true;
    return false;
}

// Tile order of one set: `lead` (index into modes, or -1) first, the rest in
// canonical order.  Each mode is one digit (no split).
std::vector<GettDigit> order_with_lead(const std::vector<GettMode>& modes, int lead)
{
    std::vector<GettDigit> out;
    if (lead >= 0)
        out.push_back({lead, modes[lead].ext, 1});
    for (int i = 0; i < (int)modes.size(); ++i)
        if (i != lead)
            out.push_back({i, modes[i].ext, 1});
    return out;
}

// Build the kernel-side dimension: one entry per digit, merging a digit into its
// predecessor when it continues it contiguously in both carrier tensors (unless `merge`
// is off).  With seg1 >= 0 the digit list is [segment 0 | segment 1 | high part]: `seg1`
// and `hi` are the positions in `digits` where segment 1 and the high part start (see
// gett_dims.h); digits never merge across these positions.  `src`, if given, receives for
// every kernel-side digit the position in `digits` it came from (meaningful without merging).
gett_status_t make_dim(const std::vector<GettMode>& modes, const std::vector<GettDigit>& digits,
                       int carrierX, int carrierY, GettDim& D, int seg1 = -1, int hi = -1, bool merge = true,
                       std::vector<int>* src = nullptr)
{
    auto stride_of = [](const GettMode& m, int which) {
        return which == 0 ? m.sA : which == 1 ? m.sB : m.sC;
    };
    memset(&D, 0, sizeof D);
    struct E {
        int64_t ext, sx, sy;
        int from;
    };
    const int n = (int)digits.size();
    const bool two = seg1 >= 0;
    if (two && !(0 < seg1 && seg1 < hi && hi <= n))
        return GETT_ERR_INVALID_ARG;
    std::vector<E> e;
    int64_t part_size[3] = {1, 1, 1}; // segment 0, segment 1, high part (plain dimension: all in [0])
    int part_first_dig[3] = {0, 0, 0};
    int64_t bx = 0, by = 0;
    size_t first = 0; // entries of `e` that belong to the part being built
    for (int i = 0; i < n; ++i) {
        const int part = !two ? 0 : i < seg1 ? 0 : i < hi ? 1 : 2;
        if (two && (i == seg1 || i == hi)) {
            part_first_dig[part] = (int)e.size();
            first = e.size();
        }
        const GettDigit& g = digits[i];
        const GettMode& m = modes[g.mode];
        E cur{g.ext, stride_of(m, carrierX) * g.mult, stride_of(m, carrierY) * g.mult, i};
        if (g.off != 0) {
            if (part != 1)
                return GETT_ERR_INVALID_ARG; // only segment 1 starts inside a mode
            bx += stride_of(m, carrierX) * g.off;
            by += stride_of(m, carrierY) * g.off;
        }
        if (cur.ext == 1)
            continue;
        part_size[part] *= cur.ext;
        if (part_size[part] >= (1ll << 31))
            return GETT_ERR_UNSUPPORTED;
        if (merge && e.size() > first && cur.sx == e.back().sx * e.back().ext &&
            cur.sy == e.back().sy * e.back().ext && e.back().ext * cur.ext < (1ll << 31))
            e.back().ext *= cur.ext;
        else
            e.push_back(cur);
    }
    if (two && hi == n)
        part_first_dig[2] = (int)e.size();
    const int64_t total = two ? (part_size[0] + part_size[1]) * part_size[2] : part_size[0];
    if ((int)e.size() > GETT_MAX_DIGITS || total >= (1ll << 31))
        return GETT_ERR_UNSUPPORTED;
    D.ndig = (int)e.size();
    if (src)
        src->clear();
    for (int d = 0; d < D.ndig; ++d) {
        D.ext[d] = (uint32_t)e[d].ext;
        gett_magic(D.ext[d], D.mul[d], D.sh[d]);
        D.sX[d] = e[d].sx;
        D.sY[d] = e[d].sy;
        if (src)
            src->push_back(e[d].from);
    }
    D.size = (uint32_t)total;
    D.seg1_dig = D.hi_dig = D.ndig;
    D.seg1_start = D.period = D.size;
    if (two) {
        if (part_first_dig[1] == 0 || part_first_dig[1] >= part_first_dig[2])
            return GETT_ERR_UNSUPPORTED; // both segments must have digits
        D.seg1_dig = part_first_dig[1];
        D.hi_dig = part_first_dig[2];
        D.seg1_start = (uint32_t)part_size[0];
        D.period = (uint32_t)(part_size[0] + part_size[1]);
        gett_magic(D.period, D.period_mul, D.period_sh);
        D.seg1_bX = bx;
        D.seg1_bY = by;
    }
    return GETT_OK;
}

int merged_count(const std::vector<GettMode>& modes, int cx, int cy)
{
    std::vector<GettDigit> canon;
    for (int i = 0; i < (int)modes.size(); ++i)
        canon.push_back({i, modes[i].ext, 1});
    GettDim D;
    if (make_dim(modes, canon, cx, cy, D) != GETT_OK)
        return (int)modes.size();
    return D.ndig;
}

int find_unit(const std::vector<GettMode>& modes, int which)
{
    for (int i = 0; i < (int)modes.size(); ++i) {
        int64_t s = which == 0 ? modes[i].sA : which == 1 ? modes[i].sB : modes[i].sC;
        if (s == 1)
            return i;
    }
    return -1;
}

int64_t min_stride(const std::vector<GettMode>& modes, int which)
{
    int64_t best = INT64_MAX;
    for (const GettMode& m : modes) {
        int64_t s = which == 0 ? m.sA : which == 1 ? m.sB : m.sC;
        best = std::min(best, s);
    }
    return best;
}

uint32_t ceil_div(uint32_t a, uint32_t b) { return (a + b - 1) / b; }

// Tensor-map recipe for one operand of the tensor-core kernel, if its tile (rows free
// indices x 64 k) is a box: the tile must stay inside digit 0 of the free dimension and
// of K (one digit only, or a digit-0 extent that the tile size divides), and the free and
// K digits together must fit the five dimensions a tensor map has.
void make_tma_recipe(const GettDim& F, bool fX, const GettDim& Kd, bool kX, int loader, uint32_t rows,
                     GettTmaRecipe& R)
{
    memset(&R, 0, sizeof R);
    if (loader != GETT_LOAD_VEC_FREE && loader != GETT_LOAD_VEC_K)
        return;
    if (F.ndig < 1 || Kd.ndig < 1 || F.ndig + Kd.ndig > 5)
        return;
    if (F.seg1_dig < F.hi_dig || Kd.seg1_dig < Kd.hi_dig)
        return;
    if (F.ndig > 1 && F.ext[0] % rows != 0)
        return;
    if (Kd.ndig > 1 && Kd.ext[0] % 64 != 0)
        return;
    const int64_t* fs = fX ? F.sX : F.sY;
    const int64_t* ks = kX ? Kd.sX : Kd.sY;
    for (int d = 0; d < GETT_MAX_DIGITS; ++d)
        R.co.fdim[d] = R.co.kdim[d] = -1;
    int n = 0;
    auto push = [&](int which, int d) {
        const GettDim& D = which ? Kd : F;
        R.dims[n] = D.ext[d];
        R.strides[n] = (uint64_t)(which ? ks[d] : fs[d]);
        (which ? R.co.kdim : R.co.fdim)[d] = (int8_t)n;
        (which ? R.co.kmul : R.co.fmul)[d] = 1;
        R.box[n] = 1;
        ++n;
    };
    const bool free_inner = loader == GETT_LOAD_VEC_FREE;
    push(free_inner ? 0 : 1, 0);
    push(free_inner ? 1 : 0, 0);
    for (int d = 1; d < F.ndig; ++d)
        push(0, d);
    for (int d = 1; d < Kd.ndig; ++d)
        push(1, d);
    R.co.rank = n;
    R.box[0] = 64;                      // 128 bytes = the swizzle span
    R.box[1] = free_inner ? 64 : rows;  // MN-major: 64 k rows per box; K-major: all rows in one box
    if (R.strides[0] != 1)
        return;
    for (int i = 1; i < n; ++i)
        if (R.strides[i] % 8 != 0 || R.strides[i] >= (1ull << 38))
            return;
    R.enabled = 1;
}

// ---- tiles of 64-wide atoms for operands whose stride-1 mode is a free mode (Sec. 3.2.1) ----
//
// Such an operand is staged as rows of 64 consecutive free indices per k.  A TMA box can fill
// one "atom" (64 free indices x 64 k) when its 64 indices are consecutive indices of the
// lead (stride-1) mode.  With that mode's extent e = 64 q + r:
//   r == 0            every atom is such a run;
//   r in {16, 32}     the first 64 q indices of every run of the lead mode form such atoms
//                     (segment 0), the remaining r are combined with 64 / r consecutive
//                     indices of a second free mode (the partner) into atoms of r x 64/r
//                     (segment 1) -- the paper's sub-tensor made of pieces of two modes, used
//                     for the remainder only, so that most of the data still moves in 128-byte
//                     rows.  Those atoms are not boxes with a 128-byte inner extent and are
//                     gathered with 16-byte copies.
// The two kinds alternate with period e * 64/r (64/r runs of the lead mode), so every tile
// holds both in the same proportion.
struct SideOrder {
    bool ok = false;
    std::vector<GettDigit> digits; // [segment 0 | segment 1 | high part] or a plain order
    int seg1 = -1, hi = -1;
    int lead = -1;
};

SideOrder atom_order(const std::vector<GettMode>& modes, const std::vector<GettDigit>& cur, int carrier)
{
    SideOrder S;
    if (cur.empty())
        return S;
    for (const GettDigit& g : cur)
        if (g.mult != 1 || g.off != 0 || g.ext != modes[g.mode].ext)
            return S; // already split for another purpose
    auto stride_of = [&](int m) { return carrier == 0 ? modes[m].sA : modes[m].sB; };
    S.lead = cur[0].mode;
    const int64_t e = modes[S.lead].ext;
    if (stride_of(S.lead) != 1 || e % 8 != 0)
        return S;
    if (e % 64 == 0) {
        S.digits = cur;
        S.ok = true;
        return S;
    }
    const int64_t q = e / 64, r = e % 64;
    // (r == 8: the remainder would be gathered in isolated 16-byte pieces, one memory request
    //  each -- measured slower than gathering the whole operand, whose copies follow the runs)
    if (q == 0 || 64 % r != 0 || r < 16)
        return S;
    const int64_t need = 64 / r;
    int partner = -1;
    for (size_t i = 1; i < cur.size() && partner < 0; ++i)
        if (modes[cur[i].mode].ext % need == 0)
            partner = cur[i].mode;
    if (partner < 0)
        return S;
    S.digits.push_back({S.lead, 64 * q, 1, 0});
    S.digits.push_back({partner, need, 1, 0});
    S.seg1 = (int)S.digits.size();
    S.digits.push_back({S.lead, r, 1, 64 * q});
    S.digits.push_back({partner, need, 1, 0});
    S.hi = (int)S.digits.size();
    S.digits.push_back({partner, modes[partner].ext / need, need, 0});
    for (size_t i = 1; i < cur.size(); ++i)
        if (cur[i].mode != partner)
            S.digits.push_back(cur[i]);
    S.ok = true;
    return S;
}

// Order of I_k in which every slab of 64 contracted indices is a box of the modes: a mode
// whose extent is a multiple of 64 first, or a p-wide piece (p a power of two) of one mode
// times 64 / p consecutive indices of a second one (Sec. 3.2.1, the sub-tensor k_C = 64 made
// of pieces of two modes).  box_u x box_v is the slab's shape on the first two modes of the
// order (box_v == 0: the slab lies in the first mode alone).
struct KOrder {
    bool ok = false;
    std::vector<GettDigit> digits;
    int u = -1, v = -1;
    int64_t box_u = 64, box_v = 0;
};

KOrder slab_order(const std::vector<GettMode>& modes, const std::vector<GettDigit>& cur)
{
    KOrder K;
    if (cur.empty())
        return K;
    for (const GettDigit& g : cur)
        if (g.mult != 1 || g.off != 0 || g.ext != modes[g.mode].ext)
            return K;
    auto rest = [&](int skip1, int skip2) {
        for (const GettDigit& g : cur)
            if (g.mode != skip1 && g.mode != skip2)
                K.digits.push_back(g);
    };
    if (cur.size() == 1) {
        K.digits = cur;
        K.u = cur[0].mode;
        K.ok = true;
        return K;
    }
    for (const GettDigit& g : cur)
        if (g.ext % 64 == 0) {
            K.u = g.mode;
            K.digits.push_back(g);
            rest(g.mode, -1);
            K.ok = true;
            return K;
        }
    int64_t best_p = 0;
    for (const GettDigit& gu : cur) {
        int64_t p = 1;
        while (p < 32 && gu.ext % (2 * p) == 0)
            p *= 2;
        if (p < 2 || p <= best_p)
            continue;
        for (const GettDigit& gv : cur)
            if (gv.mode != gu.mode && gv.ext % (64 / p) == 0) {
                best_p = p;
                K.u = gu.mode;
                K.v = gv.mode;
                break;
            }
    }
    if (best_p == 0)
        return K;
    K.box_u = best_p;
    K.box_v = 64 / best_p;
    K.digits.push_back({K.u, best_p, 1, 0});
    K.digits.push_back({K.v, modes[K.v].ext, 1, 0});
    K.digits.push_back({K.u, modes[K.u].ext / best_p, best_p, 0});
    rest(K.u, K.v);
    K.ok = true;
    return K;
}

// Tensor map of an operand fetched atom by atom (the atoms of segment 0; segment 1, if there
// is one, is gathered).  Map dimensions: the lead mode, the other free modes, then the modes
// of I_k in slab order.  `fsrc` / `ksrc` give, for each digit of the kernel-side dimensions,
// its position in S.digits / K.digits.
bool make_atom_recipe(const std::vector<GettMode>& fmodes, const SideOrder& S, const std::vector<int>& fsrc,
                      const GettDim& F, const std::vector<GettMode>& kmodes, const KOrder& K,
                      const std::vector<int>& ksrc, int carrier, GettTmaRecipe& R)
{
    memset(&R, 0, sizeof R);
    for (int d = 0; d < GETT_MAX_DIGITS; ++d)
        R.co.fdim[d] = R.co.kdim[d] = -1;
    auto stride_of = [&](const GettMode& m) { return carrier == 0 ? m.sA : m.sB; };
    std::vector<int> fdim_of(fmodes.size(), -1), kdim_of(kmodes.size(), -1);
    int n = 0;
    auto add = [&](const GettMode& m, int& slot) {
        if (slot >= 0)
            return true;
        if (n >= 5)
            return false;
        slot = n;
        R.dims[n] = (uint64_t)m.ext;
        R.strides[n] = (uint64_t)stride_of(m);
        R.box[n] = 1;
        ++n;
        return true;
    };
    if (!add(fmodes[S.lead], fdim_of[S.lead]))
        return false;
    for (const GettDigit& g : S.digits)
        if (!add(fmodes[g.mode], fdim_of[g.mode]))
            return false;
    for (const GettDigit& g : K.digits)
        if (!add(kmodes[g.mode], kdim_of[g.mode]))
            return false;
    R.co.rank = n;
    if (n < 2) // (a tensor map needs a second dimension; such a case keeps the gather)
        return false;
    if (R.strides[0] != 1)
        return false;
    for (int i = 1; i < n; ++i)
        if (R.strides[i] % 8 != 0 || R.strides[i] >= (1ull << 38))
            return false;
    R.box[fdim_of[S.lead]] = 64;
    R.box[kdim_of[K.u]] = (uint32_t)K.box_u;
    if (K.box_v)
        R.box[kdim_of[K.v]] = (uint32_t)K.box_v;
    // coordinates: the digits of segment 0 and of the high part (segment 1 is not fetched by TMA)
    for (size_t d = 0; d < fsrc.size(); ++d) {
        if ((int)d >= F.seg1_dig && (int)d < F.hi_dig)
            continue;
        const GettDigit& g = S.digits[fsrc[d]];
        R.co.fdim[d] = (int8_t)fdim_of[g.mode];
        R.co.fmul[d] = (int32_t)g.mult;
    }
    for (size_t d = 0; d < ksrc.size(); ++d) {
        const GettDigit& g = K.digits[ksrc[d]];
        R.co.kdim[d] = (int8_t)kdim_of[g.mode];
        R.co.kmul[d] = (int32_t)g.mult;
    }
    R.hybrid = S.seg1 >= 0 ? 1 : 0;
    R.enabled = 1;
    return true;
}

// 16-byte vectors of `vec` elements along the first digit of `lead` are legal for
// carrier X when that digit is stride-1, its extent is a multiple of vec, and every
// other stride of the tensor (remaining digits of `lead`, all digits of `other`)
// is a multiple of vec, so that every vector starts on a 16-byte boundary.
bool vec_ok(const GettDim& lead, bool leadIsX, const GettDim& other, bool otherIsX, uint32_t vec)
{
    if (lead.ndig < 1)
        return false;
    const int64_t* ls = leadIsX ? lead.sX : lead.sY;
    const int64_t* os = otherIsX ? other.sX : other.sY;
    if (ls[0] != 1 || lead.ext[0] % vec != 0)
        return false;
    for (int d = 1; d < lead.ndig; ++d)
        if (ls[d] % vec != 0)
            return false;
    for (int d = 0; d < other.ndig; ++d)
        if (os[d] % vec != 0)
            return false;
    return true;
}

} // namespace

gett_status_t gett_planner_build(gett_plan* p, const gett_tensor_desc_t* dA,
                                 const gett_tensor_desc_t* dB, const gett_tensor_desc_t* dC,
                                 gett_dtype_t dtype, const gett_plan_opts_t* opts, int sm_count)
{
    RawTensor A, B, C;
    gett_status_t rc;
    if ((rc = read_desc(dA, A)) || (rc = read_desc(dB, B)) || (rc = read_desc(dC, C)))
        return rc;
    if (dtype != GETT_F32 && dtype != GETT_BF16_F32 && dtype != GETT_F16_F32 && dtype != GETT_F64)
        return GETT_ERR_UNSUPPORTED;
    gett_plan_opts_t o;
    memset(&o, 0, sizeof o);
    if (opts)
        o = *opts;

    // ---- classification (Sec. 2.2) ----
    std::vector<GettMode> im, in, ik;
    for (int i = 0; i < C.n; ++i) {
        int ia = A.find(C.label[i]), ib = B.find(C.label[i]);
        if ((ia >= 0) == (ib >= 0))
            return GETT_ERR_BAD_LABELS; // in all three tensors, or only in C
        int64_t e = ia >= 0 ? A.ext[ia] : B.ext[ib];
        if (e != C.ext[i])
            return GETT_ERR_EXTENT_MISMATCH;
        GettMode m{C.label[i], e, ia >= 0 ? A.stride[ia] : 0, ib >= 0 ? B.stride[ib] : 0,
                   C.stride[i]};
        if (e > 1)
            (ia >= 0 ? im : in).push_back(m);
    }
    for (int i = 0; i < A.n; ++i) {
        if (C.find(A.label[i]) >= 0)
            continue;
        int ib = B.find(A.label[i]);
        if (ib < 0)
            return GETT_ERR_BAD_LABELS; // only in A
        if (A.ext[i] != B.ext[ib])
            return GETT_ERR_EXTENT_MISMATCH;
        if (A.ext[i] > 1)
            ik.push_back({A.label[i], A.ext[i], A.stride[i], B.stride[ib], 0});
    }
    for (int i = 0; i < B.n; ++i)
        if (C.find(B.label[i]) < 0 && A.find(B.label[i]) < 0)
            return GETT_ERR_BAD_LABELS; // only in B
    if (c_overlaps(C))
        return GETT_ERR_INVALID_ARG;

    // ---- canonical order: I_m, I_n by stride in C; I_k by stride in A ----
    auto byC = [](const GettMode& a, const GettMode& b) { return a.sC < b.sC; };
    auto byA = [](const GettMode& a, const GettMode& b) { return a.sA < b.sA; };
    std::stable_sort(im.begin(), im.end(), byC);
    std::stable_sort(in.begin(), in.end(), byC);
    std::stable_sort(ik.begin(), ik.end(), byA);
    p->dtype = dtype;

    // ---- which operand gives the kernel its rows ----
    // The kernels unpack along their columns (the N-side split below, the staged epilogues).
    // If C's stride-1 mode belongs to A but is not A's own stride-1 mode, exchange the roles of
    // A and B (C = A B is also C = B A with rows and columns exchanged): that mode becomes a
    // column mode, and A's stride-1 mode can be split around it.  The lists keep their order;
    // only the carriers change places.
    p->swapped = 0;
    {
        const int unitCm = find_unit(im, 2), unitAm = find_unit(im, 0);
        const int64_t vec = dtype == GETT_F32 ? 4 : 8;
        // (fp32 with small N and K keeps A on the row side: the small-N kernel streams it, and the
        //  same split is applied to I_m below)
        int64_t nsz = 1, ksz = 1;
        for (const GettMode& m : in)
            nsz *= m.ext;
        for (const GettMode& m : ik)
            ksz *= m.ext;
        const bool small_nk = dtype == GETT_F32 && nsz <= 64 && ksz <= gett_ffma_skinny_max_k();
        bool want = dtype != GETT_F64 && !small_nk && unitCm >= 0 && unitAm >= 0 && unitCm != unitAm && im[unitAm].ext % vec == 0 &&
                    im[unitAm].ext > vec && im[unitCm].ext % 4 == 0 && o.epilogue != GETT_EPI_DIRECT &&
                    !(o.flags & GETT_OPT_NO_EXCHANGE);
        if (want && dtype == GETT_F32) { // the same alignment the fp32 split asks for
            for (const GettMode& m : in)
                want = want && m.sC % 4 == 0;
            for (int i = 0; i < (int)im.size(); ++i)
                want = want && (i == unitCm || im[i].sC % 4 == 0);
        }
        // 16-bit types, short contraction, C's stride-1 mode is A's own: the kernel's rows would
        // run along C and each thread would update its row of C element by element, with
        // nothing to hide that behind.  With the roles exchanged the mode leads the columns
        // and C goes through the staged unpacking (whole 16-byte vectors, old values fetched
        // ahead of the accumulator).
        // (the same when A's stride-1 mode is a contracted one: I_m is then ordered for C anyway)
        if (!want && (dtype == GETT_BF16_F32 || dtype == GETT_F16_F32) && unitCm >= 0 &&
            (unitAm == unitCm || unitAm < 0) &&
            ksz <= GETT_EXCHANGE_MAX_K && im[unitCm].ext % 8 == 0 && o.epilogue != GETT_EPI_DIRECT &&
            o.tile_m != 256 && !(o.flags & GETT_OPT_NO_EXCHANGE)) { // (256-row tiles store directly)
            want = true;
            for (const GettMode& m : in)
                want = want && m.sC % 4 == 0;
            for (int i = 0; i < (int)im.size(); ++i)
                want = want && (i == unitCm || im[i].sC % 4 == 0);
        }
        if (want) {
            std::swap(im, in);
            for (std::vector<GettMode>* v : {&im, &in, &ik})
                for (GettMode& m : *v)
                    std::swap(m.sA, m.sB);
            p->swapped = 1;
        }
    }
    p->im = im;
    p->in = in;
    p->ik = ik;

    // ---- tile order: keep each operand's stride-1 mode first in its set (Sec. 3.2.1) ----
    int leadM = find_unit(im, 0); // A's stride-1 mode, if it is free
    int leadN = find_unit(in, 1); // B's stride-1 mode, if it is free
    int leadK = find_unit(ik, 0); // A's stride-1 mode, if it is contracted ...
    if (leadK < 0)
        leadK = find_unit(ik, 1); // ... else B's
    // Sec. 3.2.1 applied to I_n: B's stride-1 mode and C's stride-1 mode are two different
    // modes of I_n, and B's can be split into pieces of one 16-byte vector (vecB elements).
    auto n_split_ok = [&](int64_t vecB) {
        const int unitCn = find_unit(in, 2);
        if (!(dtype != GETT_F64 && leadN >= 0 && unitCn >= 0 && unitCn != leadN && in[leadN].ext % vecB == 0 &&
              in[leadN].ext > vecB && o.epilogue != GETT_EPI_DIRECT))
            return false;
        if (dtype != GETT_F32)
            return true;
        // fp32 gives up C's order for the split, so the split must pay off in the unpacking:
        // four consecutive values of C's mode have to be one aligned 16-byte vector of C
        if (in[unitCn].ext % 4)
            return false;
        for (const GettMode& m : im)
            if (m.sC % 4)
                return false;
        for (int i = 0; i < (int)in.size(); ++i)
            if (i != unitCn && in[i].sC % 4)
                return false;
        return true;
    };
    bool m_split = false;
    if (dtype == GETT_F32) {
        // fp32 operands can also be gathered element by element (4-byte cp.async), so when
        // the contraction is short (C's traffic outweighs the operands') the set that
        // carries C's stride-1 mode is ordered for C: its canonical order starts with
        // that mode, and the operand whose own stride-1 mode loses the lead is gathered
        // by elements (or along K).
        int64_t ksize = 1;
        for (const GettMode& m : ik)
            ksize *= m.ext;
        // Small N and K (the small-N kernel streams A, four consecutive rows per thread and
        // consecutive threads on consecutive row quads): if C's stride-1 mode is a mode of I_m
        // other than A's stride-1 mode, split A's mode into 4-wide pieces and put C's mode
        // right after the piece (Sec. 3.2.1 on I_m): A is still copied in 16-byte vectors and
        // a warp's stores run along C.
        int64_t nsize = 1;
        for (const GettMode& m : in)
            nsize *= m.ext;
        const int unitCm = find_unit(im, 2);
        m_split = leadM >= 0 && unitCm >= 0 && unitCm != leadM && im[leadM].ext % 4 == 0 && nsize <= 64 &&
                  ksize <= gett_ffma_skinny_max_k() && o.split_k <= 1 && o.tile_n == 0 && o.tile_k == 0 &&
                  o.stages == 0 && (o.tile_m == 0 || o.tile_m == gett_ffma_skinny_rows()) &&
                  (o.path == GETT_PATH_AUTO || o.path == GETT_PATH_FFMA);
        if (ksize <= 512) {
            if (find_unit(im, 2) >= 0 && leadM != find_unit(im, 2) && !m_split)
                leadM = -1;
            if (find_unit(in, 2) >= 0 && leadN != find_unit(in, 2) && !n_split_ok(4))
                leadN = -1;
        }
    }
    p->tm = order_with_lead(im, leadM);
    if (m_split) {
        const int unitCm = find_unit(im, 2);
        std::vector<GettDigit> t;
        t.push_back({leadM, 4, 1});
        t.push_back({unitCm, im[unitCm].ext, 1});
        if (im[leadM].ext > 4)
            t.push_back({leadM, im[leadM].ext / 4, 4});
        for (int i = 0; i < (int)im.size(); ++i)
            if (i != leadM && i != unitCm)
                t.push_back({i, im[i].ext, 1});
        p->tm = t;
    }
    p->tn = order_with_lead(in, leadN);
    {
        // Sec. 3.2.1: when B's stride-1 mode and C's stride-1 mode are two different
        // modes of I_n, split B's mode by the width of one 16-byte vector and put C's
        // mode right after that piece, so that a tile holds vectors of B and runs of C.
        const int unitCn = find_unit(in, 2);
        const int64_t vecB = dtype == GETT_F32 ? 4 : 8;
        if (n_split_ok(vecB)) {
            std::vector<GettDigit> t;
            t.push_back({leadN, vecB, 1});
            t.push_back({unitCn, in[unitCn].ext, 1});
            t.push_back({leadN, in[leadN].ext / vecB, vecB});
            for (int i = 0; i < (int)in.size(); ++i)
                if (i != leadN && i != unitCn)
                    t.push_back({i, in[i].ext, 1});
            p->tn = t;
        }
    }
    p->tk = order_with_lead(ik, leadK);
    // Operands whose stride-1 modes are two different contracted modes u (A's) and v (B's):
    // slabs of W consecutive indices of u times 8 consecutive indices of v (Sec. 3.2.1: a
    // sub-tensor made of pieces of two modes), W = one 16-byte vector (8 elements of 16 bits,
    // 4 of 32).  A is then read in 16-byte pieces along u as usual; B is read in 16-byte
    // pieces along v and its W x W blocks are transposed on the way (Sec. 3.2.2).
    bool k_transposed = false;
    if (dtype == GETT_BF16_F32 || dtype == GETT_F16_F32 || dtype == GETT_F32) {
        const int64_t W = dtype == GETT_F32 ? 4 : 8;
        const int uA = find_unit(ik, 0), uB = find_unit(ik, 1);
        if (uA >= 0 && uB >= 0 && uA != uB && ik[uA].ext % W == 0 && ik[uB].ext % 8 == 0) {
            // Consecutive slabs first walk f blocks of u under the same block of v, then the
            // blocks of v: the 16-byte pieces that share a 32-byte sector (a 128-byte line) of
            // A are asked for by neighbouring slabs, those of B at most f slabs apart, while
            // the line is still in L2.
            const int64_t eu = ik[uA].ext, ev = ik[uB].ext;
            const int64_t f = eu % (8 * W) == 0 ? 8 : eu % (4 * W) == 0 ? 4 : eu % (2 * W) == 0 ? 2 : 1;
            std::vector<GettDigit> t;
            t.push_back({uA, W, 1, 0});
            t.push_back({uB, 8, 1, 0});
            if (f > 1)
                t.push_back({uA, f, W, 0});
            if (ev > 8)
                t.push_back({uB, ev / 8, 8, 0});
            if (eu > W * f)
                t.push_back({uA, eu / (W * f), W * f, 0});
            for (int i = 0; i < (int)ik.size(); ++i)
                if (i != uA && i != uB)
                    t.push_back({i, ik[i].ext, 1, 0});
            p->tk = t;
            k_transposed = true;
        }
    }
    p->tm_seg1 = p->tn_seg1 = p->tm_hi = p->tn_hi = -1;
    if ((rc = make_dim(im, p->tm, 0, 2, p->M)) || (rc = make_dim(in, p->tn, 1, 2, p->N)) ||
        (rc = make_dim(ik, p->tk, 0, 1, p->K)))
        return rc;
    p->a_kmajor = (!ik.empty() && (im.empty() || min_stride(ik, 0) < min_stride(im, 0))) ? 1 : 0;
    p->b_kmajor = (!ik.empty() && (in.empty() || min_stride(ik, 1) < min_stride(in, 1))) ? 1 : 0;

    gett_plan_info_t& info = p->info;
    memset(&info, 0, sizeof info);
    info.M = p->M.size;
    info.N = p->N.size;
    info.K = p->K.size;
    info.n_m = (int)im.size();
    info.n_n = (int)in.size();
    info.n_k = (int)ik.size();
    for (int i = 0; i < info.n_m; ++i)
        info.labels_m[i] = im[i].label;
    for (int i = 0; i < info.n_n; ++i)
        info.labels_n[i] = in[i].label;
    for (int i = 0; i < info.n_k; ++i)
        info.labels_k[i] = ik[i].label;
    info.merged_m = merged_count(im, 0, 2);
    info.merged_n = merged_count(in, 1, 2);
    info.merged_k = merged_count(ik, 0, 1);
    info.digits_m = p->M.ndig;
    info.digits_n = p->N.ndig;
    info.digits_k = p->K.ndig;
    info.device = -1;

    // ---- which operands can be gathered in 16-byte vectors ----
    const uint32_t vec = dtype == GETT_F32 ? 4 : 8;
    info.loader_a = vec_ok(p->M, true, p->K, true, vec)    ? GETT_LOAD_VEC_FREE
                    : vec_ok(p->K, true, p->M, true, vec)  ? GETT_LOAD_VEC_K
                                                           : GETT_LOAD_SCALAR;
    info.loader_b = vec_ok(p->N, true, p->K, false, vec)   ? GETT_LOAD_VEC_FREE
                    : vec_ok(p->K, false, p->N, true, vec) ? GETT_LOAD_VEC_K
                                                           : GETT_LOAD_SCALAR;
    if (k_transposed && info.loader_a == GETT_LOAD_VEC_K && info.loader_b == GETT_LOAD_SCALAR && p->K.ndig >= 2 &&
        p->K.ext[0] == vec && p->K.sY[1] == 1 && p->K.ext[1] % 8 == 0) {
        // B in 16-byte pieces along K's second digit: every other stride of B must keep them aligned
        bool ok = p->K.sY[0] % vec == 0;
        for (int d = 2; d < p->K.ndig; ++d)
            ok = ok && p->K.sY[d] % vec == 0;
        for (int d = 0; d < p->N.ndig; ++d)
            ok = ok && p->N.sX[d] % vec == 0;
        if (ok)
            info.loader_b = GETT_LOAD_VEC_KT;
    }

    // ---- path ----
    int path = o.path;
    if (path < GETT_PATH_AUTO || path > GETT_PATH_UMMA)
        return GETT_ERR_INVALID_ARG;
    const bool both_vec = info.loader_a != GETT_LOAD_SCALAR && info.loader_b != GETT_LOAD_SCALAR;
    // The vectorised kernels keep operand offsets in 32 bits (elements for fp32, 16-byte units
    // for the 16-bit types, two top values reserved as markers).  An operand whose largest
    // offset does not fit goes to the scalar-gather kernel, whose offsets are 64-bit.
    bool offsets_fit = true;
    {
        int64_t maxA = 0, maxB = 0;
        for (const GettMode& m : im)
            maxA += (m.ext - 1) * m.sA;
        for (const GettMode& m : in)
            maxB += (m.ext - 1) * m.sB;
        for (const GettMode& m : ik) {
            maxA += (m.ext - 1) * m.sA;
            maxB += (m.ext - 1) * m.sB;
        }
        const int64_t worst = std::max(maxA, maxB);
        offsets_fit = dtype == GETT_F32 ? worst < (int64_t)0xFFFFFFF0ll : (worst >> 3) < (int64_t)0xFFFFFFF0ll;
    }
    const bool umma_ok = dtype != GETT_F32 && dtype != GETT_F64 && both_vec && offsets_fit;
    // fp32 with small N and K and a K-major A: B is read once element by element, so
    // only A has to be gatherable in 16-byte vectors
    const bool skinny_ok = dtype == GETT_F32 &&
                           (info.loader_a == GETT_LOAD_VEC_K || info.loader_a == GETT_LOAD_VEC_FREE) &&
                           p->N.size <= 64 &&
                           p->K.size <= (uint32_t)gett_ffma_skinny_max_k() && o.split_k <= 1 &&
                           (o.tile_m == 0 || o.tile_m == gett_ffma_skinny_rows()) && o.tile_n == 0 &&
                           o.tile_k == 0 && o.stages == 0 && o.epilogue != GETT_EPI_STAGED;
    const bool ffma_ok = dtype == GETT_F32 && offsets_fit; // any layout: operands without usable vectors go scalar
    if (path == GETT_PATH_AUTO)
        path = umma_ok ? GETT_PATH_UMMA : ffma_ok ? GETT_PATH_FFMA : GETT_PATH_SIMT;
    if ((path == GETT_PATH_UMMA && !umma_ok) || (path == GETT_PATH_FFMA && !ffma_ok))
        return GETT_ERR_UNSUPPORTED;
    // four consecutive tile rows (1) or columns (2) of C form one aligned 16-byte vector
    p->c_vec = vec_ok(p->M, false, p->N, false, 4) ? 1 : vec_ok(p->N, false, p->M, false, 4) ? 2 : 0;
    // every C stride except that of N digit `skip_n_digit` is a multiple of four elements
    auto others_mult4 = [&](int skip_n_digit) {
        for (int d = 0; d < p->M.ndig; ++d)
            if (p->M.sY[d] % 4)
                return false;
        for (int d = 0; d < p->N.ndig; ++d)
            if (d != skip_n_digit && p->N.sY[d] % 4)
                return false;
        return true;
    };
    // fp32, columns = a + 4 p with p running along C's stride-1 mode (the N order above):
    // four consecutive p of one a are one aligned 16-byte vector of C
    const bool split4 = dtype == GETT_F32 && p->c_vec == 0 && p->N.ndig >= 2 && p->N.ext[0] == 4 &&
                        p->N.sY[1] == 1 && p->N.ext[1] % 4 == 0 && others_mult4(1);
    info.path = path;
    p->debug = o.experiment;
    p->flags = o.flags;
    if (o.wait_limit_us < 0)
        return GETT_ERR_INVALID_ARG;
    p->wait_limit_us = o.wait_limit_us;
    p->skinny = 0;
    p->epi_lean = 0;
    memset(&p->tma_a, 0, sizeof p->tma_a);
    memset(&p->tma_b, 0, sizeof p->tma_b);

    // ---- blocking (Sec. 3.3) ----
    if (o.tile_m < 0 || o.tile_n < 0 || o.tile_k < 0 || o.stages < 0 || o.split_k < 0)
        return GETT_ERR_INVALID_ARG;
    const int sms = sm_count > 0 ? sm_count : 148;
    if (dtype == GETT_F64 && o.split_k > 1)
        return GETT_ERR_UNSUPPORTED; // (the workspace of the K slices holds fp32 sums)
    if (path == GETT_PATH_SIMT) {
        if ((o.tile_m && o.tile_m != 64) || (o.tile_n && o.tile_n != 64) ||
            (o.tile_k && o.tile_k != 16) || (o.stages && o.stages != 1) ||
            (o.epilogue && o.epilogue != GETT_EPI_DIRECT))
            return GETT_ERR_UNSUPPORTED;
        info.tile_m = 64;
        info.tile_n = 64;
        info.tile_k = 16;
        info.stages = 1;
        info.block = 256;
        info.smem_bytes = 0;
        info.epilogue = GETT_EPI_DIRECT;
        info.loader_a = info.loader_b = GETT_LOAD_SCALAR;
    } else if (path == GETT_PATH_FFMA && skinny_ok) {
        // tensor times small matrix: B stays in shared memory, A is streamed once
        p->skinny = 1;
        info.tile_m = gett_ffma_skinny_rows();
        info.tile_n = p->N.size <= 32 ? 32 : 64;
        info.tile_k = (int)p->K.size;
        info.stages = 3;
        info.block = 256;
        info.smem_bytes = info.loader_a == GETT_LOAD_VEC_K
                              ? gett_ffma_skinny_smem_bytes((int)p->N.size, (int)p->K.size, p->c_vec == 1)
                              : gett_ffma_skinny_mn_smem_bytes((int)p->N.size, (int)p->K.size);
        info.epilogue = GETT_EPI_DIRECT;
        info.loader_b = GETT_LOAD_SCALAR; // B is read once, element by element
    } else if (path == GETT_PATH_FFMA) {
        if ((o.tile_m && o.tile_m != 128 && o.tile_m != 64) || (o.tile_k && o.tile_k != 32))
            return GETT_ERR_UNSUPPORTED;
        int tn = o.tile_n ? o.tile_n : (p->N.size <= 32 ? 32 : 128);
        if (tn != 32 && tn != 128)
            return GETT_ERR_UNSUPPORTED;
        if (split4 && tn == 128)
            p->c_vec = 4; // unpacking through the shared-memory transpose with the slot pattern
        if (o.epilogue == GETT_EPI_STAGED && p->c_vec != 4)
            return GETT_ERR_UNSUPPORTED;
        // A short contraction (a few slabs) leaves a CTA's life dominated by latencies --
        // offset tables, the first copies, the read-modify-write of C -- that only other
        // resident CTAs can hide: 64-row tiles (128 threads) fit four CTAs per SM instead
        // of two.  Long contractions keep the 128-row tile's higher flops per byte.
        int tmh = o.tile_m;
        if (tmh == 0)
            tmh = (tn == 128 && ((p->K.size <= 128 && p->M.size > 128 &&
                                  (uint64_t)ceil_div(p->M.size, 64) * ceil_div(p->N.size, 128) >= 8ull * sms) ||
                                 p->M.size <= 64)) // (all rows fit the lower tile: half the padding)
                      ? 64
                      : 128;
        if (tmh == 64 && tn != 128)
            return GETT_ERR_UNSUPPORTED;
        int st = o.stages ? o.stages : (tmh == 64 ? 2 : tn == 128 ? 3 : 4);
        if (st < 2 || st > 4)
            return GETT_ERR_UNSUPPORTED;
        info.tile_m = tmh;
        info.tile_n = tn;
        info.tile_k = 32;
        info.stages = st;
        info.block = 2 * tmh;
        info.smem_bytes = gett_ffma_smem_bytes(tmh, tn, st);
        info.epilogue = p->c_vec == 4 ? GETT_EPI_STAGED : GETT_EPI_DIRECT;
    } else { // GETT_PATH_UMMA
        if ((o.tile_m && o.tile_m != 128 && o.tile_m != 256) || (o.tile_k && o.tile_k != 64))
            return GETT_ERR_UNSUPPORTED;
        // Unpacking (Eq. 11).  Direct stores are already coalesced when C's stride-1
        // mode leads the M order (a warp's 32 rows are 32 consecutive floats).  When it
        // is a mode of I_n instead, the accumulator goes through a shared-memory
        // transpose if four consecutive "slots" are one aligned 16-byte vector of C.
        int staged_cv = 0;
        if (!(p->M.ndig >= 1 && p->M.sY[0] == 1)) {
            if (p->N.ndig >= 2 && p->N.ext[0] == 8 && p->N.sY[1] == 1 && p->N.ext[1] % 4 == 0 &&
                others_mult4(1))
                staged_cv = 8;
            else if (p->N.ndig >= 1 && p->N.sY[0] == 1 && p->N.ext[0] % 4 == 0 && others_mult4(0))
                staged_cv = 1;
        }
        {
            // the staged epilogue keeps C offsets in 32 bits, in units of 16 bytes
            int64_t maxC = 0;
            for (const GettMode& m : im)
                maxC += (m.ext - 1) * m.sC;
            for (const GettMode& m : in)
                maxC += (m.ext - 1) * m.sC;
            if ((maxC >> 2) >= (int64_t)0xFFFFFFF0ll)
                staged_cv = 0;
        }
        if (o.epilogue == GETT_EPI_DIRECT)
            staged_cv = 0;
        if (o.epilogue == GETT_EPI_STAGED && !staged_cv)
            return GETT_ERR_UNSUPPORTED;
        info.epilogue = staged_cv ? GETT_EPI_STAGED : GETT_EPI_DIRECT;
        if (staged_cv)
            p->c_vec = staged_cv;
        int tn = o.tile_n;
        if (tn == 0 && staged_cv == 8) {
            // one tile = all 8-wide pieces x the whole of C's stride-1 mode, if that is a legal width
            // (the widest legal width that holds whole runs: fewer, larger tiles)
            const uint32_t want = 8 * p->N.ext[1];
            for (uint32_t cand : {256u, 192u, 128u, 64u})
                if (cand % want == 0) {
                    tn = (int)cand;
                    break;
                }
        }
        if (tn == 0) {
            // fewest waves x per-tile cost; ties go to the wider tile
            const uint32_t tm_count = ceil_div(p->M.size, 128);
            uint64_t best = UINT64_MAX;
            for (int cand : {256, 192, 128, 64}) {
                if (cand > 64 && (uint32_t)cand >= p->N.size + 64)
                    continue; // a narrower tile already covers N
                uint64_t t = (uint64_t)tm_count * ceil_div(p->N.size, (uint32_t)cand);
                uint64_t cost = ((t + sms - 1) / sms) * (uint64_t)(cand + 64); // MMA width + A reload
                if (cost < best) {
                    best = cost;
                    tn = cand;
                }
            }
        }
        // A small output with a long contraction is cut along K until every SM has a piece
        // (below), so the tile count no longer matters; what the tile shape then decides is
        // how often the operands are delivered: A once per column of tiles, B once per row
        // of tiles, padding included.  Take the shape that moves the fewest bytes.
        int tm_few = 0;
        if (o.tile_n == 0 && staged_cv != 8 && o.split_k != 1 && p->K.size >= 8 * 64 &&
            (uint64_t)ceil_div(p->M.size, 128) * ceil_div(p->N.size, (uint32_t)tn) * 2 <= (uint64_t)sms) {
            uint64_t best = UINT64_MAX;
            for (int cm : {128, 256})
                for (int cn : {64, 128, 192, 256}) {
                    if (cm == 256 && (cn != 256 || staged_cv || (o.tile_m && o.tile_m != 256)))
                        continue;
                    if (cm == 128 && o.tile_m == 256)
                        continue;
                    const uint64_t rows = ceil_div(p->M.size, (uint32_t)cm), cols = ceil_div(p->N.size, (uint32_t)cn);
                    if (rows * cols * 2 > (uint64_t)sms)
                        continue;
                    const uint64_t moved = cols * rows * cm + rows * cols * cn; // x K elements
                    if (moved < best) {
                        best = moved;
                        tn = cn;
                        tm_few = cm;
                    }
                }
        }
        if (tn != 64 && tn != 128 && tn != 192 && tn != 256)
            return GETT_ERR_UNSUPPORTED;
        const int smem_limit = 227 * 1024;
        // The staging rows take shared memory from the operand ring.  A long contraction
        // needs the ring (three stages, or one per slab) more than it needs the old values of
        // C one chunk ahead: its unpacking hides behind the next tile's main loop, so it gets
        // the lean staging (one narrow buffer per warp).
        int lean = 0;
        if (staged_cv) {
            const int need = (int)std::min<uint32_t>(3, ceil_div(p->K.size, 64));
            if (gett_umma_max_stages(128, tn, smem_limit, staged_cv, 0) < need)
                lean = 1;
        }
        p->epi_lean = lean;
        const int staged = info.epilogue == GETT_EPI_STAGED;
        // 256-row tiles (both accumulator buffers for one tile) cut the operand bytes per
        // flop by a third; worth it when the contraction is long enough to be bound by
        // operand delivery and there are still at least two waves of tiles.  The epilogue
        // then no longer overlaps the next tile's main loop.
        int tmh = o.tile_m;
        if (tmh == 0) {
            const uint64_t t256 = (uint64_t)ceil_div(p->M.size, 256) * ceil_div(p->N.size, 256);
            tmh = tm_few ? tm_few : (tn == 256 && !staged && p->K.size >= 2048 && t256 >= 2ull * sms) ? 256 : 128;
        }
        if (tmh == 256 && (tn != 256 || staged))
            return GETT_ERR_UNSUPPORTED;
        int st = o.stages ? o.stages : gett_umma_max_stages(tmh, tn, smem_limit, staged_cv, lean);
        if (st < 1 || st > gett_umma_max_stages(tmh, tn, smem_limit, staged_cv, lean) || st % gett_umma_prod_groups(st))
            return GETT_ERR_UNSUPPORTED;
        info.tile_m = tmh;
        info.tile_n = tn;
        info.tile_k = 64;
        info.stages = st;
        info.block = gett_umma_block();
        info.smem_bytes = gett_umma_smem_bytes(tmh, tn, st, staged_cv, lean);
        if (!(p->flags & GETT_OPT_NO_TMA)) {
            make_tma_recipe(p->M, true, p->K, true, info.loader_a, (uint32_t)tmh, p->tma_a);
            make_tma_recipe(p->N, true, p->K, false, info.loader_b, (uint32_t)tn, p->tma_b);
            // Both operands staged as rows of 64 free indices and not both tiles boxes: order
            // I_m, I_n and I_k so that the tiles consist of 64 x 64 atoms that are boxes
            // (Sec. 3.2.1: sub-tensors made of pieces of one or two modes), and fetch those by TMA.
            if (!(p->tma_a.enabled && p->tma_b.enabled) && info.loader_a == GETT_LOAD_VEC_FREE &&
                info.loader_b == GETT_LOAD_VEC_FREE && !staged_cv && !ik.empty() && !(p->flags & GETT_OPT_NO_ATOMS)) {
                const KOrder ko = slab_order(ik, p->tk);
                const SideOrder sa = atom_order(im, p->tm, 0), sb = atom_order(in, p->tn, 1);
                GettDim M2, N2, K2;
                std::vector<int> srcm, srcn, srck;
                if (ko.ok && (sa.ok || sb.ok) &&
                    make_dim(im, sa.ok ? sa.digits : p->tm, 0, 2, M2, sa.ok ? sa.seg1 : -1, sa.hi, false, &srcm) == GETT_OK &&
                    make_dim(in, sb.ok ? sb.digits : p->tn, 1, 2, N2, sb.ok ? sb.seg1 : -1, sb.hi, false, &srcn) == GETT_OK &&
                    make_dim(ik, ko.digits, 0, 1, K2, -1, -1, false, &srck) == GETT_OK) {
                    GettTmaRecipe ra, rb;
                    const bool oka = sa.ok && make_atom_recipe(im, sa, srcm, M2, ik, ko, srck, 0, ra);
                    const bool okb = sb.ok && make_atom_recipe(in, sb, srcn, N2, ik, ko, srck, 1, rb);
                    if ((int)oka + (int)okb > p->tma_a.enabled + p->tma_b.enabled) {
                        if (oka) {
                            p->tm = sa.digits;
                            p->tm_seg1 = sa.seg1;
                            p->tm_hi = sa.hi;
                            p->tma_a = ra;
                        } else {
                            memset(&p->tma_a, 0, sizeof p->tma_a);
                        }
                        if (okb) {
                            p->tn = sb.digits;
                            p->tn_seg1 = sb.seg1;
                            p->tn_hi = sb.hi;
                            p->tma_b = rb;
                        } else {
                            memset(&p->tma_b, 0, sizeof p->tma_b);
                        }
                        p->tk = ko.digits;
                        // (a side that keeps the gather keeps its order; its digits are only no longer merged)
                        if ((rc = make_dim(im, p->tm, 0, 2, p->M, p->tm_seg1, p->tm_hi, false)) ||
                            (rc = make_dim(in, p->tn, 1, 2, p->N, p->tn_seg1, p->tn_hi, false)))
                            return rc;
                        p->K = K2;
                        info.digits_m = p->M.ndig;
                        info.digits_n = p->N.ndig;
                        info.digits_k = p->K.ndig;
                    }
                }
            }
            if (p->tma_a.enabled)
                info.loader_a = info.loader_a == GETT_LOAD_VEC_FREE ? GETT_LOAD_TMA_FREE : GETT_LOAD_TMA_K;
            if (p->tma_b.enabled)
                info.loader_b = info.loader_b == GETT_LOAD_VEC_FREE ? GETT_LOAD_TMA_FREE : GETT_LOAD_TMA_K;
        }
    }
    p->tiles_m = ceil_div(p->M.size, (uint32_t)info.tile_m);
    p->tiles_n = ceil_div(p->N.size, (uint32_t)info.tile_n);
    uint64_t tiles = (uint64_t)p->tiles_m * p->tiles_n;
    if (tiles >= (1ull << 31))
        return GETT_ERR_UNSUPPORTED;
    info.tiles = (int64_t)tiles;

    // ---- split-K: slice I_k when the output alone cannot fill the machine ----
    uint32_t kslabs = ceil_div(p->K.size, (uint32_t)info.tile_k);
    uint32_t split = 1;
    if (o.split_k > 1) {
        split = std::min<uint32_t>((uint32_t)o.split_k, kslabs);
    } else if (o.split_k == 0 && dtype != GETT_F64 && sm_count > 0 && tiles * 2 <= (uint64_t)sm_count && kslabs >= 8) {
        // choose the slice count whose (waves of work items) x (slabs per item + a fixed
        // per-item cost for the epilogue and the reduction) is smallest
        const uint64_t slots = (uint64_t)sm_count * (path == GETT_PATH_UMMA ? 1 : path == GETT_PATH_FFMA ? 2 : 4);
        uint64_t best = UINT64_MAX;
        for (uint32_t s = 1; s <= std::min<uint32_t>(kslabs / 4, 256); ++s) {
            const uint64_t waves = (tiles * s + slots - 1) / slots;
            const uint64_t cost = waves * (ceil_div(kslabs, s) + 6) + s / 2;
            if (cost < best) {
                best = cost;
                split = s;
            }
        }
    }
    uint32_t slabs_per = ceil_div(kslabs, split);
    split = ceil_div(kslabs, slabs_per); // no empty slice
    if (tiles * split >= (1ull << 31))
        return GETT_ERR_UNSUPPORTED;
    info.split_k = (int32_t)split;
    p->k_per_split = slabs_per * (uint32_t)info.tile_k;
    info.workspace_bytes = split > 1 ? (int64_t)split * p->M.size * p->N.size * 4 : 0;
    info.grid = (int32_t)(tiles * split);
    if (path == GETT_PATH_UMMA) // persistent: one CTA per SM walks the work list
        info.grid = (int32_t)std::min<uint64_t>(tiles * split, (uint64_t)sms);
    // ---- stream-K: no idle SMs in a last partial wave of tiles ----
    // With more tiles than SMs but a tile count that leaves much of the last wave empty, the
    // tiles of the whole rounds are dealt out as usual and the left-over tiles are cut along K
    // (one more way of cutting the three loops, Sec. 2.1 / Sec. 3.3): their tiles x slabs space
    // is dealt out in equal shares, the pieces go through the workspace and a second kernel adds
    // them.  Only with the direct epilogue, without K slices.
    p->stream_k = p->sk_full = p->sk_units = p->sk_slabs = p->sk_pmax = 0;
    if (path == GETT_PATH_UMMA && split == 1 && info.epilogue == GETT_EPI_DIRECT && !(p->flags & GETT_OPT_NO_STREAMK) &&
        tiles > (uint64_t)sms && tiles % sms != 0 && kslabs >= 2 && tiles * kslabs < (1ull << 31)) {
        const uint64_t full = tiles / sms, left = tiles - full * sms;
        const uint64_t units = (left * kslabs + sms - 1) / sms; // slab units per CTA
        uint64_t pmax = 1;
        for (uint64_t r = 0; r < left; ++r)
            pmax = std::max<uint64_t>(pmax, ((r + 1) * kslabs - 1) / units - (r * kslabs) / units + 1);
        const int64_t ws_bytes = (int64_t)(left * pmax) * info.tile_m * info.tile_n * 4;
        // worth it when the time of the SMs that would idle through the last round exceeds what the
        // pieces cost (their trip through memory and the second launch), with a margin
        const double slab_us = 2.0 * info.tile_m * info.tile_n * 64 / (1.67e15 / sms) * 1e6 / 0.8; // one SM
        const double saved_us = (1.0 - (double)left / sms) * kslabs * slab_us;
        const double cost_us = 2.0 * (double)ws_bytes / 6.5e6 + 10.0;
        if (((saved_us > 1.5 * cost_us && units >= 4) || (p->flags & GETT_OPT_STREAMK)) && ws_bytes <= (1ll << 30)) {
            p->stream_k = 1;
            p->sk_full = (uint32_t)full;
            p->sk_slabs = kslabs;
            p->sk_units = (uint32_t)units;
            p->sk_pmax = (uint32_t)pmax;
            info.workspace_bytes = ws_bytes;
            info.grid = sms;
        }
    }
    info.stream_k = (int32_t)p->stream_k;
    if (p->skinny) // persistent: two CTAs per SM stream the row tiles
        info.grid = (int32_t)std::min<uint64_t>(p->tiles_m, 2ull * sms);
    // two neighbouring 256 x 256 tiles per CTA pair, A shared between the two CTAs
    p->pair_ok = path == GETT_PATH_UMMA && p->tma_a.enabled && p->tma_b.enabled && !p->tma_a.hybrid &&
                 !p->tma_b.hybrid && info.tile_m == 256 &&
                 info.tile_n == 256 && info.epilogue == GETT_EPI_DIRECT && split == 1 && p->tiles_n % 2 == 0 &&
                 !p->stream_k && !(p->flags & GETT_OPT_NO_PAIR);
    info.swapped = p->swapped;
    if (p->swapped) { // report the caller's view
        std::swap(info.M, info.N);
        std::swap(info.n_m, info.n_n);
        std::swap(info.merged_m, info.merged_n);
        std::swap(info.digits_m, info.digits_n);
        std::swap(info.loader_a, info.loader_b);
        for (int i = 0; i < GETT_MAX_MODES; ++i)
            std::swap(info.labels_m[i], info.labels_n[i]);
    }
    return GETT_OK;
}

// Canonical table `which`: every tile-order fused index t is taken apart into its digits
// (the digits the kernels receive), which give both the per-mode indices -- hence the
// canonical fused index the entry belongs to -- and, through gett_decompose(), the offset.
gett_status_t gett_planner_table(const gett_plan* p, int which, int64_t* dst, size_t capacity)
{
    const std::vector<GettMode>* modes;
    const std::vector<GettDigit>* digits;
    const GettDim* D;
    bool wantX;
    int seg1 = -1, hi = -1;
    if (p->swapped) { // the caller's A is the kernels' B: rows <-> columns, X <-> Y for K
        switch (which) {
        case GETT_TABLE_A_M: which = GETT_TABLE_B_N; break;
        case GETT_TABLE_C_M: which = GETT_TABLE_C_N; break;
        case GETT_TABLE_B_N: which = GETT_TABLE_A_M; break;
        case GETT_TABLE_C_N: which = GETT_TABLE_C_M; break;
        case GETT_TABLE_A_K: which = GETT_TABLE_B_K; break;
        case GETT_TABLE_B_K: which = GETT_TABLE_A_K; break;
        default: break;
        }
    }
    switch (which) {
    case GETT_TABLE_A_M: modes = &p->im; digits = &p->tm; D = &p->M; wantX = true; seg1 = p->tm_seg1; hi = p->tm_hi; break;
    case GETT_TABLE_C_M: modes = &p->im; digits = &p->tm; D = &p->M; wantX = false; seg1 = p->tm_seg1; hi = p->tm_hi; break;
    case GETT_TABLE_B_N: modes = &p->in; digits = &p->tn; D = &p->N; wantX = true; seg1 = p->tn_seg1; hi = p->tn_hi; break;
    case GETT_TABLE_C_N: modes = &p->in; digits = &p->tn; D = &p->N; wantX = false; seg1 = p->tn_seg1; hi = p->tn_hi; break;
    case GETT_TABLE_A_K: modes = &p->ik; digits = &p->tk; D = &p->K; wantX = true; break;
    case GETT_TABLE_B_K: modes = &p->ik; digits = &p->tk; D = &p->K; wantX = false; break;
    default: return GETT_ERR_INVALID_ARG;
    }
    if (!dst || capacity < D->size)
        return GETT_ERR_INVALID_ARG;
    const int nm = (int)modes->size();
    const int nd = (int)digits->size();
    std::vector<int64_t> idx(nm);
    std::vector<uint64_t> weight(nm); // of a mode in the canonical fused index, first mode fastest
    uint64_t w = 1;
    for (int j = 0; j < nm; ++j) {
        weight[j] = w;
        w *= (uint64_t)(*modes)[j].ext;
    }
    // sizes of the two segments of the low part (a plain order is one "segment" with no high part)
    const bool two = seg1 > 0;
    const int s1 = two ? seg1 : nd, h = two ? hi : nd;
    uint64_t size0 = 1, size1 = 1;
    for (int i = 0; i < s1; ++i)
        size0 *= (uint64_t)(*digits)[i].ext;
    for (int i = s1; i < h; ++i)
        size1 *= (uint64_t)(*digits)[i].ext;
    const uint64_t period = two ? size0 + size1 : size0;
    auto take = [&](int from, int to, uint64_t rem) {
        for (int i = from; i < to; ++i) {
            const GettDigit& g = (*digits)[i];
            idx[g.mode] += g.off + (int64_t)(rem % (uint64_t)g.ext) * g.mult;
            rem /= (uint64_t)g.ext;
        }
    };
    std::vector<bool> seen(D->size, false);
    for (uint32_t t = 0; t < D->size; ++t) {
        std::fill(idx.begin(), idx.end(), 0);
        const uint64_t lo = two ? t % period : t;
        if (two && lo >= size0)
            take(s1, h, lo - size0);
        else
            take(0, s1, lo);
        if (two)
            take(h, nd, t / period);
        uint64_t c = 0;
        for (int j = 0; j < nm; ++j)
            c += (uint64_t)idx[j] * weight[j];
        if (c >= D->size || seen[c])
            return GETT_ERR_INVALID_ARG; // the tile order is not a permutation of the canonical one
        seen[c] = true;
        int64_t ox, oy;
        gett_decompose(*D, t, ox, oy);
        dst[c] = wantX ? ox : oy;
    }
    return GETT_OK;
}
