// C-ABI entry points of libgaconv: argument validation, workspace planning, kernel dispatch and the
// approximation-schedule driver (paper Section 2.5).  Every step of the path runs in this library's
// kernels; there is no CPU or library fallback.
#include <atomic>
#include <cstring>
#include <mutex>
#include <new>
#include <utility>
#include <vector>

#include "gaconv_internal.h"

using namespace gaconv;

static std::atomic<uint64_t> g_launches{0};
void gaconv::note_launch(int count) { g_launches.fetch_add((uint64_t)count, std::memory_order_relaxed); }

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

gaconv_status_t make_geom(const gaconv_conv_desc_t* d, Geom* g)
{
    if (d == nullptr) return GACONV_ERR_NULL_POINTER;
    if (d->struct_size != sizeof(gaconv_conv_desc_t)) return GACONV_ERR_BAD_DESC;
    if (d->n < 1 || d->c < 1 || d->h < 1 || d->w < 1 || d->k < 1 || d->r < 1 || d->s < 1) return GACONV_ERR_BAD_DESC;
    if (d->stride_h < 1 || d->stride_w < 1 || d->pad_h < 0 || d->pad_w < 0) return GACONV_ERR_BAD_DESC;
    if (d->h + 2 * d->pad_h < d->r || d->w + 2 * d->pad_w < d->s) return GACONV_ERR_BAD_DESC;
    if (d->in_dtype != GACONV_F32 && d->in_dtype != GACONV_BF16) return GACONV_ERR_BAD_DESC;
    if (d->x_layout != GACONV_X_NHWC && d->x_layout != GACONV_X_NCHW) return GACONV_ERR_BAD_DESC;
    if (d->dy_layout != GACONV_DY_NKPQ && d->dy_layout != GACONV_DY_NPQK) return GACONV_ERR_BAD_DESC;
    if (d->dw_layout != GACONV_DW_KRSC && d->dw_layout != GACONV_DW_KCRS && d->dw_layout != GACONV_DW_RSCK) return GACONV_ERR_BAD_DESC;
    if (d->math != GACONV_MATH_DEFAULT && d->math != GACONV_MATH_TF32) return GACONV_ERR_BAD_DESC;
    if (d->algo < GACONV_ALGO_AUTO || d->algo > GACONV_ALGO_TENSOR) return GACONV_ERR_BAD_DESC;
    g->n = d->n; g->c = d->c; g->h = d->h; g->w = d->w; g->k = d->k; g->r = d->r; g->s = d->s;
    g->stride_h = d->stride_h; g->stride_w = d->stride_w; g->pad_h = d->pad_h; g->pad_w = d->pad_w;
    g->p = (d->h + 2 * d->pad_h - d->r) / d->stride_h + 1;
    g->q = (d->w + 2 * d->pad_w - d->s) / d->stride_w + 1;
    if (g->p < 1 || g->q < 1) return GACONV_ERR_BAD_DESC;
    // element counts must fit comfortably in 63 bits and per-map sizes in 31
    if ((long long)g->p * g->q > (1ll << 30) || (long long)g->r * g->s * g->c > (1ll << 30)) return GACONV_ERR_UNSUPPORTED;
    if (d->x_layout == GACONV_X_NHWC) {
        g->xs_c = 1; g->xs_w = d->c; g->xs_h = (long long)d->w * d->c; g->xs_n = (long long)d->h * d->w * d->c;
    } else {
        g->xs_w = 1; g->xs_h = d->w; g->xs_c = (long long)d->h * d->w; g->xs_n = (long long)d->c * d->h * d->w;
    }
    if (d->dw_layout == GACONV_DW_KRSC) {
        g->ws_c = 1; g->ws_s = d->c; g->ws_r = (long long)d->s * d->c; g->ws_k = (long long)d->r * d->s * d->c;
    } else if (d->dw_layout == GACONV_DW_KCRS) {
        g->ws_s = 1; g->ws_r = d->s; g->ws_c = (long long)d->r * d->s; g->ws_k = (long long)d->c * d->r * d->s;
    } else {
        g->ws_k = 1; g->ws_c = d->k; g->ws_s = (long long)d->c * d->k; g->ws_r = (long long)d->s * d->c * d->k;
    }
    g->bf16 = d->in_dtype == GACONV_BF16;
    g->alpha = d->alpha;
    if (d->sm_budget < 0) return GACONV_ERR_BAD_DESC;
    g->sm_budget = d->sm_budget;
    return GACONV_OK;
}

// ---- plans are kept: the planners run once per (problem, device), not once per call --------------------------------
// A key is every field a plan depends on, plus the device (SM count and resident clusters differ between devices).
struct PlanKey {
    long long v[26];
    bool operator==(const PlanKey& o) const { return memcmp(v, o.v, sizeof(v)) == 0; }
};
PlanKey plan_key(const Geom& g, int a, int b)
{
    int dev = 0;
    cudaGetDevice(&dev);
    uint32_t alpha_bits;
    memcpy(&alpha_bits, &g.alpha, sizeof(alpha_bits));
    return PlanKey{{g.n, g.c, g.h, g.w, g.k, g.r, g.s, g.p, g.q, g.stride_h, g.stride_w, g.pad_h, g.pad_w, g.xs_n, g.xs_c, g.xs_h,
                    g.xs_w, g.ws_k, g.ws_c, g.ws_r, g.ws_s, g.bf16 ? 1 : 0, (long long)alpha_bits, g.sm_budget, ((long long)a << 32) | (uint32_t)b, dev}};
}
template <typename L>
class PlanCache {
public:
    template <typename Build>
    L get(const PlanKey& key, Build build)
    {
#ifndef GACONV_TUNING            // tuning builds read planner overrides from the environment on every call
        {
            std::lock_guard<std::mutex> lock(m_);
            for (size_t i = 0; i < e_.size(); ++i)
                if (e_[i].first == key) {
                    if (i != 0) std::swap(e_[i], e_[i - 1]);       // frequently used entries drift to the front
                    return e_[i != 0 ? i - 1 : 0].second;
                }
        }
#endif
        L made = build();
#ifndef GACONV_TUNING
        std::lock_guard<std::mutex> lock(m_);
        if (e_.size() >= kMaxEntries) e_.pop_back();
        e_.emplace_back(key, made);
#endif
        return made;
    }
private:
    static constexpr size_t kMaxEntries = 256;
    std::mutex m_;
    std::vector<std::pair<PlanKey, L>> e_;
};

// Small maps with many channels (up to 4x4 pixels from 128 channels, up to 8x8 from 256): the N*K patch accumulations (N*K*R*S*C FMAs on the FP32 pipes,
// the same number of bytes gathered from L2) cost more than the dense contraction on tensor cores, and with so few
// pixels per map the sparse tensor is not that sparse (1 - 1/(PQ), Section 2.3).  Then the method is run
// literally as the paper states it: build the sparse version of dY (one entry per map, the signed sum) and take
// its exact filter gradient with the tensor-core kernel.  (8x8 maps: the gather kernel is faster with 128 channels;
// with 256 the two tie alone and the dense route is cheaper among other layers, so it is taken from 256 channels on.)
bool top1_dense_route(const Geom& g, TcPlan* tp)
{
    return g.bf16 && ((g.p * g.q <= 16 && g.c >= 128) || (g.p * g.q <= 64 && g.c >= 256)) && plan_tc(g, tp);
}

struct Top1Layout { size_t idx_off, sum_off, partial_off, sparse_off, scratch_off, total; GatherPlan gp; TcPlan tp; bool dense; };
Top1Layout build_top1_layout(const Geom& g)
{
    Top1Layout L;
    L.gp = plan_gather(g);
    L.dense = top1_dense_route(g, &L.tp);
    const size_t maps = (size_t)g.n * g.k;
    L.idx_off = kWsDataOffset;
    L.sum_off = align_up(L.idx_off + maps * sizeof(int32_t), 256);
    L.partial_off = align_up(L.sum_off + maps * sizeof(float), 256);
    size_t partial = L.gp.partial_bytes;
    if (L.dense && L.tp.partial_bytes > partial) partial = L.tp.partial_bytes;
    L.sparse_off = align_up(L.partial_off + partial, 256);
    L.scratch_off = align_up(L.sparse_off + (L.dense ? maps * g.p * g.q * 2 : 0), 256);
    L.total = align_up(L.scratch_off + (L.dense ? L.tp.scratch_bytes : 0), 256);
    return L;
}

Top1Layout top1_layout(const Geom& g)
{
    static PlanCache<Top1Layout> cache;
    return cache.get(plan_key(g, 0, 0), [&] { return build_top1_layout(g); });
}

struct ExactLayout { size_t partial_off, scratch_off, total; DirectPlan dp; TcPlan tp; StemPlan sp; bool tc_ok, stem_ok; };
// fp32 inputs take the tcgen05 kernel (TF32 MMAs on split operands) where the layer is wide enough for the
// tensor cores to pay for the extra pass that splits the operands: 64 input channels, or 32 when the filter
// rows share one MMA (measured: 32->32@16x16 18.7 us against 19.9 us on the warp-level path; without the
// stacking 24 us); the one-pass TF32 mode needs no split
bool tc_f32_wanted(const Geom& g, int math, int algo) { return !g.bf16 && (math == GACONV_MATH_TF32 || algo == GACONV_ALGO_TENSOR || g.c >= 32); }

ExactLayout build_exact_layout(const Geom& g, int math, int algo)
{
    ExactLayout L;
    L.dp = plan_direct(g);
    L.tc_ok = g.bf16 ? plan_tc(g, &L.tp) : (tc_f32_wanted(g, math, algo) && plan_tc_f32(g, math == GACONV_MATH_TF32 ? 1 : 3, &L.tp));
    // (32 channels: only with stacked rows and operands small enough that writing and re-reading their split planes
    //  stays cheap -- 32->16@32x32 with 25 MB of inputs measured 36 us on this path)
    const size_t in_bytes = ((size_t)g.n * g.c * g.h * g.w + (size_t)g.n * g.k * g.p * g.q) * 4;
    if (L.tc_ok && !g.bf16 && g.c < 64 && (!L.tp.stacked_rows || in_bytes > ((size_t)12 << 20)) && math != GACONV_MATH_TF32 &&
        algo != GACONV_ALGO_TENSOR) L.tc_ok = false;
    L.partial_off = kWsDataOffset;
    size_t partial = L.dp.partial_bytes;
    if (L.tc_ok && L.tp.partial_bytes > partial) partial = L.tp.partial_bytes;
    L.stem_ok = plan_stem(g, &L.sp);
    if (L.stem_ok && L.sp.partial_bytes > partial) partial = L.sp.partial_bytes;
    L.scratch_off = align_up(L.partial_off + partial, 256);
    L.total = align_up(L.scratch_off + (L.tc_ok ? L.tp.scratch_bytes : 0), 256);
    return L;
}

ExactLayout exact_layout(const Geom& g, int math, int algo)
{
    static PlanCache<ExactLayout> cache;
    return cache.get(plan_key(g, math, algo), [&] { return build_exact_layout(g, math, algo); });
}

// entries retained per map by the top-k method: desc->topk clamped to the map size; 0 = invalid
int topk_of(const gaconv_conv_desc_t* d, const Geom& g)
{
    if (d->topk < 1 || d->topk > GACONV_MAX_TOPK) return 0;
    const long long pq = (long long)g.p * g.q;
    return d->topk < pq ? d->topk : (int)pq;
}

struct TopkLayout { size_t idx_off, sum_off, partial_off, total; GatherPlan gp; };
TopkLayout topk_layout(const Geom& g, int topk)
{
    TopkLayout L;
    L.gp = plan_gather(g);
    const size_t maps = (size_t)g.n * g.k;
    L.idx_off = kWsDataOffset;
    L.sum_off = align_up(L.idx_off + maps * topk * sizeof(int32_t), 256);
    L.partial_off = align_up(L.sum_off + maps * sizeof(float), 256);
    L.total = align_up(L.partial_off + L.gp.partial_bytes, 256);
    return L;
}

gaconv_status_t check_ws(const gaconv_conv_desc_t* d, size_t need)
{
    if (d->workspace == nullptr) return GACONV_ERR_NULL_POINTER;
    if (!aligned16(d->workspace)) return GACONV_ERR_MISALIGNED;
    if (d->workspace_bytes < need) return GACONV_ERR_WORKSPACE_TOO_SMALL;
    return GACONV_OK;
}

uint64_t splitmix64(uint64_t x)
{
    uint64_t z = x + 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// ---- operand layouts other than the kernels' own ---------------------------------------------------------------
// The fast kernels (tensor-core, stem, vectorised gather) read channels-last activations, and every kernel reads dY
// as N x K x P x Q.  An N x P x Q x K gradient (what a channels-last framework hands over) is always transposed into
// the tail of the workspace; an N x C x H x W input is transposed where a fast kernel serves the channels-last
// version of the problem, and read in place by the FP32-pipe and scalar-gather kernels otherwise (odd shapes,
// GACONV_ALGO_DIRECT).  The call then continues with an inner descriptor in the kernels' layouts whose workspace is
// the head of the caller's.
struct Relayout { size_t inner_bytes; bool move_x, move_dy; gaconv_conv_desc_t inner; };
size_t x_bytes_of(const gaconv_conv_desc_t* d) { return (size_t)d->n * d->c * d->h * d->w * (d->in_dtype == GACONV_BF16 ? 2 : 4); }
size_t dy_bytes_of(const Geom& g) { return (size_t)g.n * g.k * g.p * g.q * (g.bf16 ? 2 : 4); }

// workspace of a call in the kernels' own dY layout (x in either layout); 0 with *ok = false when the descriptor is bad
size_t native_ws_bytes(const gaconv_conv_desc_t* desc, const Geom& g, int32_t method, bool* ok)
{
    *ok = true;
    switch (method) {
        case GACONV_METHOD_EXACT: return exact_layout(g, desc->math, desc->algo).total;
        case GACONV_METHOD_TOP1: return top1_layout(g).total;
        case GACONV_METHOD_TOPK: {
            const int t = topk_of(desc, g);
            if (t < 1) { *ok = false; return 0; }
            return topk_layout(g, t).total;
        }
        case GACONV_METHOD_ZERO:
        case GACONV_METHOD_RANDOM: return kWsDataOffset;
    }
    *ok = false;
    return 0;
}

// which operands move, and the inner call's workspace size; move_x == move_dy == false: the call runs as it is
Relayout plan_relayout(const gaconv_conv_desc_t* desc, int32_t method)
{
    Relayout R{};
    R.inner = *desc;
    const bool reads_inputs = method == GACONV_METHOD_EXACT || method == GACONV_METHOD_TOP1 || method == GACONV_METHOD_TOPK;
    if (!reads_inputs) return R;
    R.move_dy = desc->dy_layout == GACONV_DY_NPQK && desc->k > 1;          // (one output channel: the two orders coincide)
    R.inner.dy_layout = GACONV_DY_NKPQ;
    if (desc->x_layout == GACONV_X_NCHW && desc->c >= 2 && desc->algo != GACONV_ALGO_DIRECT) {
        gaconv_conv_desc_t cl = R.inner;
        cl.x_layout = GACONV_X_NHWC;
        Geom gi;
        if (make_geom(&cl, &gi) == GACONV_OK) {
            if (method == GACONV_METHOD_EXACT) {
                const ExactLayout L = exact_layout(gi, desc->math, desc->algo);
                R.move_x = L.tc_ok || L.stem_ok || direct_mma_supported(gi, L.dp);
            } else if (method == GACONV_METHOD_TOP1) {
                R.move_x = top1_layout(gi).dense || (top1_fused_supported(gi) && gi.c % 4 == 0);
            } else {
                R.move_x = topk_of(desc, gi) >= 1 && top1_fused_supported(gi) && gi.c % 4 == 0;
            }
            if (R.move_x) R.inner = cl;
        }
    }
    if (R.move_x || R.move_dy) {
        Geom gi;
        bool ok = false;
        if (make_geom(&R.inner, &gi) == GACONV_OK) R.inner_bytes = native_ws_bytes(&R.inner, gi, method, &ok);
        if (!ok) { R.move_x = R.move_dy = false; R.inner = *desc; R.inner_bytes = 0; }
    }
    return R;
}

// Transposes what has to move into the workspace tail and hands back the inner descriptor and operand pointers.
// *moved == false: nothing to do, the caller goes on with its own descriptor.
gaconv_status_t relayout_operands(const void* x, const void* dy, const gaconv_conv_desc_t* desc, int32_t method, cudaStream_t cs,
                                  gaconv_conv_desc_t* inner, const void** x_out, const void** dy_out, bool* moved)
{
    const Relayout R = plan_relayout(desc, method);
    *moved = R.move_x || R.move_dy;
    if (!*moved) return GACONV_OK;
    Geom g;
    gaconv_status_t st = make_geom(desc, &g);
    if (st != GACONV_OK) return st;
    const size_t head = align_up(R.inner_bytes, 256);
    const size_t x_tail = R.move_x ? align_up(x_bytes_of(desc), 256) : 0;
    st = check_ws(desc, head + x_tail + (R.move_dy ? dy_bytes_of(g) : 0));
    if (st != GACONV_OK) return st;
    char* ws = static_cast<char*>(desc->workspace);
    *x_out = x; *dy_out = dy;
    if (R.move_x) {
        if (launch_transpose_batched(x, ws + head, g.c, g.h * g.w, g.n, g.bf16, cs) != cudaSuccess) return GACONV_ERR_CUDA;
        *x_out = ws + head;
    }
    if (R.move_dy) {
        if (launch_transpose_batched(dy, ws + head + x_tail, g.p * g.q, g.k, g.n, g.bf16, cs) != cudaSuccess) return GACONV_ERR_CUDA;
        *dy_out = ws + head + x_tail;
    }
    *inner = R.inner;
    inner->workspace_bytes = head;
    return GACONV_OK;
}

}  // namespace

struct gaconv_schedule {
    int32_t num_layers, kind, method;
    double fraction;
    uint64_t seed;
    bool* mask;   // SEEDED_FRACTION: layers in the approximated subset
};

extern "C" {

const char* gaconv_status_string(gaconv_status_t s)
{
    switch (s) {
        case GACONV_OK: return "ok";
        case GACONV_ERR_NULL_POINTER: return "null pointer";
        case GACONV_ERR_BAD_DESC: return "bad descriptor";
        case GACONV_ERR_UNSUPPORTED: return "unsupported request";
        case GACONV_ERR_MISALIGNED: return "pointer not 16-byte aligned";
        case GACONV_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case GACONV_ERR_CUDA: return "CUDA error";
        case GACONV_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

uint64_t gaconv_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

gaconv_status_t gaconv_workspace_size(const gaconv_conv_desc_t* desc, int32_t method, size_t* bytes)
{
    if (bytes == nullptr) return GACONV_ERR_NULL_POINTER;
    Geom g;
    gaconv_status_t st = make_geom(desc, &g);
    if (st != GACONV_OK) return st;
    {   // operands that are transposed first: the inner call's scratch, then the transposed copies
        const Relayout R = plan_relayout(desc, method);
        if (R.move_x || R.move_dy) {
            *bytes = align_up(R.inner_bytes, 256) + (R.move_x ? align_up(x_bytes_of(desc), 256) : 0) + (R.move_dy ? dy_bytes_of(g) : 0);
            return GACONV_OK;
        }
    }
    switch (method) {
        case GACONV_METHOD_EXACT: *bytes = exact_layout(g, desc->math, desc->algo).total; return GACONV_OK;
        case GACONV_METHOD_TOP1: *bytes = top1_layout(g).total; return GACONV_OK;
        case GACONV_METHOD_TOPK: {
            const int t = topk_of(desc, g);
            if (t < 1) return GACONV_ERR_BAD_DESC;
            *bytes = topk_layout(g, t).total;
            return GACONV_OK;
        }
        case GACONV_METHOD_ZERO:
        case GACONV_METHOD_RANDOM: *bytes = kWsDataOffset; return GACONV_OK;
    }
    return GACONV_ERR_BAD_DESC;
}

gaconv_status_t gaconv_workspace_init(void* workspace, size_t bytes, void* stream)
{
    if (workspace == nullptr) return GACONV_ERR_NULL_POINTER;
    if (!aligned16(workspace)) return GACONV_ERR_MISALIGNED;
    if (bytes < kWsDataOffset) return GACONV_ERR_WORKSPACE_TOO_SMALL;
    if (cudaMemsetAsync(workspace, 0, kWsDataOffset, static_cast<cudaStream_t>(stream)) != cudaSuccess) return GACONV_ERR_CUDA;
    return GACONV_OK;
}

gaconv_status_t gaconv_dw_exact(const void* x, const void* dy, float* dw, const gaconv_conv_desc_t* desc, void* stream)
{
    Geom g;
    gaconv_status_t st = make_geom(desc, &g);
    if (st != GACONV_OK) return st;
    if (x == nullptr || dy == nullptr || dw == nullptr) return GACONV_ERR_NULL_POINTER;
    if (!aligned16(x) || !aligned16(dy) || !aligned16(dw)) return GACONV_ERR_MISALIGNED;
    if (desc->math == GACONV_MATH_TF32 && g.bf16) return GACONV_ERR_BAD_DESC;
    if (desc->dy_layout == GACONV_DY_NPQK && g.k > 1 && desc->algo != GACONV_ALGO_DIRECT) {
        // Small maps: the tensor-core kernel's dY operand IS the channels-last order (its pre-pass would transpose an
        // N x K x P x Q gradient into it), so a channels-last gradient is read where it lies; only X may have to move.
        const Relayout R = plan_relayout(desc, GACONV_METHOD_EXACT);
        Geom gi;
        if (make_geom(&R.inner, &gi) == GACONV_OK) {
            const ExactLayout Li = exact_layout(gi, desc->math, desc->algo);
            if (Li.tc_ok && Li.tp.reads_transposed_dy) {
                const size_t head = align_up(Li.total, 256);
                st = check_ws(desc, head + (R.move_x ? x_bytes_of(desc) : 0));
                if (st != GACONV_OK) return st;
                char* ws = static_cast<char*>(desc->workspace);
                const void* xs = x;
                if (R.move_x) {
                    if (launch_transpose_batched(x, ws + head, g.c, g.h * g.w, g.n, g.bf16, static_cast<cudaStream_t>(stream)) != cudaSuccess)
                        return GACONV_ERR_CUDA;
                    xs = ws + head;
                }
                cudaError_t e = launch_tc(xs, nullptr, dw, reinterpret_cast<float*>(ws + Li.partial_off), const_cast<void*>(dy),
                                          reinterpret_cast<uint32_t*>(ws + kWsCounterOffset), reinterpret_cast<uint32_t*>(ws), Li.tp,
                                          static_cast<cudaStream_t>(stream));
                return e == cudaSuccess ? GACONV_OK : GACONV_ERR_CUDA;
            }
        }
    }
    {
        gaconv_conv_desc_t inner;
        const void *xt = nullptr, *dyt = nullptr;
        bool moved = false;
        st = relayout_operands(x, dy, desc, GACONV_METHOD_EXACT, static_cast<cudaStream_t>(stream), &inner, &xt, &dyt, &moved);
        if (st != GACONV_OK) return st;
        if (moved) return gaconv_dw_exact(xt, dyt, dw, &inner, stream);
    }
    const ExactLayout L = exact_layout(g, desc->math, desc->algo);
    const bool mma_ok = direct_mma_supported(g, L.dp);
    if (desc->math == GACONV_MATH_TF32 && !mma_ok && !L.tc_ok) return GACONV_ERR_UNSUPPORTED;
    if (desc->algo == GACONV_ALGO_TENSOR && !L.tc_ok) return GACONV_ERR_UNSUPPORTED;
    st = check_ws(desc, L.total);
    if (st != GACONV_OK) return st;
    char* ws = static_cast<char*>(desc->workspace);
    if (L.tc_ok && desc->algo != GACONV_ALGO_DIRECT) {
        cudaError_t e = launch_tc(x, dy, dw, reinterpret_cast<float*>(ws + L.partial_off), ws + L.scratch_off,
                                  reinterpret_cast<uint32_t*>(ws + kWsCounterOffset), reinterpret_cast<uint32_t*>(ws), L.tp,
                                  static_cast<cudaStream_t>(stream));
        return e == cudaSuccess ? GACONV_OK : GACONV_ERR_CUDA;
    }
    if (L.stem_ok && desc->algo != GACONV_ALGO_DIRECT && desc->math == GACONV_MATH_DEFAULT) {
        cudaError_t e = launch_stem(x, dy, dw, reinterpret_cast<float*>(ws + L.partial_off), reinterpret_cast<uint32_t*>(ws), L.sp,
                                    static_cast<cudaStream_t>(stream));
        return e == cudaSuccess ? GACONV_OK : GACONV_ERR_CUDA;
    }
    if (mma_ok && (desc->algo != GACONV_ALGO_DIRECT || desc->math == GACONV_MATH_TF32)) {
        cudaError_t e = launch_direct_mma(x, dy, dw, reinterpret_cast<float*>(ws + L.partial_off), reinterpret_cast<uint32_t*>(ws),
                                          g, L.dp, desc->math != GACONV_MATH_TF32, static_cast<cudaStream_t>(stream));
        return e == cudaSuccess ? GACONV_OK : GACONV_ERR_CUDA;
    }
    cudaError_t e = launch_direct(x, dy, dw, reinterpret_cast<float*>(ws + L.partial_off),
                                  reinterpret_cast<uint32_t*>(ws), g, L.dp,
                                  static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? GACONV_OK : GACONV_ERR_CUDA;
}

gaconv_status_t gaconv_dw_approx(int32_t method, const void* x, const void* dy, float* dw,
                                 const gaconv_conv_desc_t* desc, uint64_t seed, void* stream)
{
    Geom g;
    gaconv_status_t st = make_geom(desc, &g);
    if (st != GACONV_OK) return st;
    if (dw == nullptr) return GACONV_ERR_NULL_POINTER;
    if (!aligned16(dw)) return GACONV_ERR_MISALIGNED;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const size_t count = (size_t)g.k * g.c * g.r * g.s;
    if (method == GACONV_METHOD_ZERO) return launch_zero(dw, count, cs) == cudaSuccess ? GACONV_OK : GACONV_ERR_CUDA;
    if (method == GACONV_METHOD_RANDOM)
        return launch_random(dw, g, seed, desc->rand_std, cs) == cudaSuccess ? GACONV_OK : GACONV_ERR_CUDA;
    if (method != GACONV_METHOD_TOP1 && method != GACONV_METHOD_TOPK) return GACONV_ERR_BAD_DESC;
    if (x == nullptr || dy == nullptr) return GACONV_ERR_NULL_POINTER;
    if (!aligned16(x) || !aligned16(dy)) return GACONV_ERR_MISALIGNED;
    {
        gaconv_conv_desc_t inner;
        const void *xt = nullptr, *dyt = nullptr;
        bool moved = false;
        st = relayout_operands(x, dy, desc, method, cs, &inner, &xt, &dyt, &moved);
        if (st != GACONV_OK) return st;
        if (moved) return gaconv_dw_approx(method, xt, dyt, dw, &inner, seed, stream);
    }
    if (method == GACONV_METHOD_TOPK) {
        // selection of the topk largest magnitudes per map, then the patch accumulation over the retained entries
        const int t = topk_of(desc, g);
        if (t < 1) return GACONV_ERR_BAD_DESC;
        const TopkLayout L = topk_layout(g, t);
        st = check_ws(desc, L.total);
        if (st != GACONV_OK) return st;
        char* ws = static_cast<char*>(desc->workspace);
        int32_t* idx = reinterpret_cast<int32_t*>(ws + L.idx_off);
        float* sum = reinterpret_cast<float*>(ws + L.sum_off);
        if (launch_select_topk(dy, idx, sum, g, t, cs) != cudaSuccess) return GACONV_ERR_CUDA;
        // the one-launch kernel of the top-1 method, fed with the selected list (t records per image), where its
        // shared-memory block fits; else the ticketed gather kernel
        if (top1_fused_supported(g) && (size_t)g.n * t * 16 <= 48 * 1024 && desc->algo != GACONV_ALGO_DIRECT)   // (16 bytes per record)
            return launch_top1_fused(x, dy, dw, g, cs, idx, sum, t) == cudaSuccess ? GACONV_OK : GACONV_ERR_CUDA;
        if (launch_gather(x, idx, sum, dw, reinterpret_cast<float*>(ws + L.partial_off),
                          reinterpret_cast<uint32_t*>(ws + kWsCounterOffset), g, L.gp, t, cs) != cudaSuccess)
            return GACONV_ERR_CUDA;
        return GACONV_OK;
    }
    const Top1Layout L = top1_layout(g);
    st = check_ws(desc, L.total);       // required by every route, so that behaviour does not depend on the kernel picked
    if (st != GACONV_OK) return st;
    char* ws = static_cast<char*>(desc->workspace);
    int32_t* idx = reinterpret_cast<int32_t*>(ws + L.idx_off);
    float* sum = reinterpret_cast<float*>(ws + L.sum_off);
    if (L.dense && desc->algo != GACONV_ALGO_DIRECT) {
        void* sparse = ws + L.sparse_off;
        if (L.tp.reads_transposed_dy) {       // the dense kernel's operand layout is written directly: no separate transpose
            if (launch_select_sparse_transposed(dy, ws + L.scratch_off, g, cs) != cudaSuccess) return GACONV_ERR_CUDA;
            sparse = nullptr;
        } else if (launch_select(dy, idx, sum, sparse, g, cs) != cudaSuccess) return GACONV_ERR_CUDA;
        return launch_tc(x, sparse, dw, reinterpret_cast<float*>(ws + L.partial_off), ws + L.scratch_off,
                         reinterpret_cast<uint32_t*>(ws + kWsCounterOffset), reinterpret_cast<uint32_t*>(ws), L.tp,
                         cs) == cudaSuccess ? GACONV_OK : GACONV_ERR_CUDA;
    }
    if (top1_fused_supported(g) && desc->algo != GACONV_ALGO_DIRECT)
        return launch_top1_fused(x, dy, dw, g, cs) == cudaSuccess ? GACONV_OK : GACONV_ERR_CUDA;
    if (launch_select(dy, idx, sum, nullptr, g, cs) != cudaSuccess) return GACONV_ERR_CUDA;
    if (launch_gather(x, idx, sum, dw, reinterpret_cast<float*>(ws + L.partial_off),
                      reinterpret_cast<uint32_t*>(ws + kWsCounterOffset), g, L.gp, 1, cs) != cudaSuccess)
        return GACONV_ERR_CUDA;
    return GACONV_OK;
}

gaconv_status_t gaconv_approx_select(const void* dy, int32_t* idx, float* sum, void* dy_sparse,
                                     const gaconv_conv_desc_t* desc, void* stream)
{
    Geom g;
    gaconv_status_t st = make_geom(desc, &g);
    if (st != GACONV_OK) return st;
    if (dy == nullptr || idx == nullptr || sum == nullptr) return GACONV_ERR_NULL_POINTER;
    if (desc->dy_layout == GACONV_DY_NPQK && g.k > 1) return GACONV_ERR_UNSUPPORTED;      // selection alone has no scratch to transpose into
    if (!aligned16(dy) || !aligned16(idx) || !aligned16(sum) || !aligned16(dy_sparse)) return GACONV_ERR_MISALIGNED;
    return launch_select(dy, idx, sum, dy_sparse, g, static_cast<cudaStream_t>(stream)) == cudaSuccess ? GACONV_OK
                                                                                                         : GACONV_ERR_CUDA;
}

gaconv_status_t gaconv_approx_select_topk(const void* dy, int32_t* idx, float* sum, const gaconv_conv_desc_t* desc, void* stream)
{
    Geom g;
    gaconv_status_t st = make_geom(desc, &g);
    if (st != GACONV_OK) return st;
    if (dy == nullptr || idx == nullptr || sum == nullptr) return GACONV_ERR_NULL_POINTER;
    if (desc->dy_layout == GACONV_DY_NPQK && g.k > 1) return GACONV_ERR_UNSUPPORTED;
    if (!aligned16(dy) || !aligned16(idx) || !aligned16(sum)) return GACONV_ERR_MISALIGNED;
    const int t = topk_of(desc, g);
    if (t < 1) return GACONV_ERR_BAD_DESC;
    return launch_select_topk(dy, idx, sum, g, t, static_cast<cudaStream_t>(stream)) == cudaSuccess ? GACONV_OK : GACONV_ERR_CUDA;
}

static gaconv_status_t dw_from_host(int32_t method, const void* x_host, const void* dy_host, float* dw_host,
                                    void* x_dev, void* dy_dev, float* dw_dev, const gaconv_conv_desc_t* desc,
                                    uint64_t seed, void* stream, bool wait)
{
    Geom g;
    gaconv_status_t st = make_geom(desc, &g);
    if (st != GACONV_OK) return st;
    if (dw_host == nullptr || dw_dev == nullptr) return GACONV_ERR_NULL_POINTER;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const bool needs_inputs = method == GACONV_METHOD_EXACT || method == GACONV_METHOD_TOP1 || method == GACONV_METHOD_TOPK;
    // everything the compute call would reject is rejected here, before the first copy is enqueued
    if (method < GACONV_METHOD_EXACT || method > GACONV_METHOD_TOPK) return GACONV_ERR_BAD_DESC;
    if (!aligned16(dw_dev)) return GACONV_ERR_MISALIGNED;
    if (needs_inputs) {
        // both host inputs NULL: the staging buffers already hold this layer's inputs (an earlier call of the step copied them)
        if ((x_host == nullptr) != (dy_host == nullptr) || x_dev == nullptr || dy_dev == nullptr) return GACONV_ERR_NULL_POINTER;
        if (!aligned16(x_dev) || !aligned16(dy_dev)) return GACONV_ERR_MISALIGNED;
        if (method == GACONV_METHOD_EXACT && desc->math == GACONV_MATH_TF32 && g.bf16) return GACONV_ERR_BAD_DESC;
        size_t need = 0;
        st = gaconv_workspace_size(desc, method, &need);
        if (st != GACONV_OK) return st;
        st = check_ws(desc, need);
        if (st != GACONV_OK) return st;
        if (method == GACONV_METHOD_EXACT) {
            const ExactLayout L = exact_layout(g, desc->math, desc->algo);
            if (desc->math == GACONV_MATH_TF32 && !direct_mma_supported(g, L.dp) && !L.tc_ok) return GACONV_ERR_UNSUPPORTED;
            if (desc->algo == GACONV_ALGO_TENSOR && !L.tc_ok) return GACONV_ERR_UNSUPPORTED;
        }
        const size_t eb = g.bf16 ? 2 : 4;
        if (x_host != nullptr &&
            (cudaMemcpyAsync(x_dev, x_host, (size_t)g.n * g.c * g.h * g.w * eb, cudaMemcpyHostToDevice, cs) != cudaSuccess ||
             cudaMemcpyAsync(dy_dev, dy_host, (size_t)g.n * g.k * g.p * g.q * eb, cudaMemcpyHostToDevice, cs) != cudaSuccess))
            return GACONV_ERR_CUDA;
    }
    st = method == GACONV_METHOD_EXACT ? gaconv_dw_exact(x_dev, dy_dev, dw_dev, desc, stream)
                                       : gaconv_dw_approx(method, x_dev, dy_dev, dw_dev, desc, seed, stream);
    if (st != GACONV_OK) return st;
    if (cudaMemcpyAsync(dw_host, dw_dev, (size_t)g.k * g.c * g.r * g.s * sizeof(float), cudaMemcpyDeviceToHost, cs) != cudaSuccess)
        return GACONV_ERR_CUDA;
    if (!wait) return GACONV_OK;
    return cudaStreamSynchronize(cs) == cudaSuccess ? GACONV_OK : GACONV_ERR_CUDA;
}

gaconv_status_t gaconv_dw_from_host(int32_t method, const void* x_host, const void* dy_host, float* dw_host,
                                    void* x_dev, void* dy_dev, float* dw_dev, const gaconv_conv_desc_t* desc,
                                    uint64_t seed, void* stream)
{
    return dw_from_host(method, x_host, dy_host, dw_host, x_dev, dy_dev, dw_dev, desc, seed, stream, true);
}

gaconv_status_t gaconv_dw_from_host_async(int32_t method, const void* x_host, const void* dy_host, float* dw_host,
                                          void* x_dev, void* dy_dev, float* dw_dev, const gaconv_conv_desc_t* desc,
                                          uint64_t seed, void* stream)
{
    return dw_from_host(method, x_host, dy_host, dw_host, x_dev, dy_dev, dw_dev, desc, seed, stream, false);
}

gaconv_status_t gaconv_poll_async_status(const gaconv_conv_desc_t* desc, void* stream)
{
    if (desc == nullptr || desc->workspace == nullptr) return GACONV_ERR_NULL_POINTER;
    if (desc->workspace_bytes < kWsDataOffset) return GACONV_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    uint32_t word = 0;
    if (cudaMemcpyAsync(&word, desc->workspace, sizeof(word), cudaMemcpyDeviceToHost, cs) != cudaSuccess) return GACONV_ERR_CUDA;
    if (cudaStreamSynchronize(cs) != cudaSuccess) return GACONV_ERR_CUDA;
    if (word == 0) return GACONV_OK;
    if (cudaMemsetAsync(desc->workspace, 0, sizeof(word), cs) != cudaSuccess) return GACONV_ERR_CUDA;
    return GACONV_ERR_TIMEOUT;
}

// ---- approximation schedules ----------------------------------------------------------------

gaconv_status_t gaconv_schedule_create(gaconv_schedule_t** out, int32_t num_layers, int32_t kind, int32_t method,
                                       double fraction, uint64_t seed)
{
    if (out == nullptr) return GACONV_ERR_NULL_POINTER;
    *out = nullptr;
    if (num_layers < 1 || num_layers > (1 << 20)) return GACONV_ERR_BAD_DESC;
    if (kind < GACONV_SCHED_EVERY_4TH_LAYER || kind > GACONV_SCHED_SEEDED_FRACTION_ALT_BATCH) return GACONV_ERR_BAD_DESC;
    if (method != GACONV_METHOD_ZERO && method != GACONV_METHOD_RANDOM && method != GACONV_METHOD_TOP1 && method != GACONV_METHOD_TOPK)
        return GACONV_ERR_BAD_DESC;
    if (!(fraction >= 0.0 && fraction <= 1.0)) return GACONV_ERR_BAD_DESC;
    gaconv_schedule* s = new (std::nothrow) gaconv_schedule{num_layers, kind, method, fraction, seed, nullptr};
    if (s == nullptr) return GACONV_ERR_BAD_DESC;
    if (kind == GACONV_SCHED_SEEDED_FRACTION_ALT_BATCH) {
        s->mask = new (std::nothrow) bool[num_layers]();
        uint64_t* hash = new (std::nothrow) uint64_t[num_layers];
        if (s->mask == nullptr || hash == nullptr) { delete[] s->mask; delete[] hash; delete s; return GACONV_ERR_BAD_DESC; }
        for (int l = 0; l < num_layers; ++l) hash[l] = splitmix64(seed + (uint64_t)l);
        int m = (int)(fraction * num_layers + 0.5);
        if (m > num_layers) m = num_layers;
        // a layer is chosen when fewer than m layers precede it in (hash, index) order
        for (int l = 0; l < num_layers; ++l) {
            int before = 0;
            for (int o = 0; o < num_layers; ++o)
                if (hash[o] < hash[l] || (hash[o] == hash[l] && o < l)) ++before;
            s->mask[l] = before < m;
        }
        delete[] hash;
    }
    *out = s;
    return GACONV_OK;
}

int32_t gaconv_schedule_method(const gaconv_schedule_t* s, int32_t layer, int64_t step)
{
    if (s == nullptr || layer < 0 || layer >= s->num_layers || step < 0) return -2;
    const int one_based = layer + 1;
    bool approx = false;
    switch (s->kind) {
        case GACONV_SCHED_EVERY_4TH_LAYER: approx = one_based >= 2 && (one_based - 2) % 4 == 0; break;
        case GACONV_SCHED_ALT_LAYER_ALT_BATCH: approx = one_based % 2 == 0 && step % 2 == 1; break;
        case GACONV_SCHED_ALL_LAYERS_EVERY_4TH_BATCH: approx = step % 4 == 3; break;
        case GACONV_SCHED_LAYER2_ALT_BATCH: approx = one_based == 2 && step % 2 == 1; break;
        case GACONV_SCHED_SEEDED_FRACTION_ALT_BATCH: approx = step % 2 == 1 && s->mask[layer]; break;
    }
    return approx ? s->method : GACONV_METHOD_EXACT;
}

gaconv_status_t gaconv_schedule_run_layer(const gaconv_schedule_t* s, int32_t layer, int64_t step, const void* x,
                                          const void* dy, float* dw, const gaconv_conv_desc_t* desc, void* stream)
{
    const int32_t m = gaconv_schedule_method(s, layer, step);
    if (m == -2) return GACONV_ERR_BAD_DESC;
    if (m == GACONV_METHOD_EXACT) return gaconv_dw_exact(x, dy, dw, desc, stream);
    const uint64_t seed = splitmix64(s->seed ^ splitmix64((uint64_t)step * 0x100000001B3ull + (uint64_t)layer));
    return gaconv_dw_approx(m, x, dy, dw, desc, seed, stream);
}

// ---- lanes: side streams on which the layers of a step run next to one another ----------------------
namespace {

constexpr int kMaxLanes = 16, kMaxLaneDevices = 64;
struct LanePool {
    bool ready = false;
    cudaStream_t side[kMaxLanes - 1] = {};
    cudaEvent_t fork = nullptr, join[kMaxLanes - 1] = {};
};
std::mutex g_lane_mutex;
LanePool g_lanes[kMaxLaneDevices];

// streams and events of the current device, created on first use (host objects; no device memory)
LanePool* lane_pool()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxLaneDevices) return nullptr;
    LanePool& p = g_lanes[dev];
    if (!p.ready) {
        if (cudaEventCreateWithFlags(&p.fork, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        for (int i = 0; i < kMaxLanes - 1; ++i)
            if (cudaStreamCreateWithFlags(&p.side[i], cudaStreamNonBlocking) != cudaSuccess ||
                cudaEventCreateWithFlags(&p.join[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
        p.ready = true;
    }
    return &p;
}

}  // namespace

gaconv_status_t gaconv_schedule_run_step(const gaconv_schedule_t* s, int64_t step, int32_t num_layers, const void* const* x,
                                         const void* const* dy, float* const* dw, const gaconv_conv_desc_t* const* descs,
                                         int32_t lanes, void* stream)
{
    if (s == nullptr || x == nullptr || dy == nullptr || dw == nullptr || descs == nullptr) return GACONV_ERR_NULL_POINTER;
    if (num_layers < 1 || num_layers > s->num_layers || step < 0 || lanes < 1 || lanes > kMaxLanes) return GACONV_ERR_BAD_DESC;
    for (int l = 0; l < num_layers; ++l) {
        if (descs[l] == nullptr) return GACONV_ERR_NULL_POINTER;
        // layers that run next to one another must not share scratch
        if (lanes > 1 && descs[l]->workspace != nullptr)
            for (int o = 0; o < l; ++o)
                if (descs[o]->workspace == descs[l]->workspace) return GACONV_ERR_BAD_DESC;
    }
    cudaStream_t main_stream = static_cast<cudaStream_t>(stream);
    if (lanes == 1 || num_layers == 1) {
        for (int l = 0; l < num_layers; ++l) {
            const gaconv_status_t st = gaconv_schedule_run_layer(s, l, step, x[l], dy[l], dw[l], descs[l], stream);
            if (st != GACONV_OK) return st;
        }
        return GACONV_OK;
    }
    std::lock_guard<std::mutex> lock(g_lane_mutex);          // one set of lanes per device: enqueueing is serialised
    LanePool* pool = lane_pool();
    if (pool == nullptr) return GACONV_ERR_CUDA;
    const int used = lanes < num_layers ? lanes : num_layers;
    // fork: the side streams start after everything already enqueued on the caller's stream
    if (cudaEventRecord(pool->fork, main_stream) != cudaSuccess) return GACONV_ERR_CUDA;
    for (int i = 0; i < used - 1; ++i)
        if (cudaStreamWaitEvent(pool->side[i], pool->fork, 0) != cudaSuccess) return GACONV_ERR_CUDA;
    gaconv_status_t result = GACONV_OK;
    for (int l = 0; l < num_layers && result == GACONV_OK; ++l) {
        const int lane = l % used;
        result = gaconv_schedule_run_layer(s, l, step, x[l], dy[l], dw[l], descs[l], lane == 0 ? stream : static_cast<void*>(pool->side[lane - 1]));
    }
    // join (also after an error, so that the side streams never stay forked from a capturing stream)
    for (int i = 0; i < used - 1; ++i)
        if (cudaEventRecord(pool->join[i], pool->side[i]) != cudaSuccess || cudaStreamWaitEvent(main_stream, pool->join[i], 0) != cudaSuccess)
            return GACONV_ERR_CUDA;
    return result;
}

void gaconv_schedule_destroy(gaconv_schedule_t* s)
{
    if (s == nullptr) return;
    delete[] s->mask;
    delete s;
}

}  // extern "C"
