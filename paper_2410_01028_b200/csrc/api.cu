// Host side of libasd: workspace layout, pass scheduling under the skip mask, Algorithm 1, the decode loops
// and the C ABI declared in include/asd.h.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <mutex>
#include <string>
#include <vector>

#include "../../include/asd.h"
#include "common.cuh"
#include "pass.cuh"
#include "prefill.h"
#include "sample.h"

namespace asd {

constexpr int kPrefillRows = kPassMaxRows;  // prompt rows per pass of the chunked prefill
constexpr size_t kAlign = 256;
constexpr int kMaxGemvGrid = 1024;
constexpr long long kShortWaitCycles = 2000000LL;  // ASD_DEBUG_SHORT_WAITS: about a millisecond per wait

static size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

// ---------------------------------------------------------------- shared-memory budgets
size_t gemv_smem_bytes(int M, int n_rows, int n_in, int grid, bool x_in_smem) {
    const size_t n_pairs = ((size_t)n_rows + 1) / 2;
    const size_t max_np = (n_pairs + grid - 1) / grid;
    const size_t n_seg = ((size_t)n_in + kSeg - 1) / kSeg;
    size_t psum = (max_np * n_seg * 2 * M + 3) & ~(size_t)3;
    size_t b = (size_t)kGemvWarps * kMaxRows * 4 * 4 + 16 + psum * 4;
    if (x_in_smem) b += (size_t)M * n_in * 2;
    return b;
}
static cudaError_t launch_gemv(int M, int epi, bool norm, const GemvParams& p, int grid, size_t smem, cudaStream_t s) {
    switch (M) {
        case 1: return launch_gemv_m1(epi, norm, p, grid, smem, s);
        case 2: return launch_gemv_m2(epi, norm, p, grid, smem, s);
        case 3: return launch_gemv_m3(epi, norm, p, grid, smem, s);
        case 4: return launch_gemv_m4(epi, norm, p, grid, smem, s);
        case 5: return launch_gemv_m5(epi, norm, p, grid, smem, s);
        case 6: return launch_gemv_m6(epi, norm, p, grid, smem, s);
        case 7: return launch_gemv_m7(epi, norm, p, grid, smem, s);
        case 8: return launch_gemv_m8(epi, norm, p, grid, smem, s);
        case 9: return launch_gemv_m9(epi, norm, p, grid, smem, s);
    }
    return cudaErrorInvalidValue;
}
static cudaError_t launch_pass(int M, const PassParams& p, int grid, size_t smem, cudaStream_t s) {
    switch (M) {
        case 1: return launch_pass_m1(p, grid, smem, s);
        case 2: return launch_pass_m2(p, grid, smem, s);
        case 3: return launch_pass_m3(p, grid, smem, s);
        case 4: return launch_pass_m4(p, grid, smem, s);
        case 5: return launch_pass_m5(p, grid, smem, s);
        case 6: return launch_pass_m6(p, grid, smem, s);
        case 7: return launch_pass_m7(p, grid, smem, s);
        case 8: return launch_pass_m8(p, grid, smem, s);
        case 9: return launch_pass_m9(p, grid, smem, s);
        case 16: return launch_pass_m16(p, grid, smem, s);
    }
    return cudaErrorInvalidValue;
}

// per-device facts and one-time kernel configuration
struct DeviceInfo {
    bool ready = false;
    int num_sms = 0, max_smem = 0;
};
static DeviceInfo g_dev[64];
static std::mutex g_dev_mutex;  // first calls from several host threads set the per-device records up one at a time

static cudaError_t device_info(DeviceInfo** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    DeviceInfo& d = g_dev[dev];
    if (!d.ready) {
        if ((e = cudaDeviceGetAttribute(&d.num_sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
        if ((e = cudaDeviceGetAttribute(&d.max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev)) != cudaSuccess) return e;
        if ((e = configure_m1(d.max_smem)) != cudaSuccess) return e;
        if ((e = configure_m2(d.max_smem)) != cudaSuccess) return e;
        if ((e = configure_m3(d.max_smem)) != cudaSuccess) return e;
        if ((e = configure_m4(d.max_smem)) != cudaSuccess) return e;
        if ((e = configure_m5(d.max_smem)) != cudaSuccess) return e;
        if ((e = configure_m6(d.max_smem)) != cudaSuccess) return e;
        if ((e = configure_m7(d.max_smem)) != cudaSuccess) return e;
        if ((e = configure_m8(d.max_smem)) != cudaSuccess) return e;
        if ((e = configure_m9(d.max_smem)) != cudaSuccess) return e;
        if ((e = configure_m16(d.max_smem)) != cudaSuccess) return e;
        if ((e = configure_prefill(d.max_smem)) != cudaSuccess) return e;
        d.ready = true;
    }
    *out = &d;
    return cudaSuccess;
}

// Choose the launch shape of one fused GEMV: one CTA per SM; more CTAs only when the per-CTA partial-sum
// buffer would not fit in shared memory; activations fall back to L1 reads when they do not fit.
static bool plan_gemv(const DeviceInfo& dv, int M, int n_rows, int n_in, bool norm, int* grid, int* x_in_smem, size_t* smem) {
    for (int g = dv.num_sms; g <= kMaxGemvGrid; g += dv.num_sms) {
        size_t b = gemv_smem_bytes(M, n_rows, n_in, g, true);
        if (b <= (size_t)dv.max_smem) {
            *grid = g, *x_in_smem = 1, *smem = b;
            return true;
        }
        if (!norm) {
            b = gemv_smem_bytes(M, n_rows, n_in, g, false);
            if (b <= (size_t)dv.max_smem) {
                *grid = g, *x_in_smem = 0, *smem = b;
                return true;
            }
        }
    }
    return false;
}

// Shared-memory plan of the persistent pass kernel for M rows: ring slots, barriers, reduction scratch,
// per-pair partial sums, activation window / attention scratch.
struct PassPlan {
    int ns, attn_groups, off_bars, off_misc, off_psum, off_reg_a, xs_bytes;
    size_t smem;
};

static bool plan_pass(const DeviceInfo& dv, const asd_config& c, int M, PassPlan* pl) {
    const int kvd = c.n_kv_heads * c.head_dim;
    const long long max_rows = std::max<long long>(std::max(c.vocab, 2 * c.d_ffn), std::max(c.d_model + 2 * kvd, c.d_model));
    const long long np_max = ((max_rows + 1) / 2 + dv.num_sms - 1) / dv.num_sms + 2;
    if ((max_rows + 1) / 2 * dv.num_sms >= (1LL << 31)) return false;  // the kernel splits a matrix's pairs over the CTAs in 32-bit arithmetic
    // per-pair partial sums; when a CTA has fewer than 8 groups of 8 pairs up to 15 warps keep copies (at most 15 / groups
    // copies of at most 8 * groups pairs: 120 pairs in all)
    const size_t psum = ((size_t)std::max<long long>(np_max, 120) * 2 * M * 4 + 15) & ~(size_t)15;
    const size_t misc = ((size_t)16 * kPassMaxRows * 4 * 4 + 32 + 64 * 4 + 8 * 4 * 4 + 15) & ~(size_t)15;  // reduction scratch, flags, slot generations, split table
    const size_t attn_scratch = ((size_t)M * c.head_dim * 4 + (size_t)M * kAttnChunk * 4 + 4 * kPassMaxRows * 4 + 16 + 15) & ~(size_t)15;
    // Activation window: the longest reduction dimension (in segments of 256 inputs) cut into as few windows as leave
    // the ring 20 slots. Every further window costs a stage of a multi-row pass a block-wide refill, every slot less
    // costs bandwidth (one row, 7B shape: 24 slots 0.402 ms per 4 layers, 21: 0.409, 16: 0.422, 12: 0.481); 20 was the
    // best trade for three and four rows (measured again with 22 and 24 after the kernel had changed: four and five rows
    // 0.7 % slower). Windows do not get shorter than a row of d_model while that leaves 16 slots: the RMSNorm stages want
    // their rows whole (six to nine rows: 1-2.5 % faster than with W_d's row cut into equal parts). One row always fits whole.
    const size_t seg_max = ((size_t)std::max(c.d_model, c.d_ffn) + kSegK - 1) / kSegK;
    const size_t seg_norm = ((size_t)c.d_model + kSegK - 1) / kSegK;  // the RMSNorm stages want their rows whole in the window
    const long long fixed = 1024 + (long long)(psum + misc) + 2 * 64 * 8;
    size_t wseg_plan = seg_max;
    auto leaves_ring = [&](size_t wseg, long long slots) {
        const size_t bytes = (size_t)M * (wseg * kSegK + kXsPad) * 2;
        return (long long)dv.max_smem - fixed - (long long)((bytes + 15) & ~(size_t)15) >= slots * kSlotBytes;
    };
    for (size_t nw = 1; nw <= seg_max; ++nw) {
        wseg_plan = (seg_max + nw - 1) / nw;
        if (leaves_ring(wseg_plan, 20)) break;
    }
    // not shorter than a row of d_model while the ring keeps 16 slots: the RMSNorm stages want their rows whole
    if (wseg_plan < seg_norm && leaves_ring(seg_norm, 16)) wseg_plan = seg_norm;
    const int xs_bytes = (int)((size_t)M * (wseg_plan * kSegK + kXsPad) * 2);
    const size_t xs = (size_t)M * ((size_t)pass_wseg(M, xs_bytes) * kSegK + kXsPad) * 2;
    // up to three groups of four warps work on attention items, as many as their scratch fits the window's bytes
    const int groups_by_scratch = (int)std::max<size_t>(1, std::min<size_t>(3, (size_t)kXsBudget / attn_scratch));
    const size_t reg_a = (std::max(xs, groups_by_scratch * attn_scratch) + 15) & ~(size_t)15;
    const long long avail = (long long)dv.max_smem - 1024 - (long long)(psum + misc + reg_a) - 2 * 64 * 8;
    int ns = (int)std::min<long long>(64, avail / kSlotBytes);
    const int tile_slots = (kAttnChunk / kBoxKeys) * std::max(1, c.head_dim / 64);
    if (ns < 2 * tile_slots || ns < 8) return false;
    pl->ns = ns;
    pl->xs_bytes = xs_bytes;
    pl->attn_groups = std::max(1, std::min(groups_by_scratch, ns / (2 * tile_slots)));
    pl->off_bars = ns * kSlotBytes;
    pl->off_misc = pl->off_bars + 2 * 64 * 8;
    pl->off_psum = pl->off_misc + (int)misc;
    pl->off_reg_a = pl->off_psum + (int)psum;
    pl->smem = (size_t)pl->off_reg_a + reg_a + 1024;
    return pl->smem <= (size_t)dv.max_smem;
}

// ---------------------------------------------------------------- workspace layout
struct Layout {
    size_t embed, lm_head, final_norm, layers, layer_stride;
    size_t l_attn_norm, l_wqkv, l_wo, l_mlp_norm, l_wgu, l_wd;  // offsets inside one layer block
    size_t rope_cos, rope_sin, kcache, vcache, kv_layer_stride;
    size_t x, q, a, t, xl, al, tl, ql, kl, vl, pl_acc, pl_ml, part_acc, part_ml, partials, counters, cosv, sumcos;
    size_t tok_in, draft_toks, gen_toks, prompt_toks, argmax, accept, logits, probs_p, probs_q;
    size_t stage_tab, tmaps, sync_words, trace, resid_tab;
    int max_stages;
    size_t total;
    int chunk_stride;
    // dense prompt path: row-major copies of the sublayer matrices (one block per layer) and activations of a chunk
    size_t rm_layers, rm_layer_stride, rm_wqkv, rm_wo, rm_wgu, rm_wd;
    size_t pf_x, pf_xn, pf_q, pf_a, pf_t, pf_c, pf_cos;  // pf_c: two buffers (the halves of a product cut along its reduction dimension)
    int pf_rows;  // prompt rows per chunk of the dense path (0: shape not supported by it)
};

constexpr int kPrefillChunk = 2048;      // most prompt rows one chunk of the dense prompt path holds
constexpr int kPrefillGemmMinRows = 32;  // shorter prompts take the row passes (default mode)

// the dense prompt path needs whole 32-column groups inside a head (rotary epilogue) and a flash kernel for head_dim
static bool dense_prefill_supported(const asd_config& c) { return c.n_layers > 0 && (c.head_dim == 64 || c.head_dim == 128); }

static bool check_config(const asd_config& c) {
    if (c.n_layers < 0 || c.d_model <= 0 || c.n_heads <= 0 || c.n_kv_heads <= 0 || c.head_dim <= 0 || c.d_ffn <= 0 ||
        c.vocab <= 0 || c.max_seq <= 0)
        return false;
    if ((long long)c.n_heads * c.head_dim != c.d_model || c.n_heads % c.n_kv_heads) return false;
    if ((c.head_dim != 16 && c.head_dim != 32 && c.head_dim != 64 && c.head_dim != 128 && c.head_dim != 256) || c.d_model % 8 ||
        c.d_ffn % 8)
        return false;
    if (c.max_draft < 0 || c.max_draft > kMaxRows - 1) return false;
    if (!(c.rms_eps >= 0.f) || !(c.rope_theta > 0.f)) return false;
    return true;
}

// bytes of a matrix in the packed layout of the pass kernel: (pairs of rows) x (column blocks of 32 inputs) x 128 bytes
static size_t packed_bytes(size_t n_rows, size_t n_in) { return ((n_rows + 1) / 2) * ((n_in + 31) / 32) * (size_t)128; }

static Layout make_layout(const asd_config& c) {
    Layout L{};
    const size_t d = c.d_model, f = c.d_ffn, V = c.vocab, kvd = (size_t)c.n_kv_heads * c.head_dim, S = c.max_seq;
    size_t o = 0;
    auto take = [&](size_t bytes) {
        size_t at = o;
        o = align_up(o + bytes);
        return at;
    };
    L.embed = take(V * d * 2);
    L.lm_head = take(packed_bytes(V, d));
    L.final_norm = take(d * 2);
    {
        size_t lo = 0;
        auto ltake = [&](size_t bytes) {
            size_t at = lo;
            lo = align_up(lo + bytes);
            return at;
        };
        L.l_attn_norm = ltake(d * 2);
        L.l_wqkv = ltake(packed_bytes(d + 2 * kvd, d));
        L.l_wo = ltake(packed_bytes(d, d));
        L.l_mlp_norm = ltake(d * 2);
        L.l_wgu = ltake(packed_bytes(2 * f, d));
        L.l_wd = ltake(packed_bytes(d, f));
        L.layer_stride = lo;
    }
    L.layers = take(L.layer_stride * c.n_layers);
    L.rope_cos = take(S * (c.head_dim / 2) * 4);
    L.rope_sin = take(S * (c.head_dim / 2) * 4);
    L.kv_layer_stride = align_up(S * kvd * 2);
    L.kcache = take(L.kv_layer_stride * c.n_layers);
    L.vcache = take(L.kv_layer_stride * c.n_layers);
    L.x = take(kPassMaxRows * d * 4);
    L.q = take(kPassMaxRows * d * 2);
    L.a = take(kPassMaxRows * d * 2);
    L.t = take(kPassMaxRows * f * 2);
    // the same activations as (value, tag) words for the one-row passes (see pass.cuh, "tagged handoff")
    L.xl = take((size_t)2 * d * 8);
    L.al = take((size_t)2 * (d / 2) * 8);
    L.tl = take((size_t)2 * (f / 2) * 8);
    L.chunk_stride = (int)((S + kAttnChunk - 1) / kAttnChunk);
    L.ql = take((size_t)d * 8);
    L.kl = take((size_t)kvd * 8);
    L.vl = take((size_t)kvd * 8);
    L.pl_acc = take((size_t)c.n_heads * L.chunk_stride * c.head_dim * 8);
    L.pl_ml = take((size_t)c.n_heads * L.chunk_stride * 2 * 8);
    L.part_acc = take((size_t)c.n_heads * L.chunk_stride * kPassMaxRows * c.head_dim * 4);
    L.part_ml = take((size_t)c.n_heads * L.chunk_stride * kPassMaxRows * 2 * 4);
    L.partials = take((size_t)(2 * c.n_layers + 1) * kMaxGemvGrid * kPassMaxRows * 4 * 4);
    L.counters = take((size_t)(c.n_kv_heads + 64) * 4);
    L.cosv = take((size_t)2 * std::max(c.n_layers, 1) * kPassMaxRows * 4);
    L.sumcos = take((size_t)2 * std::max(c.n_layers, 1) * 8);
    L.tok_in = take(64 * 4);
    L.draft_toks = take(64 * 4);
    L.gen_toks = take((S + 16) * 4);
    L.prompt_toks = take((S + 16) * 4);
    L.argmax = take(64 * 4);
    L.accept = take(64 * 4);
    L.logits = take((size_t)kPassMaxRows * V * 4);
    L.probs_p = take((size_t)kMaxRows * V * 8);  // sampling: the full model's distributions of a verify pass
    L.probs_q = take((size_t)kMaxRows * V * 8);  // sampling: the draft model's distributions of this round's draft steps
    L.max_stages = 5 * c.n_layers + 3;
    L.stage_tab = take((size_t)3 * L.max_stages * sizeof(StageDesc));
    L.tmaps = take((size_t)2 * std::max(c.n_layers, 1) * sizeof(CUtensorMap));
    L.sync_words = take(256);
    L.resid_tab = take((size_t)2 * (2 * std::max(c.n_layers, 1)) * sizeof(ResidOut));
    L.trace = take((size_t)L.max_stages * kTraceEntries * kMaxGemvGrid * 8);
    L.pf_rows = 0;
    if (dense_prefill_supported(c)) {
        L.pf_rows = (int)std::min<size_t>(kPrefillChunk, (S + kGemmBM - 1) / kGemmBM * kGemmBM);
        const size_t R = L.pf_rows;
        size_t lo = 0;
        auto ltake = [&](size_t bytes) {
            size_t at = lo;
            lo = align_up(lo + bytes);
            return at;
        };
        L.rm_wqkv = ltake((d + 2 * kvd) * d * 2);
        L.rm_wo = ltake(d * d * 2);
        L.rm_wgu = ltake(2 * f * d * 2);
        L.rm_wd = ltake(d * f * 2);
        L.rm_layer_stride = lo;
        L.rm_layers = take(L.rm_layer_stride * c.n_layers);
        L.pf_x = take(R * d * 4);
        L.pf_xn = take(R * d * 2);
        L.pf_q = take(R * d * 2);
        L.pf_a = take(R * d * 2);
        L.pf_t = take(R * f * 2);
        L.pf_c = take((size_t)2 * R * d * 4);
        L.pf_cos = take((size_t)2 * c.n_layers * R * 4);
    }
    L.total = o;
    return L;
}

}  // namespace asd

using namespace asd;

// ---------------------------------------------------------------- context
struct asd_ctx {
    asd_config c;
    Layout lay;
    unsigned char* ws = nullptr;
    cudaStream_t stream = nullptr;
    DeviceInfo* dev = nullptr;
    int kv_dim = 0;
    bool have_weights = false;
    int n_committed = 0, draft_cursor = 0;
    std::vector<uint8_t> skip_attn, skip_mlp;
    int64_t n_sim_rows = 0;
    // running similarities (ASD_RUNNING_C): sums over the rows committed after the prompt, kept on the host
    bool running_c = false;
    std::vector<double> run_attn, run_mlp;
    int64_t n_run_rows = 0;
    int last_M = 0;
    bool debug_logits = false, last_has_logits = false, last_had_lm_head = false, trace = false;
    bool short_waits = false, inject_missing_arrival = false;  // test hooks of the bounded device waits (asd_set_debug)
    bool no_tagged_handoff = false;  // asd_set_debug: one-row passes use the grid barrier like the others
    // sampling (temperature > 0): every token is drawn; the draft steps of a round keep their distributions for the verify
    double temperature = 0.0;
    uint64_t seed = 0;
    std::vector<int32_t> drafted;  // tokens drawn by the single-step draft calls of this round (host copy)
    bool dev_failed = false;     // a kernel gave up waiting: nothing more is launched until asd_reset
    std::string dev_failed_msg;
    int last_n_stages = 0;
    int prefill_mode = ASD_PREFILL_AUTO;
    // tensor maps of the dense prompt path (host copies, passed to the kernels by value): activations with boxes of
    // 64 x 128, and per layer the four matrices with boxes of 64 x 128 ([0..3]) and 64 x 256 ([4..7])
    CUtensorMap tm_xn{}, tm_a{}, tm_t{};
    std::vector<CUtensorMap> tm_w;
    asd_stats stats{};
    int32_t* pinned = nullptr;  // small host staging buffer
    uint32_t bar_base = 0;      // value of the grid-barrier counter at the start of the next pass
    uint32_t pass_tag = 0x1000; // tag of stage 0 of the next pass in the tagged handoff buffers (never 0: the workspace starts zeroed)
    int n_stages_full = 0, n_stages_draft = 0, n_resid_full = 0, n_resid_draft = 0;
    std::vector<cudaEvent_t> events;
    size_t events_used = 0;
    struct Span { int kind; size_t e0, e1; };
    std::vector<Span> spans;
    std::string err;

    template <class T>
    T* at(size_t off) const { return reinterpret_cast<T*>(ws + off); }
    unsigned char* layer(int l) const { return ws + lay.layers + (size_t)l * lay.layer_stride; }
};

enum { SPAN_PREFILL, SPAN_FULL, SPAN_DRAFT, SPAN_VERIFY };

static int fail(asd_ctx* x, int code, const std::string& what) {
    if (x) x->err = what;
    return code;
}
#define ASD_CUDA(x, expr)                                                                             \
    do {                                                                                              \
        cudaError_t e__ = (expr);                                                                     \
        if (e__ != cudaSuccess)                                                                       \
            return fail((x), ASD_ERR_CUDA, std::string(#expr) + ": " + cudaGetErrorString(e__));      \
    } while (0)

static int new_event(asd_ctx* x, size_t* idx) {
    if (x->events_used == x->events.size()) {
        cudaEvent_t e;
        ASD_CUDA(x, cudaEventCreate(&e));
        x->events.push_back(e);
    }
    *idx = x->events_used++;
    ASD_CUDA(x, cudaEventRecord(x->events[*idx], x->stream));
    return ASD_OK;
}

// turn the recorded spans into statistics; requires the stream to be idle
static int resolve_spans(asd_ctx* x) {
    for (const auto& s : x->spans) {
        float ms = 0.f;
        ASD_CUDA(x, cudaEventElapsedTime(&ms, x->events[s.e0], x->events[s.e1]));
        switch (s.kind) {
            case SPAN_PREFILL: x->stats.ms_prefill += ms; break;
            case SPAN_FULL: x->stats.ms_full += ms; break;
            case SPAN_DRAFT: x->stats.ms_draft += ms; break;
            case SPAN_VERIFY: x->stats.ms_verify += ms; break;
        }
    }
    x->spans.clear();
    x->events_used = 0;
    return ASD_OK;
}

// ---------------------------------------------------------------- stage tables and tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// bf16 matrix [rows, inner] row-major as a GEMM operand: boxes of 64 x box_rows elements, 128-byte swizzle, zeros
// outside the matrix
static bool encode_operand_map(EncodeTiledFn encode, CUtensorMap* m, void* base, size_t inner, size_t rows, uint32_t box_rows) {
    const cuuint64_t gdim[2] = {(cuuint64_t)inner, (cuuint64_t)rows};
    const cuuint64_t gstride[1] = {(cuuint64_t)inner * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kGemmBK, box_rows};
    const cuuint32_t estr[2] = {1u, 1u};
    return encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static EncodeTiledFn tensor_map_encoder() {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess)
        return nullptr;
    return reinterpret_cast<EncodeTiledFn>(fn);
}

// One 2-D tensor map per layer and per cache: [max_seq rows, kv_dim columns] bf16, boxes of 64 keys x (up to) 64
// columns; 128-byte rows are stored with the 128-byte swizzle so that one thread per key reads its row without
// shared-memory bank conflicts.
static int make_tensor_maps(asd_ctx* x) {
    EncodeTiledFn encode = tensor_map_encoder();
    if (!encode) return fail(x, ASD_ERR_CUDA, "cuTensorMapEncodeTiled is not available");
    const asd_config& c = x->c;
    const int L = c.n_layers;
    std::vector<CUtensorMap> maps((size_t)2 * std::max(L, 1));
    const int box_cols = c.head_dim > 64 ? 64 : c.head_dim;
    const cuuint64_t gdim[2] = {(cuuint64_t)x->kv_dim, (cuuint64_t)c.max_seq};
    const cuuint64_t gstride[1] = {(cuuint64_t)x->kv_dim * 2};
    const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)kBoxKeys};
    const cuuint32_t estr[2] = {1u, 1u};
    const CUtensorMapSwizzle swz = (box_cols * 2 == 128) ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE;
    for (int l = 0; l < L; ++l)
        for (int which = 0; which < 2; ++which) {
            void* base = x->ws + (which ? x->lay.vcache : x->lay.kcache) + (size_t)l * x->lay.kv_layer_stride;
            const CUresult r = encode(&maps[(size_t)l * 2 + which], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, gdim, gstride, box,
                                      estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) return fail(x, ASD_ERR_CUDA, "cuTensorMapEncodeTiled failed for the KV cache");
        }
    ASD_CUDA(x, cudaMemcpyAsync(x->ws + x->lay.tmaps, maps.data(), maps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice, x->stream));
    ASD_CUDA(x, cudaStreamSynchronize(x->stream));
    if (x->lay.pf_rows > 0) {
        // operands of the dense prompt path: bf16 [rows, inner] row-major, boxes of 64 inner elements (128 bytes, the
        // swizzle span) x box_rows rows
        const Layout& ly = x->lay;
        const size_t d = c.d_model, f = c.d_ffn, kvd = x->kv_dim, R = ly.pf_rows;
        bool ok = encode_operand_map(encode, &x->tm_xn, x->ws + ly.pf_xn, d, R, kGemmBM) &&
                  encode_operand_map(encode, &x->tm_a, x->ws + ly.pf_a, d, R, kGemmBM) &&
                  encode_operand_map(encode, &x->tm_t, x->ws + ly.pf_t, f, R, kGemmBM);
        x->tm_w.assign((size_t)8 * L, CUtensorMap{});
        for (int l = 0; l < L && ok; ++l) {
            unsigned char* rw = x->ws + ly.rm_layers + (size_t)l * ly.rm_layer_stride;
            for (int v = 0; v < 2 && ok; ++v) {
                const uint32_t bn = v ? 256u : 128u;
                CUtensorMap* m = &x->tm_w[(size_t)l * 8 + v * 4];
                ok = encode_operand_map(encode, m + 0, rw + ly.rm_wqkv, d, d + 2 * kvd, bn) &&
                     encode_operand_map(encode, m + 1, rw + ly.rm_wo, d, d, bn) &&
                     encode_operand_map(encode, m + 2, rw + ly.rm_wgu, d, 2 * f, bn) &&
                     encode_operand_map(encode, m + 3, rw + ly.rm_wd, f, d, bn);
            }
        }
        if (!ok) return fail(x, ASD_ERR_CUDA, "cuTensorMapEncodeTiled failed for an operand of the dense prompt path");
    }
    return ASD_OK;
}

// Stage tables of the persistent pass kernel: table 0 = the full model M, table 1 = the draft model D (M
// without the sublayers in the skip mask: they get no stage, so nothing is streamed or touched for them),
// table 2 = the LM head alone on a hidden state that is already in place (last row of a dense prompt pass).
static int build_stage_tables(asd_ctx* x) {
    const asd_config& c = x->c;
    const Layout& ly = x->lay;
    const int d = c.d_model, f = c.d_ffn, kvd = x->kv_dim, L = c.n_layers;
    float* cosv = x->at<float>(ly.cosv);
    const CUtensorMap* maps = x->at<CUtensorMap>(ly.tmaps);
    std::vector<StageDesc> tab((size_t)3 * ly.max_stages);
    const int max_resid = 2 * std::max(L, 1);
    std::vector<ResidOut> resid((size_t)2 * max_resid);
    for (int which = 0; which < 2; ++which) {
        StageDesc* t = tab.data() + (size_t)which * ly.max_stages;
        int n = 0, nr = 0;
        int x_writer = 0;  // index of the stage that wrote the current hidden state (stage 0 = embedding)
        ResidOut* ro = resid.data() + (size_t)which * max_resid;
        t[n] = StageDesc{};
        t[n++].type = kStEmbed;
        for (int l = 0; l < L; ++l) {
            unsigned char* lw = x->layer(l);
            __nv_bfloat16* kc = reinterpret_cast<__nv_bfloat16*>(x->ws + ly.kcache + (size_t)l * ly.kv_layer_stride);
            __nv_bfloat16* vc = reinterpret_cast<__nv_bfloat16*>(x->ws + ly.vcache + (size_t)l * ly.kv_layer_stride);
            if (!(which && x->skip_attn[l])) {
                StageDesc q{};
                q.type = kStQkv, q.layer = l, q.n_rows = d + 2 * kvd, q.n_in = d;
                q.W = lw + ly.l_wqkv;
                q.gain = reinterpret_cast<const __nv_bfloat16*>(lw + ly.l_attn_norm);
                q.k_cache = kc, q.v_cache = vc;
                q.src_stage = x_writer;
                t[n++] = q;
                StageDesc a{};
                a.type = kStAttn, a.layer = l;
                a.k_cache = kc, a.v_cache = vc;
                a.tm_k = maps + (size_t)l * 2, a.tm_v = maps + (size_t)l * 2 + 1;
                t[n++] = a;
                StageDesc o{};
                o.type = kStOproj, o.layer = l, o.n_rows = d, o.n_in = d;
                o.W = lw + ly.l_wo;
                o.resid_slot = nr;
                o.src_stage = x_writer;
                ro[nr++] = ResidOut{cosv + (size_t)(0 * L + l) * kPassMaxRows, x->at<double>(ly.sumcos) + l};
                x_writer = n;
                t[n++] = o;
            }
            if (!(which && x->skip_mlp[l])) {
                StageDesc g{};
                g.type = kStGateUp, g.layer = l, g.n_rows = 2 * f, g.n_in = d;
                g.W = lw + ly.l_wgu;
                g.gain = reinterpret_cast<const __nv_bfloat16*>(lw + ly.l_mlp_norm);
                g.src_stage = x_writer;
                t[n++] = g;
                StageDesc w{};
                w.type = kStDown, w.layer = l, w.n_rows = d, w.n_in = f;
                w.W = lw + ly.l_wd;
                w.resid_slot = nr;
                w.src_stage = x_writer;
                ro[nr++] = ResidOut{cosv + (size_t)(1 * L + l) * kPassMaxRows, x->at<double>(ly.sumcos) + L + l};
                x_writer = n;
                t[n++] = w;
            }
        }
        StageDesc fin{};  // turns the residual stages' partial sums into cosine similarities
        fin.type = kStFinish, fin.layer = L;
        t[n++] = fin;
        StageDesc h{};
        h.type = kStLmHead, h.layer = L, h.n_rows = c.vocab, h.n_in = d;
        h.W = x->ws + ly.lm_head;
        h.gain = x->at<__nv_bfloat16>(ly.final_norm);
        h.src_stage = x_writer;
        t[n++] = h;
        (which ? x->n_stages_draft : x->n_stages_full) = n;
        (which ? x->n_resid_draft : x->n_resid_full) = nr;
        if (which == 0) {  // table 2: a finish stage without residual stages (nothing to do), then the LM head
            StageDesc* t2 = tab.data() + (size_t)2 * ly.max_stages;
            t2[0] = fin;
            t2[1] = h;
            t2[1].src_stage = 0;
        }
    }
    ASD_CUDA(x, cudaMemcpyAsync(x->ws + ly.stage_tab, tab.data(), tab.size() * sizeof(StageDesc), cudaMemcpyHostToDevice, x->stream));
    ASD_CUDA(x, cudaMemcpyAsync(x->ws + ly.resid_tab, resid.data(), resid.size() * sizeof(ResidOut), cudaMemcpyHostToDevice, x->stream));
    return ASD_OK;
}

// ---------------------------------------------------------------- one pass of M rows through the decoder
// tokens (DEVICE) feed rows at positions pos0..pos0+M-1. use_mask selects the draft model D. acc_sim adds the
// rows' cosines to the prompt sums behind C_l. One cooperative launch of the persistent pass kernel.
static int run_pass(asd_ctx* x, int M, int pos0, const int* dev_tokens, bool use_mask, bool acc_sim, bool lm_head,
                    int* dev_argmax_out, bool accept, double* bytes_out, bool head_only = false) {
    const asd_config& c = x->c;
    const Layout& ly = x->lay;
    const int d = c.d_model, f = c.d_ffn, kvd = x->kv_dim, L = c.n_layers;
    cudaStream_t s = x->stream;
    if (x->dev_failed) return fail(x, ASD_ERR_DEVICE_TIMEOUT, x->dev_failed_msg);  // the caches hold an abandoned pass
    if (M < 1 || (M > kMaxRows && M != kPassMaxRows)) return fail(x, ASD_ERR_ARG, "row count out of range");
    if ((long long)pos0 + M > c.max_seq) return fail(x, ASD_ERR_OVERFLOW, "pass would exceed max_seq positions");
    PassPlan pl;
    if (!plan_pass(*x->dev, c, M, &pl)) return fail(x, ASD_ERR_ARG, "decoder shape does not fit the pass kernel's shared-memory plan");

    float* cosv = x->at<float>(ly.cosv);
    ASD_CUDA(x, cudaMemsetAsync(cosv, 0xFF, (size_t)2 * std::max(L, 1) * kPassMaxRows * 4, s));  // NaN = skipped

    unsigned* words = x->at<unsigned>(ly.sync_words);
    PassParams p{};
    p.pos0 = pos0;
    p.tokens = dev_tokens;
    p.embed = x->at<__nv_bfloat16>(ly.embed);
    p.d_model = d, p.vocab = c.vocab, p.kv_dim = kvd, p.head_dim = c.head_dim, p.n_heads = c.n_heads;
    p.n_kv_heads = c.n_kv_heads, p.d_ffn = f;
    p.hd_shift = 0;
    if ((c.head_dim & (c.head_dim - 1)) == 0)
        while ((1 << p.hd_shift) < c.head_dim) ++p.hd_shift;
    p.eps = c.rms_eps;
    p.attn_scale = 1.0f / sqrtf((float)c.head_dim);
    p.rope_cos = x->at<float>(ly.rope_cos);
    p.rope_sin = x->at<float>(ly.rope_sin);
    p.x = x->at<float>(ly.x);
    p.q = x->at<__nv_bfloat16>(ly.q);
    p.a = x->at<__nv_bfloat16>(ly.a);
    p.t = x->at<__nv_bfloat16>(ly.t);
    p.xl = x->at<uint2>(ly.xl), p.al = x->at<uint2>(ly.al), p.tl = x->at<uint2>(ly.tl);
    p.ql = x->at<uint2>(ly.ql), p.kl = x->at<uint2>(ly.kl), p.vl = x->at<uint2>(ly.vl);
    p.pl_acc = x->at<uint2>(ly.pl_acc), p.pl_ml = x->at<uint2>(ly.pl_ml);
    p.pass_tag = x->pass_tag;
    p.part_acc = x->at<float>(ly.part_acc);
    p.part_ml = x->at<float>(ly.part_ml);
    p.attn_counters = x->at<unsigned>(ly.counters) + 64;
    p.chunk_stride = ly.chunk_stride;
    p.partials = x->at<float>(ly.partials);
    p.resid = x->at<ResidOut>(ly.resid_tab) + (size_t)(use_mask ? 1 : 0) * (2 * std::max(L, 1));
    p.n_resid = head_only ? 0 : (use_mask ? x->n_resid_draft : x->n_resid_full);
    p.fin_counter = words + 0;
    p.grid_bar = words + 16;
    p.err = reinterpret_cast<int*>(words + 32);
    p.bar_base = x->bar_base;
    p.wait_cycles = x->short_waits ? kShortWaitCycles : kWaitCycles;
    p.bar_extra_last = x->inject_missing_arrival ? 1u : 0u;
    const int table = head_only ? 2 : (use_mask ? 1 : 0);
    p.stages = x->at<StageDesc>(ly.stage_tab) + (size_t)table * ly.max_stages;
    const int n_table = head_only ? 2 : (use_mask ? x->n_stages_draft : x->n_stages_full);
    p.n_stages = lm_head ? n_table : n_table - 1;
    p.row_tokens = accept ? dev_tokens : nullptr;
    p.argmax_out = dev_argmax_out ? dev_argmax_out : x->at<int>(ly.argmax);
    p.margin_out = reinterpret_cast<float*>(x->at<int>(ly.argmax) + 32);  // second half of the argmax block
    p.accept_out = accept ? x->at<int>(ly.accept) : nullptr;
    p.logits_out = (x->debug_logits || x->temperature > 0.0) ? x->at<float>(ly.logits) : nullptr;
    p.acc_sim = acc_sim ? 1 : 0;
    p.trace = x->trace ? x->at<long long>(ly.trace) : nullptr;
    x->last_n_stages = p.n_stages;
    p.ns = pl.ns, p.attn_groups = pl.attn_groups;
    p.ns_magic = (unsigned)((1ull << 32) / (unsigned)pl.ns + 1);
    p.off_bars = pl.off_bars, p.off_misc = pl.off_misc, p.off_psum = pl.off_psum, p.off_reg_a = pl.off_reg_a;
    p.xs_bytes = pl.xs_bytes;
    // tagged handoff: one-row passes whose activation window holds whole rows (always so on the benchmark shapes). Measured
    // against the barrier variant of the same kernel: 1 % faster at one row, 2 % slower at two rows (twice the words to poll).
    p.use_ll = (!x->no_tagged_handoff && !head_only && M == 1 && d <= kPassConsumers * 12 && d % 8 == 0 && f % 8 == 0 && c.head_dim <= 256 &&
                (long long)pass_wseg(M, pl.xs_bytes) * kSegK >= std::max(d, f)) ? 1 : 0;
    const int grid = x->dev->num_sms;
    ASD_CUDA(x, launch_pass(M, p, grid, pl.smem, s));
    x->bar_base += (uint32_t)p.n_stages * (uint32_t)grid;
    x->pass_tag += (uint32_t)ly.max_stages + 1u;
    if (x->pass_tag < 0x1000u) x->pass_tag = 0x1000u;  // wrapped around
    x->stats.kernel_launches += 1;

    // algorithmic bytes of the pass: weights of the stages that ran, plus K/V read by the kept attention sublayers
    double bytes = 0;
    for (int l = 0; l < L && !head_only; ++l) {
        if (!(use_mask && x->skip_attn[l]))
            bytes += 2.0 * ((double)(d + 2 * kvd) * d + (double)d * d) + 2.0 * 2.0 * kvd * (double)(pos0 + M);
        if (!(use_mask && x->skip_mlp[l])) bytes += 2.0 * 3.0 * (double)d * f;
    }
    if (lm_head) bytes += 2.0 * (double)c.vocab * d;
    x->last_has_logits = lm_head && x->debug_logits;
    x->last_had_lm_head = lm_head;
    x->last_M = M;
    if (bytes_out) *bytes_out = bytes;
    return ASD_OK;
}

// the bounded waits of the pass kernel report through eight device words; word 0 = 0 means no error
static int check_device_error(asd_ctx* x, const int32_t* w) {
    if (w[0] == 0) return ASD_OK;
    static const char* names[] = {"", "a ring slot was never filled", "a ring slot was never released", "the grid barrier never completed",
                                  "a pipeline barrier of the prompt GEMM never completed"};
    char buf[256];
    snprintf(buf, sizeof buf, "a kernel gave up waiting: %s (stage %d, item %d, slot %d, CTA %d, thread %d, tag %d, parity %d)",
             (w[0] >= 1 && w[0] <= 4) ? names[w[0]] : "unknown", w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
    x->dev_failed = true;
    x->dev_failed_msg = std::string(buf) + " (call asd_reset before going on)";
    return fail(x, ASD_ERR_DEVICE_TIMEOUT, x->dev_failed_msg);
}

// copy n ints from the device and the pass kernel's error words to the pinned buffer, wait, and check them
static int read_back(asd_ctx* x, const int* dev_src, int n) {
    if (n > 0) ASD_CUDA(x, cudaMemcpyAsync(x->pinned, dev_src, (size_t)n * 4, cudaMemcpyDeviceToHost, x->stream));
    ASD_CUDA(x, cudaMemcpyAsync(x->pinned + 32, x->at<unsigned>(x->lay.sync_words) + 32, 32, cudaMemcpyDeviceToHost, x->stream));
    ASD_CUDA(x, cudaStreamSynchronize(x->stream));
    return check_device_error(x, x->pinned + 32);
}

// Sampling: row `row` of the pass that has just been launched chooses the token at `position`. Its distribution
// softmax(logits / T) goes to probs (device, vocab doubles) and a draw of the given kind to token_out (and token_out2).
static int sample_row(asd_ctx* x, int row, double* probs, int position, int kind, int* token_out, int* token_out2) {
    const int V = x->c.vocab;
    ASD_CUDA(x, launch_softmax_rows(x->at<float>(x->lay.logits) + (size_t)row * V, 1, V, x->temperature, probs, x->stream));
    ASD_CUDA(x, launch_draw(probs, V, x->seed, position, kind, token_out, token_out2, x->stream));
    x->stats.kernel_launches += 2;
    return ASD_OK;
}
// Sampling: acceptance of the k drafts of the verify pass that has just been launched at position pos0 (rows in
// dev_row_tokens); the result replaces the greedy one in the accept block.
static int sample_accept(asd_ctx* x, int k, int pos0, const int* dev_row_tokens) {
    const int V = x->c.vocab;
    double* P = x->at<double>(x->lay.probs_p);
    ASD_CUDA(x, launch_softmax_rows(x->at<float>(x->lay.logits), k + 1, V, x->temperature, P, x->stream));
    ASD_CUDA(x, launch_accept(P, x->at<double>(x->lay.probs_q), dev_row_tokens, k, V, x->seed, pos0, x->at<int>(x->lay.accept), x->stream));
    x->stats.kernel_launches += 2;
    return ASD_OK;
}

// Running similarities: request the per-row cosines of the pass that has just been launched (before the caller's
// read_back, whose synchronisation also covers this copy) ...
static int request_cosines(asd_ctx* x) {
    if (!x->running_c) return ASD_OK;
    const size_t n = (size_t)2 * std::max(x->c.n_layers, 1) * kPassMaxRows;
    ASD_CUDA(x, cudaMemcpyAsync(x->pinned + 1024, x->ws + x->lay.cosv, n * 4, cudaMemcpyDeviceToHost, x->stream));
    return ASD_OK;
}
// ... and add its first n_rows rows, which the caller has just committed, to the sums (rows in order, in double).
static void fold_committed_rows(asd_ctx* x, int n_rows) {
    if (!x->running_c) return;
    const int L = x->c.n_layers;
    const float* h = reinterpret_cast<const float*>(x->pinned + 1024);
    for (int l = 0; l < L; ++l)
        for (int r = 0; r < n_rows; ++r) {
            x->run_attn[l] += (double)h[((size_t)0 * L + l) * kPassMaxRows + r];
            x->run_mlp[l] += (double)h[((size_t)1 * L + l) * kPassMaxRows + r];
        }
    x->n_run_rows += n_rows;
}

// ---------------------------------------------------------------- Algorithm 1
// remove_MLP = { l : l = j*m, j >= 1, l <= L-n };  remove_ATTN = { l : C_l >= alpha, l <= L-n } U remove_MLP,
// layers numbered from 1. flags drop individual rules (Table 5).
// With ASD_USE_CS_MLP (not in the paper) an MLP layer l <= L-n also goes when its own similarity reaches alpha_mlp;
// remove_ATTN keeps Algorithm 1's definition (its union is with rule 1's set only).
extern "C" int asd_admg_ext(const float* C_attn, const float* C_mlp, int32_t L, const asd_admg_params* p, uint8_t* remove_attn,
                            uint8_t* remove_mlp) {
    if (!C_attn || !p || !remove_attn || !remove_mlp || L < 0 || p->m < 0 || p->n < 0) return ASD_ERR_ARG;
    const bool cs = p->flags & ASD_USE_CS, r1 = (p->flags & ASD_USE_RULE1) && p->m >= 1, r2 = p->flags & ASD_USE_RULE2;
    const bool cs_mlp = p->flags & ASD_USE_CS_MLP;
    if (cs_mlp && !C_mlp) return ASD_ERR_ARG;
    const int32_t last_removable = L - (r2 ? p->n : 0);
    for (int32_t i = 0; i < L; ++i) {
        const int32_t l = i + 1;
        const bool free_to_go = l <= last_removable;
        const bool every_mth = r1 && free_to_go && l % p->m == 0;
        remove_attn[i] = (every_mth || (cs && free_to_go && C_attn[i] >= p->alpha)) ? 1 : 0;
        remove_mlp[i] = (every_mth || (cs_mlp && free_to_go && C_mlp[i] >= p->alpha_mlp)) ? 1 : 0;
    }
    return ASD_OK;
}

extern "C" int asd_admg(const float* C, int32_t L, const asd_admg_params* p, uint8_t* remove_attn, uint8_t* remove_mlp) {
    return asd_admg_ext(C, nullptr, L, p, remove_attn, remove_mlp);
}

// ---------------------------------------------------------------- life cycle
extern "C" size_t asd_workspace_bytes(const asd_config* cfg) {
    if (!cfg || !check_config(*cfg)) return 0;
    return make_layout(*cfg).total;
}

extern "C" int asd_create(const asd_config* cfg, void* dev_workspace, size_t bytes, void* cuda_stream, asd_ctx** out) {
    if (!cfg || !out || !dev_workspace || !check_config(*cfg)) return ASD_ERR_ARG;
    Layout lay = make_layout(*cfg);
    if (bytes < lay.total || ((uintptr_t)dev_workspace % kAlign)) return ASD_ERR_NOMEM;
    asd_ctx* x = new asd_ctx();
    x->c = *cfg;
    x->lay = lay;
    x->ws = static_cast<unsigned char*>(dev_workspace);
    x->stream = static_cast<cudaStream_t>(cuda_stream);
    x->kv_dim = cfg->n_kv_heads * cfg->head_dim;
    x->skip_attn.assign(cfg->n_layers, 0);
    x->skip_mlp.assign(cfg->n_layers, 0);
    x->run_attn.assign(cfg->n_layers, 0.0);
    x->run_mlp.assign(cfg->n_layers, 0.0);
    auto bail = [&](cudaError_t e) {
        fprintf(stderr, "asd_create: %s\n", cudaGetErrorString(e));
        if (x->pinned) cudaFreeHost(x->pinned);
        delete x;
        return ASD_ERR_CUDA;
    };
    cudaError_t e = device_info(&x->dev);
    if (e != cudaSuccess) return bail(e);
    {
        PassPlan pl;
        if (!plan_pass(*x->dev, *cfg, kPassMaxRows, &pl) || !plan_pass(*x->dev, *cfg, 1, &pl)) {
            delete x;
            return ASD_ERR_ARG;
        }
    }
    // 4 KB of token / status words, then room for the per-row cosines of one pass ([2][L][kPassMaxRows] floats)
    if ((e = cudaHostAlloc((void**)&x->pinned, 4096 + (size_t)2 * std::max(cfg->n_layers, 1) * kPassMaxRows * 4, cudaHostAllocDefault)) != cudaSuccess) return bail(e);
    // rotary table: angle(p, j) = p * theta^(-2j/head_dim), evaluated in double, stored as float
    {
        const int half = cfg->head_dim / 2;
        std::vector<float> hc((size_t)cfg->max_seq * half), hs((size_t)cfg->max_seq * half);
        std::vector<double> inv_freq(half);
        for (int j = 0; j < half; ++j) inv_freq[j] = exp(-log((double)cfg->rope_theta) * (2.0 * j / cfg->head_dim));
        for (int p = 0; p < cfg->max_seq; ++p)
            for (int j = 0; j < half; ++j) {
                const double a = (double)p * inv_freq[j];
                hc[(size_t)p * half + j] = (float)cos(a);
                hs[(size_t)p * half + j] = (float)sin(a);
            }
        if ((e = cudaMemcpyAsync(x->ws + lay.rope_cos, hc.data(), hc.size() * 4, cudaMemcpyHostToDevice, x->stream)) != cudaSuccess) return bail(e);
        if ((e = cudaMemcpyAsync(x->ws + lay.rope_sin, hs.data(), hs.size() * 4, cudaMemcpyHostToDevice, x->stream)) != cudaSuccess) return bail(e);
        if ((e = cudaStreamSynchronize(x->stream)) != cudaSuccess) return bail(e);
    }
    // zero everything behind the weights: KV cache, scratch, counters
    if ((e = cudaMemsetAsync(x->ws + lay.kcache, 0, lay.total - lay.kcache, x->stream)) != cudaSuccess) return bail(e);
    if ((e = cudaStreamSynchronize(x->stream)) != cudaSuccess) return bail(e);
    if (make_tensor_maps(x) != ASD_OK || build_stage_tables(x) != ASD_OK) {
        fprintf(stderr, "asd_create: %s\n", x->err.c_str());
        cudaFreeHost(x->pinned);
        delete x;
        return ASD_ERR_CUDA;
    }
    if ((e = cudaStreamSynchronize(x->stream)) != cudaSuccess) return bail(e);
    *out = x;
    return ASD_OK;
}

extern "C" int asd_destroy(asd_ctx* x) {
    if (!x) return ASD_ERR_ARG;
    cudaStreamSynchronize(x->stream);
    for (auto e : x->events) cudaEventDestroy(e);
    if (x->pinned) cudaFreeHost(x->pinned);
    delete x;
    return ASD_OK;
}

extern "C" const char* asd_last_error(asd_ctx* x) { return x ? x->err.c_str() : "null context"; }

// Repack one matrix into the pass kernel's layout and copy it to the device. The logical matrix has n_rows
// rows of n_in inputs; row(r) returns the host pointer of logical row r. CTA b of a G-CTA grid owns pairs
// [b*P/G, (b+1)*P/G) in groups of eight pairs (the last may be smaller); its slab is segment-major (for each
// segment of 256 inputs: for each group), and an item of R rows is a run of column blocks of 32 inputs, each
// block R rows x 64 bytes (8 blocks, fewer in the last segment). Inputs past n_in are zero.
template <class RowFn, class PairFn>
static int upload_packed(asd_ctx* x, unsigned char* dev_dst, size_t n_rows, size_t n_in, RowFn row, PairFn pair_rows_of,
                         std::vector<unsigned char>& staging, size_t pair_align = 1) {
    const size_t n_pairs = (n_rows + 1) / 2, row_blocks = (n_in + 31) / 32, n_seg = (n_in + kSegK - 1) / kSegK;
    const size_t total = n_pairs * row_blocks * 128;
    const int G = x->dev->num_sms;
    staging.assign(total, 0);
#pragma omp parallel for schedule(static)
    for (int b = 0; b < G; ++b) {
        // (the same split as cta_pairs() of the pass kernel; W_gu's boundaries are even so that two neighbouring SwiGLU
        // outputs, which share one tagged word, always belong to the same CTA)
        const size_t units = n_pairs / pair_align;
        const size_t pair0 = (size_t)b * units / G * pair_align, pair1 = (b + 1 == G) ? n_pairs : (size_t)(b + 1) * units / G * pair_align;
        const size_t np = pair1 - pair0;
        unsigned char* slab = staging.data() + pair0 * row_blocks * 128;
        for (size_t sg = 0; sg < n_seg; ++sg) {
            const size_t nblk = std::min<size_t>(kSegBlocks, row_blocks - sg * kSegBlocks);
            for (size_t o = 0; o * kGrpPairs < np; ++o) {
                const size_t pairs = std::min<size_t>(kGrpPairs, np - kGrpPairs * o), R = 2 * pairs;
                unsigned char* item = slab + sg * np * (kSegK * 4) + o * nblk * (kGrpRows * 64);
                for (size_t pq = 0; pq < pairs; ++pq) {
                    size_t rr[2];
                    pair_rows_of(pair0 + kGrpPairs * o + pq, rr[0], rr[1]);
                    for (int h = 0; h < 2; ++h) {
                        if (rr[h] >= n_rows) continue;
                        const uint16_t* src = row(rr[h]);
                        const size_t g = 2 * pq + h;
                        for (size_t j = 0; j < nblk; ++j) {
                            const size_t k = sg * kSegK + j * 32;
                            memcpy(item + j * (R * 64) + g * 64, src + k, std::min<size_t>(32, n_in - k) * 2);
                        }
                    }
                }
            }
        }
    }
    ASD_CUDA(x, cudaMemcpyAsync(dev_dst, staging.data(), total, cudaMemcpyHostToDevice, x->stream));
    ASD_CUDA(x, cudaStreamSynchronize(x->stream));  // staging is reused by the next matrix
    return ASD_OK;
}

// Row-major copy of one matrix for the dense prompt path: row n of the copy is host row row(n).
template <class RowFn>
static int upload_rowmajor(asd_ctx* x, unsigned char* dev_dst, size_t n_rows, size_t n_in, RowFn row, std::vector<unsigned char>& staging) {
    staging.resize(n_rows * n_in * 2);
#pragma omp parallel for schedule(static)
    for (long long n = 0; n < (long long)n_rows; ++n) memcpy(staging.data() + (size_t)n * n_in * 2, row((size_t)n), n_in * 2);
    ASD_CUDA(x, cudaMemcpyAsync(dev_dst, staging.data(), staging.size(), cudaMemcpyHostToDevice, x->stream));
    ASD_CUDA(x, cudaStreamSynchronize(x->stream));  // staging is reused by the next matrix
    return ASD_OK;
}

static int upload_weights(asd_ctx* x, const asd_host_weights& w) {
    const asd_config& c = x->c;
    const Layout& ly = x->lay;
    const size_t d = c.d_model, f = c.d_ffn, V = c.vocab, kvd = x->kv_dim, hd = c.head_dim, half = hd / 2;
    cudaStream_t s = x->stream;
    std::vector<unsigned char> staging;
    auto plain_pair = [](size_t pr, size_t& ra, size_t& rb) { ra = 2 * pr, rb = 2 * pr + 1; };
    int rc;
    ASD_CUDA(x, cudaMemcpyAsync(x->ws + ly.embed, w.embed, V * d * 2, cudaMemcpyHostToDevice, s));
    ASD_CUDA(x, cudaMemcpyAsync(x->ws + ly.final_norm, w.final_norm, d * 2, cudaMemcpyHostToDevice, s));
    if ((rc = upload_packed(x, x->ws + ly.lm_head, V, d, [&](size_t r) { return w.lm_head + r * d; }, plain_pair, staging))) return rc;
    for (int l = 0; l < c.n_layers; ++l) {
        unsigned char* lw = x->layer(l);
        ASD_CUDA(x, cudaMemcpyAsync(lw + ly.l_attn_norm, w.attn_norm + (size_t)l * d, d * 2, cudaMemcpyHostToDevice, s));
        ASD_CUDA(x, cudaMemcpyAsync(lw + ly.l_mlp_norm, w.mlp_norm + (size_t)l * d, d * 2, cudaMemcpyHostToDevice, s));
        // fused [q rows; k rows; v rows]; a pair is the two rotary partners (j, j + head_dim/2) of one head
        const uint16_t *wq = w.wq + (size_t)l * d * d, *wk = w.wk + (size_t)l * kvd * d, *wv = w.wv + (size_t)l * kvd * d;
        auto qkv_row = [&](size_t r) { return r < d ? wq + r * d : (r < d + kvd ? wk + (r - d) * d : wv + (r - d - kvd) * d); };
        auto qkv_pair = [&](size_t pr, size_t& ra, size_t& rb) {
            const size_t nq = d / 2, nk = kvd / 2;
            size_t base, pp;
            if (pr < nq) base = 0, pp = pr;
            else if (pr < nq + nk) base = d, pp = pr - nq;
            else base = d + kvd, pp = pr - nq - nk;
            ra = base + (pp / half) * hd + pp % half;
            rb = ra + half;
        };
        if ((rc = upload_packed(x, lw + ly.l_wqkv, d + 2 * kvd, d, qkv_row, qkv_pair, staging))) return rc;
        const uint16_t* wo = w.wo + (size_t)l * d * d;
        if ((rc = upload_packed(x, lw + ly.l_wo, d, d, [&](size_t r) { return wo + r * d; }, plain_pair, staging))) return rc;
        // gate_i and up_i form a pair, so that one warp holds both operands of SwiGLU
        const uint16_t *wg = w.wg + (size_t)l * f * d, *wu = w.wu + (size_t)l * f * d;
        if ((rc = upload_packed(x, lw + ly.l_wgu, 2 * f, d, [&](size_t r) { return (r & 1) ? wu + (r / 2) * d : wg + (r / 2) * d; },
                                plain_pair, staging, 2)))
            return rc;
        const uint16_t* wd = w.wd + (size_t)l * d * f;
        if ((rc = upload_packed(x, lw + ly.l_wd, d, f, [&](size_t r) { return wd + r * f; }, plain_pair, staging))) return rc;
        if (ly.pf_rows > 0) {
            // dense prompt path: inside every q and k head the rotary partners (j, j + head_dim/2) become neighbouring
            // rows (2j, 2j+1); gate_i and up_i alternate; the other matrices keep their order
            unsigned char* rw = x->ws + ly.rm_layers + (size_t)l * ly.rm_layer_stride;
            auto qkv_rm = [&](size_t n) {
                if (n >= d + kvd) return wv + (n - d - kvd) * d;
                const uint16_t* basep = n < d ? wq : wk;
                const size_t c = n < d ? n : n - d;
                const size_t head = c / hd, local = c % hd;
                return basep + (head * hd + local / 2 + (local & 1) * half) * d;
            };
            if ((rc = upload_rowmajor(x, rw + ly.rm_wqkv, d + 2 * kvd, d, qkv_rm, staging))) return rc;
            if ((rc = upload_rowmajor(x, rw + ly.rm_wo, d, d, [&](size_t r) { return wo + r * d; }, staging))) return rc;
            if ((rc = upload_rowmajor(x, rw + ly.rm_wgu, 2 * f, d, [&](size_t r) { return (r & 1) ? wu + (r / 2) * d : wg + (r / 2) * d; }, staging)))
                return rc;
            if ((rc = upload_rowmajor(x, rw + ly.rm_wd, d, f, [&](size_t r) { return wd + r * f; }, staging))) return rc;
        }
    }
    ASD_CUDA(x, cudaStreamSynchronize(s));
    x->have_weights = true;
    return ASD_OK;
}

extern "C" int asd_load_weights_host(asd_ctx* x, const asd_host_weights* w) {
    if (!x || !w) return ASD_ERR_ARG;
    const void* ptrs[] = {w->embed, w->lm_head, w->final_norm, w->attn_norm, w->wq, w->wk, w->wv, w->wo, w->mlp_norm, w->wg, w->wu, w->wd};
    for (const void* p : ptrs)
        if (!p && x->c.n_layers > 0) return fail(x, ASD_ERR_ARG, "null weight pointer");
    return upload_weights(x, *w);
}

extern "C" int asd_load_weights_file(asd_ctx* x, const char* path) {
    if (!x || !path) return ASD_ERR_ARG;
    const asd_config& c = x->c;
    const size_t d = c.d_model, f = c.d_ffn, V = c.vocab, kvd = x->kv_dim, L = c.n_layers;
    const size_t counts[12] = {V * d, V * d, d, L * d, L * d * d, L * kvd * d, L * kvd * d, L * d * d, L * d, L * f * d, L * f * d, L * d * f};
    FILE* fh = fopen(path, "rb");
    if (!fh) return fail(x, ASD_ERR_IO, std::string("cannot open ") + path);
    std::vector<std::vector<uint16_t>> bufs(12);
    for (int i = 0; i < 12; ++i) {
        bufs[i].resize(counts[i]);
        if (counts[i] && fread(bufs[i].data(), 2, counts[i], fh) != counts[i]) {
            fclose(fh);
            return fail(x, ASD_ERR_IO, "weight file is shorter than the configured shape");
        }
    }
    fclose(fh);
    asd_host_weights w{bufs[0].data(), bufs[1].data(), bufs[2].data(), bufs[3].data(), bufs[4].data(), bufs[5].data(),
                       bufs[6].data(), bufs[7].data(), bufs[8].data(), bufs[9].data(), bufs[10].data(), bufs[11].data()};
    return upload_weights(x, w);
}

extern "C" int asd_reset(asd_ctx* x) {
    if (!x) return ASD_ERR_ARG;
    ASD_CUDA(x, cudaStreamSynchronize(x->stream));
    x->n_committed = x->draft_cursor = 0;
    std::fill(x->skip_attn.begin(), x->skip_attn.end(), 0);
    std::fill(x->skip_mlp.begin(), x->skip_mlp.end(), 0);
    x->n_sim_rows = 0;
    std::fill(x->run_attn.begin(), x->run_attn.end(), 0.0);
    std::fill(x->run_mlp.begin(), x->run_mlp.end(), 0.0);
    x->n_run_rows = 0;
    x->last_M = 0;
    x->drafted.clear();
    x->dev_failed = false;
    x->stats = asd_stats{};
    x->spans.clear();
    x->events_used = 0;
    ASD_CUDA(x, cudaMemsetAsync(x->ws + x->lay.sumcos, 0, (size_t)2 * std::max(x->c.n_layers, 1) * 8, x->stream));
    ASD_CUDA(x, cudaMemsetAsync(x->at<unsigned>(x->lay.sync_words) + 32, 0, 32, x->stream));
    return build_stage_tables(x);
}

// ---------------------------------------------------------------- prefill (Section 3.2)
// One sublayer product of the dense prompt path: the 64 x 256 weight boxes when that still gives every SM a tile. A
// product with fp32 output (W_o, W_d) that has fewer such tiles than SMs is cut in two along its reduction dimension
// instead of taking the 128-column tiles, which run at half the rate per SM (bound by shared-memory bandwidth): the
// two halves are work items of their own and the row kernel that follows adds them (half 0 + half 1). *split_out
// tells the caller whether it was.
static int dense_gemm(asd_ctx* x, const CUtensorMap& tm_a, int layer, int which, int M, int N, int K, GemmEpi ep, bool* split_out = nullptr) {
    const int m_tiles = (M + kGemmBM - 1) / kGemmBM;
    const int tiles256 = ((N + 255) / 256) * m_tiles;
    // cut in two when the 256-column tiles do not fill the SMs, or when twice as many half-length work items take fewer
    // rounds' worth of time over the SMs (a half item costs a little more than half an item: 0.525)
    const int sms = x->dev->num_sms;
    const bool fewer_rounds = 525LL * ((2 * tiles256 + sms - 1) / sms) < 1000LL * ((tiles256 + sms - 1) / sms);
    const bool split = ep.mode == kGemmF32 && split_out && K >= 2048 && (tiles256 < sms || fewer_rounds);
    const int bn = (tiles256 >= x->dev->num_sms || split) ? 256 : 128;
    ep.k_split = split ? 2 : 1;
    if (split_out) *split_out = split;
    const CUtensorMap& tm_w = x->tm_w[(size_t)layer * 8 + (bn == 256 ? 4 : 0) + which];
    ASD_CUDA(x, launch_gemm_tn(tm_a, tm_w, M, N, K, bn, ep, x->stream));
    x->stats.kernel_launches += 1;
    return ASD_OK;
}

// Prompt rows [0, n) at positions pos0 + r through every layer of M as dense products: K/V appended to the cache,
// each row's cosine similarity of every sublayer added to the sums behind C_l. No LM head: the caller runs it on
// the last row's hidden state, which stays in the residual buffer of the last chunk.
static int prefill_dense(asd_ctx* x, const int32_t* dev_tokens, int n, int pos0) {
    const asd_config& c = x->c;
    const Layout& ly = x->lay;
    const int d = c.d_model, f = c.d_ffn, kvd = x->kv_dim, L = c.n_layers, R = ly.pf_rows;
    cudaStream_t s = x->stream;
    float* px = x->at<float>(ly.pf_x);
    float* pc = x->at<float>(ly.pf_c);
    float* pcos = x->at<float>(ly.pf_cos);
    __nv_bfloat16* pxn = x->at<__nv_bfloat16>(ly.pf_xn);
    __nv_bfloat16* pq = x->at<__nv_bfloat16>(ly.pf_q);
    __nv_bfloat16* pa = x->at<__nv_bfloat16>(ly.pf_a);
    __nv_bfloat16* pt = x->at<__nv_bfloat16>(ly.pf_t);
    int* err = reinterpret_cast<int*>(x->at<unsigned>(ly.sync_words) + 32);
    const float scale = 1.0f / sqrtf((float)c.head_dim);
    int rc;
    for (int c0 = 0; c0 < n; c0 += R) {
        const int rows = std::min(R, n - c0), p0 = pos0 + c0;
        auto gain = [&](int l, size_t off) { return reinterpret_cast<const __nv_bfloat16*>(x->layer(l) + off); };
        ASD_CUDA(x, launch_embed_norm(dev_tokens + c0, rows, d, c.vocab, x->at<__nv_bfloat16>(ly.embed), gain(0, ly.l_attn_norm), c.rms_eps, px, pxn, s));
        for (int l = 0; l < L; ++l) {
            __nv_bfloat16* kc = reinterpret_cast<__nv_bfloat16*>(x->ws + ly.kcache + (size_t)l * ly.kv_layer_stride);
            __nv_bfloat16* vc = reinterpret_cast<__nv_bfloat16*>(x->ws + ly.vcache + (size_t)l * ly.kv_layer_stride);
            GemmEpi e{};
            e.err = err;
            e.mode = kGemmQkv;
            e.q = pq, e.k_cache = kc, e.v_cache = vc;
            e.rope_cos = x->at<float>(ly.rope_cos), e.rope_sin = x->at<float>(ly.rope_sin);
            e.pos0 = p0, e.d_model = d, e.kv_dim = kvd, e.head_dim = c.head_dim;
            if ((rc = dense_gemm(x, x->tm_xn, l, 0, rows, d + 2 * kvd, d, e))) return rc;
            ASD_CUDA(x, launch_flash_prefill(pq, kc, vc, pa, rows, p0, d, kvd, c.head_dim, c.n_heads, c.n_kv_heads, c.max_seq, scale, s));
            GemmEpi o{};
            o.err = err;
            o.mode = kGemmF32;
            o.c = pc, o.ldc = d;
            o.c_split_stride = (size_t)R * d;
            bool split = false;
            if ((rc = dense_gemm(x, x->tm_a, l, 1, rows, d, d, o, &split))) return rc;
            ASD_CUDA(x, launch_resid_norm(rows, d, px, pc, split ? pc + (size_t)R * d : nullptr, gain(l, ly.l_mlp_norm), c.rms_eps, pxn,
                                          pcos + (size_t)l * R, s));
            GemmEpi g{};
            g.err = err;
            g.mode = kGemmSwiglu;
            g.t = pt, g.ldt = f;
            if ((rc = dense_gemm(x, x->tm_xn, l, 2, rows, 2 * f, d, g))) return rc;
            if ((rc = dense_gemm(x, x->tm_t, l, 3, rows, d, f, o, &split))) return rc;
            ASD_CUDA(x, launch_resid_norm(rows, d, px, pc, split ? pc + (size_t)R * d : nullptr, l + 1 < L ? gain(l + 1, ly.l_attn_norm) : nullptr, c.rms_eps, pxn,
                                          pcos + (size_t)(L + l) * R, s));
            x->stats.kernel_launches += 3;
        }
        ASD_CUDA(x, launch_sumcos(pcos, R, rows, 2 * L, x->at<double>(ly.sumcos), s));
        x->stats.kernel_launches += 2;
    }
    return ASD_OK;
}

static int prefill_device(asd_ctx* x, const int32_t* dev_tokens, int32_t n, int32_t* first_token, bool resolve) {
    if (!x->have_weights) return fail(x, ASD_ERR_STATE, "weights not loaded");
    if (x->dev_failed) return fail(x, ASD_ERR_DEVICE_TIMEOUT, x->dev_failed_msg);
    if (n <= 0) return fail(x, ASD_ERR_ARG, "empty prompt");
    if ((long long)x->n_committed + n > x->c.max_seq) return fail(x, ASD_ERR_OVERFLOW, "prompt exceeds max_seq");
    size_t e0, e1;
    int rc = new_event(x, &e0);
    if (rc) return rc;
    int last_rows = 0;
    // Long prompts: all rows as dense products on the tensor cores; the LM head then runs on the last row's hidden
    // state as a pass of its own. Short prompts (and ASD_PREFILL_ROWS): row passes only.
    int n_dense = 0;
    if (x->prefill_mode == ASD_PREFILL_GEMM && x->lay.pf_rows == 0)
        return fail(x, ASD_ERR_ARG, "the dense prompt path needs head_dim 64 or 128 and at least one layer");
    if (x->lay.pf_rows > 0 && x->prefill_mode != ASD_PREFILL_ROWS && n > 1 &&
        (x->prefill_mode == ASD_PREFILL_GEMM || n - 1 >= kPrefillGemmMinRows))
        n_dense = n;
    if (n_dense > 0) {
        if ((rc = prefill_dense(x, dev_tokens, n_dense, x->n_committed))) return rc;
        // the last row's hidden state leaves the dense path's buffer for the pass kernel's, whose LM head stage alone runs
        const int last_in_chunk = (n_dense - 1) % x->lay.pf_rows;
        ASD_CUDA(x, cudaMemcpyAsync(x->at<float>(x->lay.x), x->at<float>(x->lay.pf_x) + (size_t)last_in_chunk * x->c.d_model,
                                    (size_t)x->c.d_model * 4, cudaMemcpyDeviceToDevice, x->stream));
        if ((rc = run_pass(x, 1, x->n_committed + n - 1, dev_tokens + n - 1, false, false, true, nullptr, false, nullptr, true))) return rc;
        // "the last pass" reports the last prompt row: its cosines, which the dense path has computed, go where a pass leaves them
        ASD_CUDA(x, cudaMemcpy2DAsync(x->at<float>(x->lay.cosv), (size_t)kPassMaxRows * 4, x->at<float>(x->lay.pf_cos) + last_in_chunk,
                                      (size_t)x->lay.pf_rows * 4, 4, (size_t)2 * x->c.n_layers, cudaMemcpyDeviceToDevice, x->stream));
        last_rows = 1;
    }
    for (int c0 = n_dense, M = 0; c0 < n; c0 += M) {
        // row counts the pass kernel is built for: 16, or 1..9
        const int left = n - c0;
        M = left >= kPrefillRows ? kPrefillRows : (left > kMaxRows ? 8 : left);
        const bool last = c0 + M >= n;
        rc = run_pass(x, M, x->n_committed + c0, dev_tokens + c0, false, true, last, nullptr, false, nullptr);
        if (rc) return rc;
        last_rows = M;
    }
    rc = new_event(x, &e1);
    if (rc) return rc;
    x->spans.push_back({SPAN_PREFILL, e0, e1});
    x->n_committed += n;
    x->draft_cursor = x->n_committed;
    x->n_sim_rows += n;
    x->stats.prefill_rows += n;
    x->drafted.clear();
    if (x->temperature > 0.0) {  // t_1 is the full model's own draw for position n_committed; it takes the argmax's place
        int* slot = x->at<int>(x->lay.argmax) + (last_rows - 1);
        if ((rc = sample_row(x, last_rows - 1, x->at<double>(x->lay.probs_p), x->n_committed, kDrawTarget, slot, nullptr))) return rc;
    }
    if (first_token) {
        if ((rc = read_back(x, x->at<int>(x->lay.argmax) + (last_rows - 1), 1))) return rc;
        *first_token = x->pinned[0];
        if (resolve && (rc = resolve_spans(x))) return rc;
    }
    return ASD_OK;
}

extern "C" int asd_prefill_device(asd_ctx* x, const int32_t* dev_tokens, int32_t n, int32_t* first_token) {
    if (!x || !dev_tokens) return ASD_ERR_ARG;
    int32_t dummy;
    return prefill_device(x, dev_tokens, n, first_token ? first_token : &dummy, true);
}

static int stage_tokens(asd_ctx* x, const int32_t* tokens, int32_t n, int32_t* dev_dst) {
    for (int i = 0; i < n; ++i)
        if (tokens[i] < 0 || tokens[i] >= x->c.vocab) return fail(x, ASD_ERR_ARG, "token id out of range");
    ASD_CUDA(x, cudaMemcpyAsync(dev_dst, tokens, (size_t)n * 4, cudaMemcpyHostToDevice, x->stream));
    ASD_CUDA(x, cudaStreamSynchronize(x->stream));  // the host array is only borrowed for the call
    return ASD_OK;
}

extern "C" int asd_prefill(asd_ctx* x, const int32_t* tokens, int32_t n, int32_t* first_token) {
    if (!x || !tokens) return ASD_ERR_ARG;
    if (n <= 0) return fail(x, ASD_ERR_ARG, "empty prompt");
    if ((long long)x->n_committed + n > x->c.max_seq) return fail(x, ASD_ERR_OVERFLOW, "prompt exceeds max_seq");
    int rc = stage_tokens(x, tokens, n, x->at<int>(x->lay.prompt_toks));
    if (rc) return rc;
    int32_t dummy;
    return prefill_device(x, x->at<int>(x->lay.prompt_toks), n, first_token ? first_token : &dummy, true);
}

extern "C" int asd_get_similarity(asd_ctx* x, float* c_attn, float* c_mlp, int32_t* n_rows) {
    if (!x) return ASD_ERR_ARG;
    const int64_t rows = x->n_sim_rows + x->n_run_rows;
    if (n_rows) *n_rows = (int32_t)rows;
    if (x->n_sim_rows == 0) return fail(x, ASD_ERR_STATE, "no prompt row has been processed");
    const int L = x->c.n_layers;
    std::vector<double> h(2 * (size_t)std::max(L, 1));
    ASD_CUDA(x, cudaMemcpyAsync(h.data(), x->ws + x->lay.sumcos, h.size() * 8, cudaMemcpyDeviceToHost, x->stream));
    ASD_CUDA(x, cudaStreamSynchronize(x->stream));
    for (int l = 0; l < L; ++l) {
        if (c_attn) c_attn[l] = (float)((h[l] + x->run_attn[l]) / (double)rows);
        if (c_mlp) c_mlp[l] = (float)((h[L + l] + x->run_mlp[l]) / (double)rows);
    }
    return ASD_OK;
}

extern "C" int asd_set_skip_mask(asd_ctx* x, const uint8_t* skip_attn, const uint8_t* skip_mlp) {
    if (!x || !skip_attn || !skip_mlp) return ASD_ERR_ARG;
    for (int l = 0; l < x->c.n_layers; ++l) {
        x->skip_attn[l] = skip_attn[l] ? 1 : 0;
        x->skip_mlp[l] = skip_mlp[l] ? 1 : 0;
    }
    x->draft_cursor = x->n_committed;
    x->drafted.clear();
    return build_stage_tables(x);
}

extern "C" int asd_set_running_similarity(asd_ctx* x, int32_t on) {
    if (!x) return ASD_ERR_ARG;
    x->running_c = on != 0;
    return ASD_OK;
}

extern "C" int asd_admg_update(asd_ctx* x, const asd_admg_params* p, uint8_t* skip_attn, uint8_t* skip_mlp) {
    if (!x || !p) return ASD_ERR_ARG;
    const int L = x->c.n_layers;
    std::vector<float> C(std::max(L, 1)), Cm(std::max(L, 1));
    int rc = asd_get_similarity(x, C.data(), Cm.data(), nullptr);
    if (rc) return rc;
    std::vector<uint8_t> a(std::max(L, 1)), b(std::max(L, 1));
    rc = asd_admg_ext(C.data(), Cm.data(), L, p, a.data(), b.data());
    if (rc) return fail(x, rc, "bad ADMG parameters");
    rc = asd_set_skip_mask(x, a.data(), b.data());
    if (rc) return rc;
    if (skip_attn) memcpy(skip_attn, a.data(), L);
    if (skip_mlp) memcpy(skip_mlp, b.data(), L);
    return ASD_OK;
}

// ---------------------------------------------------------------- single passes
static int timed_pass(asd_ctx* x, int kind, int M, int pos0, const int* dev_tokens, bool use_mask, int* dev_argmax_out, bool accept) {
    size_t e0, e1;
    int rc = new_event(x, &e0);
    if (rc) return rc;
    double bytes = 0;
    rc = run_pass(x, M, pos0, dev_tokens, use_mask, false, true, dev_argmax_out, accept, &bytes);
    if (rc) return rc;
    rc = new_event(x, &e1);
    if (rc) return rc;
    x->spans.push_back({kind, e0, e1});
    switch (kind) {
        case SPAN_FULL: x->stats.full_passes += 1; x->stats.bytes_full += bytes; break;
        case SPAN_DRAFT: x->stats.draft_passes += 1; x->stats.bytes_draft += bytes; break;
        case SPAN_VERIFY: x->stats.verify_passes += 1; x->stats.bytes_verify += bytes; break;
    }
    return ASD_OK;
}

extern "C" int asd_decode_step(asd_ctx* x, int32_t token_in, int32_t* token_out) {
    if (!x) return ASD_ERR_ARG;
    if (!x->have_weights) return fail(x, ASD_ERR_STATE, "weights not loaded");
    if (x->n_committed + 1 > x->c.max_seq) return fail(x, ASD_ERR_OVERFLOW, "KV cache is full");
    int rc = stage_tokens(x, &token_in, 1, x->at<int>(x->lay.tok_in));
    if (rc) return rc;
    rc = timed_pass(x, SPAN_FULL, 1, x->n_committed, x->at<int>(x->lay.tok_in), false, nullptr, false);
    if (rc) return rc;
    if (x->temperature > 0.0 &&
        (rc = sample_row(x, 0, x->at<double>(x->lay.probs_p), x->n_committed + 1, kDrawTarget, x->at<int>(x->lay.argmax), nullptr)))
        return rc;
    if ((rc = request_cosines(x))) return rc;
    if ((rc = read_back(x, x->at<int>(x->lay.argmax), 1))) return rc;
    fold_committed_rows(x, 1);
    x->n_committed += 1;
    x->draft_cursor = x->n_committed;
    x->drafted.clear();
    if (token_out) *token_out = x->pinned[0];
    return resolve_spans(x);
}

extern "C" int asd_draft_step(asd_ctx* x, int32_t token_in, int32_t* token_out) {
    if (!x) return ASD_ERR_ARG;
    if (!x->have_weights) return fail(x, ASD_ERR_STATE, "weights not loaded");
    if (x->draft_cursor + 1 > x->c.max_seq) return fail(x, ASD_ERR_OVERFLOW, "KV cache is full");
    int rc = stage_tokens(x, &token_in, 1, x->at<int>(x->lay.tok_in));
    if (rc) return rc;
    const size_t j = x->drafted.size();
    if (x->temperature > 0.0 && (int)j >= kMaxRows - 1) return fail(x, ASD_ERR_STATE, "more draft steps in one round than a verify pass has rows");
    rc = timed_pass(x, SPAN_DRAFT, 1, x->draft_cursor, x->at<int>(x->lay.tok_in), true, nullptr, false);
    if (rc) return rc;
    // when sampling, the drafted token is a draw from the draft model's distribution q, which the verification needs again
    if (x->temperature > 0.0 && (rc = sample_row(x, 0, x->at<double>(x->lay.probs_q) + j * (size_t)x->c.vocab, x->draft_cursor + 1,
                                                 kDrawDraft, x->at<int>(x->lay.argmax), nullptr)))
        return rc;
    if ((rc = read_back(x, x->at<int>(x->lay.argmax), 1))) return rc;
    x->draft_cursor += 1;
    x->drafted.push_back(x->pinned[0]);
    if (token_out) *token_out = x->pinned[0];
    return resolve_spans(x);
}

extern "C" int asd_verify(asd_ctx* x, const int32_t* tokens, int32_t k, int32_t* n_accepted, int32_t* out_tokens) {
    if (!x || !tokens) return ASD_ERR_ARG;
    if (!x->have_weights) return fail(x, ASD_ERR_STATE, "weights not loaded");
    if (k < 0 || k > x->c.max_draft) return fail(x, ASD_ERR_ARG, "draft length out of range");
    if ((long long)x->n_committed + k + 1 > x->c.max_seq) return fail(x, ASD_ERR_OVERFLOW, "verify would exceed max_seq");
    if (x->temperature > 0.0) {
        // the k tokens to verify must be the ones the last k draft steps drew: their distributions q are needed
        bool same = (int32_t)x->drafted.size() == k;
        for (int j = 0; same && j < k; ++j) same = x->drafted[j] == tokens[j + 1];
        if (!same) return fail(x, ASD_ERR_STATE, "sampling-based verification needs exactly the tokens drawn by this round's draft steps");
    }
    int rc = stage_tokens(x, tokens, k + 1, x->at<int>(x->lay.draft_toks));
    if (rc) return rc;
    rc = timed_pass(x, SPAN_VERIFY, k + 1, x->n_committed, x->at<int>(x->lay.draft_toks), false, nullptr, true);
    if (rc) return rc;
    if (x->temperature > 0.0 && (rc = sample_accept(x, k, x->n_committed, x->at<int>(x->lay.draft_toks)))) return rc;
    x->drafted.clear();
    if ((rc = request_cosines(x))) return rc;
    if ((rc = read_back(x, x->at<int>(x->lay.accept), k + 2))) return rc;
    const int a = x->pinned[0];
    fold_committed_rows(x, a + 1);
    if (n_accepted) *n_accepted = a;
    if (out_tokens)
        for (int j = 0; j <= a; ++j) out_tokens[j] = x->pinned[1 + j];
    x->n_committed += a + 1;
    x->draft_cursor = x->n_committed;
    x->stats.drafted += k;
    x->stats.accepted += a;
    return resolve_spans(x);
}

// ---------------------------------------------------------------- the whole method
static int generate_device(asd_ctx* x, const int32_t* dev_prompt, int32_t n_prompt, const asd_gen_params* gp,
                           int32_t* dev_out, int32_t* n_out, asd_stats* stats) {
    if (!x->have_weights) return fail(x, ASD_ERR_STATE, "weights not loaded");
    if (n_prompt <= 0 || gp->max_new <= 0 || gp->draft_len < 0 || gp->draft_len > x->c.max_draft ||
        gp->mode < ASD_MODE_AR || gp->mode > ASD_MODE_SPEC_MANUAL_MASK)
        return fail(x, ASD_ERR_ARG, "bad generation parameters");
    if (n_prompt > x->c.max_seq) return fail(x, ASD_ERR_OVERFLOW, "prompt exceeds max_seq");
    std::vector<uint8_t> ka = x->skip_attn, km = x->skip_mlp;
    int rc = asd_reset(x);
    if (rc) return rc;
    if (gp->mode == ASD_MODE_SPEC_MANUAL_MASK) asd_set_skip_mask(x, ka.data(), km.data());
    x->running_c = (gp->admg.flags & ASD_RUNNING_C) != 0;
    if (!(gp->temperature >= 0.f)) return fail(x, ASD_ERR_ARG, "bad generation parameters");
    x->temperature = (double)gp->temperature;
    x->seed = gp->seed;
    const bool sampling = x->temperature > 0.0;
    int* scratch_tok = x->at<int>(x->lay.argmax);  // where a pass leaves its own argmax when the token is drawn instead
    cudaStream_t s = x->stream;
    size_t ev_begin, ev_end;
    if ((rc = new_event(x, &ev_begin))) return rc;

    int32_t first = 0;
    const bool need_host_token = gp->eos_id >= 0;
    rc = prefill_device(x, dev_prompt, n_prompt, need_host_token ? &first : nullptr, false);
    if (rc) return rc;
    const int last_rows = x->last_M;  // rows of the last prefill pass
    ASD_CUDA(x, cudaMemcpyAsync(dev_out, x->at<int>(x->lay.argmax) + (last_rows - 1), 4, cudaMemcpyDeviceToDevice, s));
    int produced = 1;
    bool stop = need_host_token && first == gp->eos_id;

    if (gp->mode == ASD_MODE_SPEC) {
        rc = asd_admg_update(x, &gp->admg, nullptr, nullptr);
        if (rc) return rc;
    }
    int* draft = x->at<int>(x->lay.draft_toks);
    int* accept = x->at<int>(x->lay.accept);

    if (gp->mode == ASD_MODE_AR) {
        // token i is read from dev_out[i-1] and written to dev_out[i]: no host round trip between steps
        while (produced < gp->max_new && !stop) {
            if (x->n_committed + 1 > x->c.max_seq) return fail(x, ASD_ERR_OVERFLOW, "KV cache is full");
            rc = timed_pass(x, SPAN_FULL, 1, x->n_committed, dev_out + produced - 1, false, sampling ? scratch_tok : dev_out + produced, false);
            if (rc) return rc;
            x->n_committed += 1;
            if (sampling && (rc = sample_row(x, 0, x->at<double>(x->lay.probs_p), x->n_committed, kDrawTarget, dev_out + produced, nullptr))) return rc;
            if (need_host_token || x->running_c) {  // running similarities: one host read-back per step
                if ((rc = request_cosines(x))) return rc;
                if ((rc = read_back(x, dev_out + produced, 1))) return rc;
                fold_committed_rows(x, 1);
                stop = need_host_token && x->pinned[0] == gp->eos_id;
            }
            ++produced;
        }
        x->draft_cursor = x->n_committed;
    } else {
        const int* last_src = dev_out;  // device address of the last emitted token
        while (produced < gp->max_new && !stop) {
            int k = std::min(gp->draft_len, gp->max_new - produced - 1);
            k = std::min(k, x->c.max_seq - x->n_committed - 1);
            if (k < 0) return fail(x, ASD_ERR_OVERFLOW, "KV cache is full");
            ASD_CUDA(x, cudaMemcpyAsync(draft, last_src, 4, cudaMemcpyDeviceToDevice, s));
            for (int j = 0; j < k; ++j) {  // k steps of the draft model, chained on the device
                rc = timed_pass(x, SPAN_DRAFT, 1, x->n_committed + j, draft + j, true, sampling ? scratch_tok : draft + j + 1, false);
                if (rc) return rc;
                if (sampling && (rc = sample_row(x, 0, x->at<double>(x->lay.probs_q) + (size_t)j * x->c.vocab, x->n_committed + j + 1, kDrawDraft,
                                                 draft + j + 1, nullptr)))
                    return rc;
                // draft exiting: a draft token whose top-2 logit margin in D falls below the threshold ends the run
                // (the token itself is still verified); costs one host read-back per draft step
                if (gp->draft_exit_margin > 0.f && j + 1 < k) {
                    if ((rc = read_back(x, x->at<int>(x->lay.argmax) + 32, 1))) return rc;
                    float mg;
                    memcpy(&mg, x->pinned, 4);
                    if (mg < gp->draft_exit_margin) k = j + 1;
                }
            }
            rc = timed_pass(x, SPAN_VERIFY, k + 1, x->n_committed, draft, false, nullptr, true);
            if (rc) return rc;
            if (sampling && (rc = sample_accept(x, k, x->n_committed, draft))) return rc;
            if ((rc = request_cosines(x))) return rc;
            if ((rc = read_back(x, accept, k + 2))) return rc;
            const int a = x->pinned[0];
            fold_committed_rows(x, a + 1);
            int emit = a + 1;
            if (gp->eos_id >= 0)
                for (int j = 0; j <= a; ++j)
                    if (x->pinned[1 + j] == gp->eos_id) {
                        emit = j + 1;
                        stop = true;
                        break;
                    }
            emit = std::min(emit, gp->max_new - produced);
            ASD_CUDA(x, cudaMemcpyAsync(dev_out + produced, accept + 1, (size_t)emit * 4, cudaMemcpyDeviceToDevice, s));
            produced += emit;
            last_src = dev_out + produced - 1;
            x->n_committed += a + 1;
            x->draft_cursor = x->n_committed;
            x->stats.rounds += 1;
            x->stats.drafted += k;
            x->stats.accepted += a;
            // running similarities: Algorithm 1 again on the refreshed C_l every `refresh` rounds (the draft cursor is
            // at the committed length here, so the new mask takes effect with the next round's first draft step)
            if (gp->mode == ASD_MODE_SPEC && x->running_c && gp->admg.refresh > 0 && x->stats.rounds % gp->admg.refresh == 0) {
                rc = asd_admg_update(x, &gp->admg, nullptr, nullptr);
                if (rc) return rc;
            }
        }
    }
    if ((rc = new_event(x, &ev_end))) return rc;
    if ((rc = read_back(x, nullptr, 0))) return rc;
    float ms = 0.f;
    ASD_CUDA(x, cudaEventElapsedTime(&ms, x->events[ev_begin], x->events[ev_end]));
    x->stats.ms_total = ms;
    rc = resolve_spans(x);
    if (rc) return rc;
    *n_out = produced;
    if (stats) *stats = x->stats;
    return ASD_OK;
}

extern "C" int asd_generate_device(asd_ctx* x, const int32_t* dev_prompt, int32_t n_prompt, const asd_gen_params* p,
                                   int32_t* dev_out, int32_t* n_out, asd_stats* stats) {
    if (!x || !dev_prompt || !p || !dev_out || !n_out) return ASD_ERR_ARG;
    return generate_device(x, dev_prompt, n_prompt, p, dev_out, n_out, stats);
}

extern "C" int asd_generate(asd_ctx* x, const int32_t* prompt, int32_t n_prompt, const asd_gen_params* p, int32_t* out,
                            int32_t* n_out, asd_stats* stats) {
    if (!x || !prompt || !p || !out || !n_out) return ASD_ERR_ARG;
    if (n_prompt <= 0 || p->max_new <= 0) return fail(x, ASD_ERR_ARG, "bad generation parameters");
    if (n_prompt > x->c.max_seq || p->max_new > x->c.max_seq) return fail(x, ASD_ERR_OVERFLOW, "request exceeds max_seq");
    int rc = stage_tokens(x, prompt, n_prompt, x->at<int>(x->lay.prompt_toks));
    if (rc) return rc;
    int* gen = x->at<int>(x->lay.gen_toks);
    rc = generate_device(x, x->at<int>(x->lay.prompt_toks), n_prompt, p, gen, n_out, stats);
    if (rc) return rc;
    ASD_CUDA(x, cudaMemcpyAsync(out, gen, (size_t)*n_out * 4, cudaMemcpyDeviceToHost, x->stream));
    ASD_CUDA(x, cudaStreamSynchronize(x->stream));
    return ASD_OK;
}

// ---------------------------------------------------------------- inspection
extern "C" int asd_get_last_cosines(asd_ctx* x, int32_t* M, float* cos_attn, float* cos_mlp) {
    if (!x) return ASD_ERR_ARG;
    if (x->last_M == 0) return fail(x, ASD_ERR_STATE, "no pass has run");
    const int L = x->c.n_layers, m = x->last_M;
    if (M) *M = m;
    std::vector<float> h((size_t)2 * std::max(L, 1) * kPassMaxRows);
    ASD_CUDA(x, cudaMemcpyAsync(h.data(), x->ws + x->lay.cosv, h.size() * 4, cudaMemcpyDeviceToHost, x->stream));
    ASD_CUDA(x, cudaStreamSynchronize(x->stream));
    for (int l = 0; l < L; ++l)
        for (int r = 0; r < m; ++r) {
            if (cos_attn) cos_attn[(size_t)l * m + r] = h[((size_t)0 * L + l) * kPassMaxRows + r];
            if (cos_mlp) cos_mlp[(size_t)l * m + r] = h[((size_t)1 * L + l) * kPassMaxRows + r];
        }
    return ASD_OK;
}

extern "C" int asd_set_debug(asd_ctx* x, int32_t flags) {
    if (!x) return ASD_ERR_ARG;
    x->debug_logits = (flags & 1) != 0;
    x->trace = (flags & 2) != 0;
    x->short_waits = (flags & ASD_DEBUG_SHORT_WAITS) != 0;
    x->inject_missing_arrival = (flags & ASD_DEBUG_MISSING_ARRIVAL) != 0;
    x->no_tagged_handoff = (flags & ASD_DEBUG_NO_TAGGED_HANDOFF) != 0;
    return ASD_OK;
}

extern "C" int asd_set_sampling(asd_ctx* x, float temperature, uint64_t seed) {
    if (!x || !(temperature >= 0.f)) return ASD_ERR_ARG;
    x->temperature = (double)temperature;
    x->seed = seed;
    x->drafted.clear();
    return ASD_OK;
}

extern "C" int asd_set_prefill_mode(asd_ctx* x, int32_t mode) {
    if (!x || mode < ASD_PREFILL_AUTO || mode > ASD_PREFILL_GEMM) return ASD_ERR_ARG;
    if (mode == ASD_PREFILL_GEMM && x->lay.pf_rows == 0)
        return fail(x, ASD_ERR_ARG, "the dense prompt path needs head_dim 64 or 128 and at least one layer");
    x->prefill_mode = mode;
    return ASD_OK;
}

extern "C" int asd_get_last_trace(asd_ctx* x, int32_t* n_stages, int32_t* n_ctas, int64_t* ns_out) {
    if (!x) return ASD_ERR_ARG;
    if (!x->trace || x->last_n_stages == 0) return fail(x, ASD_ERR_STATE, "no pass has run with tracing on (asd_set_debug bit 1)");
    if (n_stages) *n_stages = x->last_n_stages;
    if (n_ctas) *n_ctas = x->dev->num_sms;
    if (ns_out) {
        ASD_CUDA(x, cudaMemcpyAsync(ns_out, x->ws + x->lay.trace, (size_t)x->last_n_stages * kTraceEntries * x->dev->num_sms * 8, cudaMemcpyDeviceToHost, x->stream));
        ASD_CUDA(x, cudaStreamSynchronize(x->stream));
    }
    return ASD_OK;
}

extern "C" int asd_get_last_logits(asd_ctx* x, int32_t* M, float* logits) {
    if (!x) return ASD_ERR_ARG;
    if (x->last_M == 0 || !x->last_has_logits) return fail(x, ASD_ERR_STATE, "no logits recorded (asd_set_debug)");
    if (M) *M = x->last_M;
    if (logits) {
        ASD_CUDA(x, cudaMemcpyAsync(logits, x->ws + x->lay.logits, (size_t)x->last_M * x->c.vocab * 4, cudaMemcpyDeviceToHost, x->stream));
        ASD_CUDA(x, cudaStreamSynchronize(x->stream));
    }
    return ASD_OK;
}

extern "C" int asd_get_last_margins(asd_ctx* x, int32_t* M, float* margins) {
    if (!x) return ASD_ERR_ARG;
    if (x->last_M == 0 || !x->last_had_lm_head) return fail(x, ASD_ERR_STATE, "no pass with an LM head has run");
    if (M) *M = x->last_M;
    if (margins) {
        ASD_CUDA(x, cudaMemcpyAsync(margins, x->at<int>(x->lay.argmax) + 32, (size_t)x->last_M * 4, cudaMemcpyDeviceToHost, x->stream));
        ASD_CUDA(x, cudaStreamSynchronize(x->stream));
    }
    return ASD_OK;
}

extern "C" int asd_get_kv(asd_ctx* x, int32_t layer, int32_t pos, uint16_t* k, uint16_t* v) {
    if (!x || layer < 0 || layer >= x->c.n_layers || pos < 0 || pos >= x->c.max_seq) return ASD_ERR_ARG;
    const size_t off = (size_t)layer * x->lay.kv_layer_stride + (size_t)pos * x->kv_dim * 2;
    if (k) ASD_CUDA(x, cudaMemcpyAsync(k, x->ws + x->lay.kcache + off, (size_t)x->kv_dim * 2, cudaMemcpyDeviceToHost, x->stream));
    if (v) ASD_CUDA(x, cudaMemcpyAsync(v, x->ws + x->lay.vcache + off, (size_t)x->kv_dim * 2, cudaMemcpyDeviceToHost, x->stream));
    ASD_CUDA(x, cudaStreamSynchronize(x->stream));
    return ASD_OK;
}

extern "C" int asd_get_positions(asd_ctx* x, int32_t* n_committed, int32_t* draft_cursor) {
    if (!x) return ASD_ERR_ARG;
    if (n_committed) *n_committed = x->n_committed;
    if (draft_cursor) *draft_cursor = x->draft_cursor;
    return ASD_OK;
}

extern "C" int asd_get_stats(asd_ctx* x, asd_stats* stats) {
    if (!x || !stats) return ASD_ERR_ARG;
    *stats = x->stats;
    return ASD_OK;
}

// ---------------------------------------------------------------- the sublayer building block on its own
extern "C" size_t asd_fused_gemv_scratch_bytes(void) { return 256 + (size_t)kMaxGemvGrid * kMaxRows * 4 * 4; }

extern "C" int asd_fused_gemv(void* cuda_stream, int32_t M, int32_t n_in, int32_t n_rows, const void* x, const uint16_t* gain,
                              float eps, const uint16_t* W, int32_t epilogue, void* out, float* cosv, void* scratch,
                              size_t scratch_bytes) {
    if (!x || !W || !out || !scratch || M < 1 || M > kMaxRows || n_in <= 0 || n_in % 8 || n_rows <= 0) return ASD_ERR_ARG;
    if (epilogue < ASD_EPI_PLAIN || epilogue > ASD_EPI_RESIDUAL) return ASD_ERR_ARG;
    if (epilogue == ASD_EPI_SWIGLU && (n_rows & 1)) return ASD_ERR_ARG;
    if (epilogue == ASD_EPI_RESIDUAL && !cosv) return ASD_ERR_ARG;
    if (scratch_bytes < asd_fused_gemv_scratch_bytes() || ((uintptr_t)scratch % kAlign)) return ASD_ERR_NOMEM;
    DeviceInfo* dv = nullptr;
    if (device_info(&dv) != cudaSuccess) return ASD_ERR_CUDA;
    GemvParams p{};
    p.W = reinterpret_cast<const __nv_bfloat16*>(W);
    p.n_rows = n_rows;
    p.n_in = n_in;
    p.x = x;
    p.gain = reinterpret_cast<const __nv_bfloat16*>(gain);
    p.eps = eps;
    p.out = out;
    p.cos_out = cosv;
    p.counter = reinterpret_cast<unsigned*>(scratch);
    p.partials = reinterpret_cast<float*>(static_cast<unsigned char*>(scratch) + 256);
    int grid, xin;
    size_t smem;
    if (!plan_gemv(*dv, M, n_rows, n_in, gain != nullptr, &grid, &xin, &smem)) return ASD_ERR_ARG;
    p.x_in_smem = xin;
    if (launch_gemv(M, epilogue, gain != nullptr, p, grid, smem, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return ASD_ERR_CUDA;
    return ASD_OK;
}

// ---------------------------------------------------------------- the dense product of the prompt path on its own
extern "C" int asd_gemm_bf16(void* cuda_stream, int32_t M, int32_t N, int32_t K, const uint16_t* A, const uint16_t* W, float* C,
                             int32_t* dev_status) {
    if (!A || !W || !C || !dev_status || M <= 0 || N <= 0 || K <= 0 || K % 8) return ASD_ERR_ARG;
    if (((uintptr_t)A | (uintptr_t)W | (uintptr_t)C) % 16) return ASD_ERR_ARG;
    DeviceInfo* dv = nullptr;
    if (device_info(&dv) != cudaSuccess) return ASD_ERR_CUDA;
    EncodeTiledFn encode = tensor_map_encoder();
    if (!encode) return ASD_ERR_CUDA;
    const int m_tiles = (M + kGemmBM - 1) / kGemmBM;
    const int bn = (((N + 255) / 256) * m_tiles >= dv->num_sms) ? 256 : 128;
    CUtensorMap tm_a, tm_w;
    if (!encode_operand_map(encode, &tm_a, const_cast<uint16_t*>(A), (size_t)K, (size_t)M, kGemmBM) ||
        !encode_operand_map(encode, &tm_w, const_cast<uint16_t*>(W), (size_t)K, (size_t)N, (uint32_t)bn))
        return ASD_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemsetAsync(dev_status, 0, 32, s) != cudaSuccess) return ASD_ERR_CUDA;
    GemmEpi e{};
    e.mode = kGemmF32;
    e.err = dev_status;
    e.c = C, e.ldc = N;
    if (launch_gemm_tn(tm_a, tm_w, M, N, K, bn, e, s) != cudaSuccess) return ASD_ERR_CUDA;
    return ASD_OK;
}

// ---------------------------------------------------------------- the same product without any allocation
// Scratch for callers that cannot allocate device memory: a fixed array in the library image. In host code
// the symbol below is only a handle; its device address is looked up once per device.
constexpr int kStaticMaxGrid = 296;
constexpr size_t kStaticScratchBytes = 256 + (size_t)kStaticMaxGrid * kMaxRows * 4 * 4;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
static void* g_static_scratch_addr[64];

extern "C" int asd_fused_gemv_static(void* cuda_stream, int32_t M, int32_t n_in, int32_t n_rows, const void* x,
                                     const uint16_t* gain, float eps, const uint16_t* W, int32_t epilogue, void* out,
                                     float* cosv) {
    if (!x || !W || !out || M < 1 || M > kMaxRows || n_in <= 0 || n_in % 8 || n_rows <= 0) return ASD_ERR_ARG;
    if (epilogue < ASD_EPI_PLAIN || epilogue > ASD_EPI_RESIDUAL) return ASD_ERR_ARG;
    if (epilogue == ASD_EPI_SWIGLU && (n_rows & 1)) return ASD_ERR_ARG;
    if (epilogue == ASD_EPI_RESIDUAL && !cosv) return ASD_ERR_ARG;
    DeviceInfo* dv = nullptr;
    if (device_info(&dv) != cudaSuccess) return ASD_ERR_CUDA;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return ASD_ERR_CUDA;
    unsigned char* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_dev_mutex);
        if (!g_static_scratch_addr[dev]) {  // first call on this device: resolve the array's device address
            void* ptr = nullptr;
            const cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
            if (e != cudaSuccess || !ptr) {
                fprintf(stderr, "asd_fused_gemv_static: cudaGetSymbolAddress failed: %s\n", cudaGetErrorString(e));
                return ASD_ERR_CUDA;
            }
            g_static_scratch_addr[dev] = ptr;
        }
        scratch = static_cast<unsigned char*>(g_static_scratch_addr[dev]);
    }
    int grid, xin;
    size_t smem;
    if (!plan_gemv(*dv, M, n_rows, n_in, gain != nullptr, &grid, &xin, &smem)) return ASD_ERR_ARG;
    if (grid > kStaticMaxGrid) {
        fprintf(stderr,
                "asd_fused_gemv_static: this shape needs a %d-CTA launch plan but the built-in scratch array holds "
                "partials for at most %d CTAs; call asd_fused_gemv with caller-provided scratch instead\n",
                grid, kStaticMaxGrid);
        return ASD_ERR_NOMEM;
    }
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    // the array keeps whatever the previous call left: the arrival counter, which only the residual epilogue
    // uses, must start at zero
    if (epilogue == ASD_EPI_RESIDUAL && cudaMemsetAsync(scratch, 0, 256, s) != cudaSuccess) return ASD_ERR_CUDA;
    GemvParams p{};
    p.W = reinterpret_cast<const __nv_bfloat16*>(W);
    p.n_rows = n_rows;
    p.n_in = n_in;
    p.x = x;
    p.gain = reinterpret_cast<const __nv_bfloat16*>(gain);
    p.eps = eps;
    p.out = out;
    p.cos_out = cosv;
    p.counter = reinterpret_cast<unsigned*>(scratch);
    p.partials = reinterpret_cast<float*>(scratch + 256);
    p.x_in_smem = xin;
    if (launch_gemv(M, epilogue, gain != nullptr, p, grid, smem, s) != cudaSuccess) return ASD_ERR_CUDA;
    return ASD_OK;
}
