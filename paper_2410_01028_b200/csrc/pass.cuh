// One persistent kernel per decoder pass (decode, draft, verify, row pass of a short prompt).
//
// Why: at batch 1 a pass is ~200 dependent sublayer stages of 5-30 us each. Launching them one by one leaves
// HBM idle at every boundary (launch latency, RMSNorm prologue, drain). Weights, however, never depend on
// activations. So here one CTA per SM stays resident for the whole pass (cooperative launch) and is split in
// two roles:
//   * a producer warp walks this CTA's share of EVERY stage's weights (and of the old part of the KV cache)
//     in order and keeps a shared-memory ring of 8 KB slots full with TMA copies (cp.async.bulk, and
//     cp.async.bulk.tensor with 128-byte swizzle for K/V boxes). It never waits for activations, so HBM keeps
//     streaming across stage boundaries, grid barriers and prologues. Weights are stored in HBM in exactly
//     the order the ring consumes them (see "packed weights" below), so a CTA's slab of a stage is one
//     contiguous byte range;
//   * 15 consumer warps wait for the previous stage of all CTAs (a grid barrier on a monotonically increasing
//     counter, bounded spin), stage the activations in shared memory (RMSNorm fused), multiply the ring slots
//     on the tensor cores, and run the epilogue: RoPE + KV append, SwiGLU, residual add + cosine
//     similarity (summand of C_l, Section 3.2), LM-head argmax + greedy acceptance (Section 1).
// Sublayers in the skip mask (the draft model D, Algorithm 1) simply do not appear in the stage table: no
// weights are streamed and no K/V is touched for them.
//
// Packed weights: a matrix [n_rows, n_in] is cut into PAIRS of rows (the two rotary partners of a q/k head,
// gate_i and up_i, or two neighbouring rows) and SEGMENTS of 256 inputs. CTA b owns pairs [b*P/G, (b+1)*P/G)
// and groups them into GROUPS of eight pairs (the last group may hold fewer). One ring item = one group x one
// segment of 256 inputs = up to 16 rows x 512 bytes = one 8 KB slot, stored as up to 8 column blocks of 32 inputs
// (rows x 64 bytes each; the last segment of a row simply has fewer blocks). The CTA's slab is
// segment-major (for seg: for group), so consecutive ring items belong to different consumer warps and are
// consumed as soon as they land, and no padding crosses HBM for input sizes that are multiples of 32.
//
// The products run on the tensor cores (mma.sync m16n8k16, bf16 in, fp32 accumulate): the 16 weight rows of an item
// are the A operand, the activation rows the 8 columns of the B operand (two B tiles for more than 8 rows), so one
// step serves any row count up to 8 and the arithmetic of a row does not depend on how many rows share the pass. tcgen05 is not used here on
// purpose: its smallest tile (64 weight rows) does not fit a 148-way row split that leaves ~28 rows of the
// d x d matrices to a CTA, and its A operand would need the activations padded to 64+ rows in shared memory.
//
// Reduction order is fixed and independent of the row count M: an item's 16 steps alternate between two
// accumulators that are added at the end, segments are added in ascending order. Attention chunks are aligned
// to absolute positions and merged in order. Row m of a (k+1)-row verify pass is therefore bit-identical to
// a 1-row decode pass at the same position, so speculative output equals autoregressive output bit for bit.
#pragma once
#include <limits.h>

#include "common.cuh"
#include "ring.cuh"

namespace asd {

constexpr int kPassConsumerWarps = 15;
constexpr int kPassConsumers = kPassConsumerWarps * 32;
constexpr int kPassThreads = kPassConsumers + 32;  // + one producer warp
constexpr unsigned kProducerNapNs = 50;             // the producer warp's sleep after a round without a free slot
constexpr int kXsBudget = 40960;                    // most shared memory the attention scratch of all warp groups may take

enum StageType : int { kStEmbed = 0, kStQkv, kStAttn, kStOproj, kStGateUp, kStDown, kStLmHead, kStFinish };

struct StageDesc {
    int type, layer;
    int n_rows, n_in;
    const unsigned char* W;             // packed weights of this stage (4 KB items, see above)
    const __nv_bfloat16* gain;
    __nv_bfloat16 *k_cache, *v_cache;   // this layer's cache [max_seq, kv_dim]
    const CUtensorMap *tm_k, *tm_v;     // tensor maps over the same
    int resid_slot;                     // residual stages: which block of per-CTA partial sums they write
    int src_stage;                      // index of the stage that wrote the hidden state this stage reads (tagged handoff)
};

// where the cosine similarity of one residual stage goes (filled in by the finish stage of the pass)
struct ResidOut {
    float* cos_out;  // [kPassMaxRows] cosine of this sublayer, per row
    double* sumcos;  // running sum over prompt rows
};

struct PassParams {
    int pos0;
    const int* tokens;
    const __nv_bfloat16* embed;
    int d_model, vocab, kv_dim, head_dim, n_heads, n_kv_heads, d_ffn;
    int hd_shift;  // log2(head_dim) when head_dim is a power of two, else 0 (divisions instead of shifts)
    float eps, attn_scale;
    const float *rope_cos, *rope_sin;
    float* x;
    __nv_bfloat16 *q, *a, *t;
    uint2 *xl, *al, *tl;  // tagged handoff (one-row passes): hidden state [d], attention output [d/2], SwiGLU output [f/2] as (value, tag) words
    uint2 *ql, *kl, *vl;  // tagged handoff: this pass's query [d], key and value [kv_dim], one bf16 per word
    uint2 *pl_acc, *pl_ml;  // tagged handoff: attention partial results per (head, chunk): [head_dim] sums and (maximum, sum of weights)
    uint32_t pass_tag;     // tag of stage 0 of this pass; stage s writes pass_tag + s
    int use_ll;            // 1: launch the kernel variant that hands activations over through the tagged buffers (host: one row, d_model <= 5760)
    float *part_acc, *part_ml;
    unsigned* attn_counters;
    int chunk_stride;
    float* partials;        // [n_resid + 1][gridDim.x][kPassMaxRows][4] per-CTA partial sums (last block: LM head)
    const ResidOut* resid;  // [n_resid] outputs of the residual stages of this pass, in stage order
    int n_resid;
    unsigned* fin_counter;
    unsigned* grid_bar;
    unsigned bar_base;
    unsigned bar_extra_last;  // test hook: arrivals the finish stage's barrier waits for beyond the grid size (0 in normal use)
    long long wait_cycles;    // cycle budget of every bounded wait of the pass
    int* err;
    const StageDesc* stages;
    int n_stages;
    const int* row_tokens;
    int* argmax_out;
    float* margin_out;  // [M] top-1 minus top-2 logit of every row (the confidence that ends a draft run early), or null
    int* accept_out;
    float* logits_out;
    int acc_sim;
    long long* trace;  // optional [n_stages][kTraceEntries][gridDim.x] device timestamps (ns) and cycle counts, or null
    // shared-memory plan (bytes from the 1024-aligned base)
    int ns;            // ring slots
    unsigned ns_magic; // 2^32 / ns + 1, for exact division of ring item numbers by ns
    int attn_groups;   // 1 to 3 groups of 4 warps work on attention items
    int off_bars, off_misc, off_psum, off_reg_a;
    int xs_bytes;      // bytes of the activation window (as few windows per stage as leave the ring 20 slots)
};

constexpr int kTraceEntries = 12;  // per stage and CTA: 0-7 consumer side, 8-10 producer side (first / last copy issued, stall cycles), 11 descriptor read
constexpr int kSegK = 256;     // inputs per ring item (8 column blocks of 32; the last item of a row may hold fewer)
constexpr int kBoxKeys = 64;   // keys per K/V box (one ring slot)
constexpr int kGrpPairs = 8;   // pairs of weight rows per ring item: 16 rows, the M of one m16n8k16 tensor-core step
constexpr int kGrpRows = 2 * kGrpPairs;
constexpr int kSegBlocks = kSegK / 32;  // column blocks of 32 inputs per full segment
constexpr int kXsPad = 32;     // bf16 elements of padding per activation row (64 bytes: conflict-free 16-byte reads)

// 256-input segments whose activations (M rows, bf16, padded rows) fit the shared-memory window
__host__ __device__ inline int pass_wseg(int M, int xs_bytes) {
    const int w = (xs_bytes / M - kXsPad * 2) / (kSegK * 2);
    return w < 1 ? 1 : w;
}

// D (16x8, fp32) += A (16x16, bf16, row) * B (16x8, bf16, col): one warp-wide tensor-core step
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                               uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

struct PassSmem {
    unsigned char* ring;
    uint64_t *full, *empty;
    float* red;   // [16][kPassMaxRows*4]
    int* flag;    // [8]
    volatile unsigned* consumed;  // [64] generations of each ring slot that consumers have finished with
    const int* split;             // [8][4] per stage type: this CTA's first pair, pair count, groups of 16 rows, warp sets per group
    float* psum;
    unsigned char* reg_a;
};

__device__ __forceinline__ void stage_pair_rows(int type, const PassParams& p, int pair, int& ra, int& rb) {
    if (type == kStQkv) {
        const int half = p.head_dim >> 1;
        const int nq = p.d_model >> 1, nk = p.kv_dim >> 1;
        int base, pp;
        if (pair < nq) {
            base = 0;
            pp = pair;
        } else if (pair < nq + nk) {
            base = p.d_model;
            pp = pair - nq;
        } else {
            base = p.d_model + p.kv_dim;
            pp = pair - nq - nk;
        }
        const int head = p.hd_shift ? (pp >> (p.hd_shift - 1)) : pp / half, j = pp - head * half;
        ra = base + head * p.head_dim + j;
        rb = ra + half;
    } else {
        ra = 2 * pair;
        rb = 2 * pair + 1;
    }
}

// CTA b owns pairs [pair0, pair0 + np) of a matrix. W_gu is split at even pair indices (align = 2): two neighbouring
// SwiGLU outputs share one tagged word of the handoff buffer and must come from the same CTA.
__device__ __forceinline__ void cta_pairs(int n_rows, int type, int& pair0, int& np) {
    const int n_pairs = (n_rows + 1) >> 1;
    const int align = (type == kStGateUp) ? 2 : 1;
    const unsigned units = (unsigned)(n_pairs / align);  // units * gridDim.x < 2^32 (the host refuses larger matrices): 32-bit divisions
    pair0 = (int)(blockIdx.x * units / gridDim.x) * align;
    const int pair1 = (blockIdx.x + 1 == gridDim.x) ? n_pairs : (int)((blockIdx.x + 1) * units / gridDim.x) * align;
    np = pair1 - pair0;
}

// Attention work items (kv head, 128-key chunk), head-major; CTA b takes the contiguous range
// [b*T/G, (b+1)*T/G): mostly chunks of one head, so queries, tickets and DRAM pages are reused.
__device__ __forceinline__ int attn_local_items(const PassParams& p, int M, int& n_chunks, int& first) {
    n_chunks = (p.pos0 + M - 1) / kAttnChunk + 1;
    const unsigned total = (unsigned)(p.n_kv_heads * n_chunks);  // heads * chunks * CTAs stays far below 2^32
    first = (int)(blockIdx.x * total / gridDim.x);
    return (int)((blockIdx.x + 1) * total / gridDim.x) - first;
}

// ============================================================================================ ring protocol
// mbarrier waits are by phase PARITY, which is only unambiguous when the waiter is at most one phase away from
// the barrier. Consumer warps and producer lanes skip through the ring (each takes every n-th item), so a
// waiter can reach generation g of a slot while generation g-1 has not even landed. Every wait therefore
// first checks a plain per-slot counter of consumed generations (monotonic, no aliasing) and only then the
// barrier, which by then is at most one phase away.
__device__ __forceinline__ void ring_locate(const PassParams& p, uint32_t g, int& slot, uint32_t& gen) {
    gen = fast_div(g, p.ns_magic);
    slot = (int)(g - gen * (uint32_t)p.ns);
}

__device__ __forceinline__ bool ring_spin_consumed(const PassParams& p, const PassSmem& sm, int slot, uint32_t gen, int code,
                                                   int stage, uint32_t g, int tag) {
    if (sm.consumed[slot] >= gen) return true;
    volatile int* err = p.err;
    const long long t0 = clock64();
    for (unsigned spin = 1;; ++spin) {
        if (sm.consumed[slot] >= gen) return true;
        if ((spin & 255u) != 0) continue;
        if (*err != kErrNone) return false;
        if (clock64() - t0 > p.wait_cycles) {
            if (atomicCAS(p.err, kErrNone, code) == kErrNone) {
                p.err[1] = stage, p.err[2] = (int)g, p.err[3] = slot, p.err[4] = blockIdx.x, p.err[5] = threadIdx.x;
                p.err[6] = tag, p.err[7] = -1;
            }
            return false;
        }
    }
}

// consumer: wait until ring item g has landed; returns the slot
__device__ __forceinline__ int ring_wait_full(const PassParams& p, const PassSmem& sm, uint32_t g, int stage, int tag) {
    int slot;
    uint32_t gen;
    ring_locate(p, g, slot, gen);
    if (gen > 0 && !ring_spin_consumed(p, sm, slot, gen, kErrFullWait, stage, g, tag)) return slot;
    mbar_wait(&sm.full[slot], gen & 1, p.err, kErrFullWait, stage, g, slot, tag, p.wait_cycles);
    return slot;
}
// consumer: one thread, after all readers of the slot are done (warp or group barrier before the call)
__device__ __forceinline__ void ring_release(const PassParams& p, const PassSmem& sm, uint32_t g) {
    int slot;
    uint32_t gen;
    ring_locate(p, g, slot, gen);
    __threadfence_block();  // the readers' shared-memory loads are ordered before the slot is handed back
    sm.consumed[slot] = gen + 1;
    mbar_arrive(&sm.empty[slot]);
}
// producer: wait until the slot of ring item g may be overwritten; returns the slot
__device__ __forceinline__ int ring_acquire(const PassParams& p, const PassSmem& sm, uint32_t g, int stage, int tag) {
    int slot;
    uint32_t gen;
    ring_locate(p, g, slot, gen);
    if (gen > 0) {
        if (!ring_spin_consumed(p, sm, slot, gen, kErrEmptyWait, stage, g, tag)) return slot;
        mbar_wait(&sm.empty[slot], (gen - 1) & 1, p.err, kErrEmptyWait, stage, g, slot, tag, p.wait_cycles);
    }
    return slot;
}

__device__ __forceinline__ long long global_ns() {
    long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// producer side of the timeline (lane 0 of the producer warp): when it issued its first and last copy of the stage
// and how many cycles it waited for free slots in between
__device__ __forceinline__ void producer_trace(const PassParams& p, int stage, long long t_first, long long stall_cycles) {
    if (!p.trace || (threadIdx.x & 31) != 0) return;
    long long* t = p.trace + (size_t)stage * kTraceEntries * gridDim.x + blockIdx.x;
    t[(size_t)8 * gridDim.x] = t_first;
    t[(size_t)9 * gridDim.x] = global_ns();
    t[(size_t)10 * gridDim.x] = stall_cycles;
}

// ============================================================================================ producer
// The whole producer warp feeds the ring: lane l takes ring items l, l+32, ... of each stage. The lanes poll in ONE
// converged loop (each lane looks at the slot of its own next item, the lanes whose slot is free issue their copy
// and move on), so the warp costs its scheduler a dozen instructions per round however many lanes are waiting, and
// a freed slot is refilled within one round. (Asking L2 for the items beyond the ring with
// cp.async.bulk.prefetch.L2 while the ring is full was measured twice and slows the pass down, by 17 % at 32 items
// ahead and more at larger distances; the ring alone is the prefetch buffer.)
struct ProdState {
    int s, type, idx, n_items;
    uint32_t gi;  // ring index of item 0 of the stage
    // GEMV stage: this CTA's slab is contiguous and already in ring order (segment-major, octets inside)
    const unsigned char* slab;
    int np, n_oct, row_blocks;
    // attention stage
    const CUtensorMap *tm_k, *tm_v;
    int n_chunks, first;
};

// move to the next stage that streams anything for this lane; false when the pass has no more
template <int M>
__device__ __forceinline__ bool prod_next_stage(const PassParams& p, const PassSmem& sm, ProdState& c, int lane) {
    for (;;) {
        c.gi += (uint32_t)c.n_items;
        c.n_items = 0;
        if (++c.s >= p.n_stages) return false;
        const StageDesc st = p.stages[c.s];
        c.type = st.type;
        if (st.type == kStEmbed || st.type == kStFinish) continue;
        if (st.type == kStAttn) {
            const int n_local = attn_local_items(p, M, c.n_chunks, c.first);
            const int nhb = p.head_dim > 64 ? p.head_dim / 64 : 1;
            c.n_items = n_local * 2 * (kAttnChunk / kBoxKeys) * nhb;
            c.tm_k = st.tm_k, c.tm_v = st.tm_v;
        } else {
            const int pair0 = sm.split[st.type * 4 + 0];
            c.np = sm.split[st.type * 4 + 1];
            c.n_oct = sm.split[st.type * 4 + 2];
            c.n_items = c.n_oct * ((st.n_in + kSegK - 1) / kSegK);
            c.row_blocks = (st.n_in + 31) >> 5;  // 32-input column blocks per row
            c.slab = st.W + (size_t)pair0 * c.row_blocks * 128;
        }
        c.idx = lane;
        if (c.idx < c.n_items) return true;
    }
}

// Where item c.idx of the lane's current stage lives: a K/V box (tensor map + coordinates) or a run of weight bytes.
struct ItemSrc {
    const CUtensorMap* map;  // non-null: K/V box at (x, y)
    int x, y;
    const unsigned char* ptr;
    uint32_t bytes;
};
__device__ __forceinline__ ItemSrc item_source(const PassParams& p, const ProdState& c) {
    ItemSrc s;
    if (c.type == kStAttn) {
        const int nhb = p.head_dim > 64 ? p.head_dim / 64 : 1;
        const int box_cols = p.head_dim > 64 ? 64 : p.head_dim;
        const int tile_slots = (kAttnChunk / kBoxKeys) * nhb;
        const int j = c.idx / (2 * tile_slots), r = c.idx - j * 2 * tile_slots;
        const int which = r / tile_slots, t = r - which * tile_slots;
        const int rg = t / nhb, hb = t - rg * nhb;
        const int item = c.first + j;
        const int kvh = item / c.n_chunks, chunk = item - kvh * c.n_chunks;
        s.map = which ? c.tm_v : c.tm_k;
        s.x = kvh * p.head_dim + hb * 64;
        s.y = chunk * kAttnChunk + rg * kBoxKeys;
        s.ptr = nullptr;
        s.bytes = (uint32_t)kBoxKeys * box_cols * 2u;
    } else {
        const int seg = c.idx / c.n_oct, o = c.idx - seg * c.n_oct;
        const int nblk = min(kSegBlocks, c.row_blocks - seg * kSegBlocks);  // column blocks of this segment
        const int rows = 2 * min(kGrpPairs, c.np - kGrpPairs * o);
        s.map = nullptr;
        s.x = s.y = 0;
        s.ptr = c.slab + (size_t)seg * c.np * (kSegK * 4) + (size_t)o * nblk * (kGrpRows * 64);
        s.bytes = (uint32_t)(nblk * rows * 64);
    }
    return s;
}

template <int M>
__device__ void pass_producer(const PassParams& p, const PassSmem& sm) {
    const int lane = threadIdx.x & 31;
    volatile int* err = p.err;
    uint32_t issued[2] = {0, 0};
    int n_issued = 0;
    const uint64_t pol_stream = make_policy_evict_first();  // weights are read once per pass: do not let them age in L2
    ProdState c{};
    c.s = -1;
    bool active = prod_next_stage<M>(p, sm, c, lane);
    long long t_progress = clock64();
    long long tp_first = (p.trace && lane == 0) ? global_ns() : 0, stall = 0, t_blocked = 0;
    bool blocked = false;
    for (unsigned round = 1; __any_sync(0xffffffffu, active); ++round) {
        bool copied = false;
        if (active) {
            const uint32_t g = c.gi + (uint32_t)c.idx;
            int slot;
            uint32_t gen;
            ring_locate(p, g, slot, gen);
            // the slot may be overwritten once generation gen-1 of it has been consumed (counter first: the barrier's
            // phase parity alone is ambiguous for a waiter that is more than one phase behind)
            const bool free_now = gen == 0 || (sm.consumed[slot] >= gen && mbar_try_wait(&sm.empty[slot], (gen - 1) & 1));
            if (free_now) {
                if (p.trace && lane == 0 && blocked) stall += clock64() - t_blocked;
                blocked = false;
                unsigned char* dst = sm.ring + (size_t)slot * kSlotBytes;
                const ItemSrc src = item_source(p, c);
                mbar_expect_tx(&sm.full[slot], src.bytes);
                if (src.map) tma_load_2d(dst, src.map, src.x, src.y, &sm.full[slot]);
                else tma_load_1d_hint(dst, src.ptr, src.bytes, &sm.full[slot], pol_stream);
                issued[1] = issued[0], issued[0] = g, ++n_issued;
                copied = true;
                t_progress = clock64();
                c.idx += 32;
                if (c.idx >= c.n_items) {
                    if (p.trace && lane == 0) {
                        producer_trace(p, c.s, tp_first, stall);
                        stall = 0;
                    }
                    active = prod_next_stage<M>(p, sm, c, lane);
                    if (p.trace && lane == 0) tp_first = global_ns();
                }
            } else {
                if (p.trace && lane == 0 && !blocked) t_blocked = clock64();
                blocked = true;
                if ((round & 255u) == 0) {  // the error word lives in global memory: look at it only now and then
                    if (*err != kErrNone) {
                        active = false;
                    } else if (clock64() - t_progress > p.wait_cycles) {
                        if (atomicCAS(p.err, kErrNone, kErrEmptyWait) == kErrNone) {
                            p.err[1] = c.s, p.err[2] = (int)g, p.err[3] = slot, p.err[4] = blockIdx.x, p.err[5] = threadIdx.x;
                            p.err[6] = M, p.err[7] = (int)((gen - 1) & 1);
                        }
                        active = false;
                    }
                }
            }
        }
        // A round in which no lane found a free slot: sleep a moment instead of polling again at once. The warp shares
        // its scheduler with three consumer warps, and a refill that starts some tens of nanoseconds later costs
        // nothing against a memory latency of microseconds.
        if (!__any_sync(0xffffffffu, copied)) __nanosleep(kProducerNapNs);
        __syncwarp();
    }
    // If the pass was abandoned, copies may still be in flight into this CTA's shared memory: let this lane's
    // last two copies land (bounded) before the CTA exits (the ring holds at most two items of a lane).
    if (*err != kErrNone) {
        for (int k = 0; k < 2 && k < n_issued; ++k) {
            int slot;
            uint32_t gen;
            ring_locate(p, issued[k], slot, gen);
            const long long t0 = clock64();
            while (!mbar_try_wait(&sm.full[slot], gen & 1) && clock64() - t0 < 20000000LL) {
            }
        }
    }
}

// per-stage timeline of every CTA (debugging aid): 0 = stage entered, 1 = inputs ready, 2 = streaming done, 3 = stage left
__device__ __forceinline__ void trace_mark(const PassParams& p, int stage, int k) {
    if (p.trace && threadIdx.x == 0) p.trace[((size_t)stage * kTraceEntries + k) * gridDim.x + blockIdx.x] = global_ns();
}

// ============================================================================================ grid barrier
__device__ __forceinline__ void consumers_sync() { bar_sync(1, kPassConsumers); }

// release = false: the arrival only counts (nobody will wait for this stage before a later, releasing arrival of the
// same CTA, whose release is cumulative); the CTA does not wait for its stores to be acknowledged.
__device__ __forceinline__ void grid_arrive(const PassParams& p, bool release = true) {
    consumers_sync();
    // one release at GPU scope: cumulative over the writes of the whole CTA, which the barrier above ordered before it
    if (threadIdx.x == 0) {
        if (release) asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p.grid_bar), "r"(1u) : "memory");
        else asm volatile("red.relaxed.gpu.global.add.u32 [%0], %1;" ::"l"(p.grid_bar), "r"(1u) : "memory");
    }
}
__device__ __forceinline__ void grid_wait(const PassParams& p, unsigned target) {
    if (threadIdx.x == 0) {
        volatile int* err = p.err;
        const long long t0 = clock64();
        // every poll is a round trip to L2; the error word and the clock are looked at only now and then
        for (unsigned spin = 1; (int)(ld_acquire_gpu(p.grid_bar) - target) < 0; ++spin) {
            if ((spin & 63u) != 0) continue;
            if (*err != kErrNone) break;
            if (clock64() - t0 > p.wait_cycles) {
                if (atomicCAS(p.err, kErrNone, kErrGridWait) == kErrNone) {
                    p.err[1] = (int)((target - p.bar_base) / gridDim.x), p.err[2] = (int)ld_acquire_gpu(p.grid_bar);
                    p.err[3] = (int)target, p.err[4] = blockIdx.x;
                }
                break;
            }
        }
    }
    consumers_sync();
}

// consumers only: true in every thread of the last CTA to arrive on a global counter
__device__ __forceinline__ bool last_cta_consumers(unsigned* counter, int* flag_smem) {
    __threadfence();
    consumers_sync();
    if (threadIdx.x == 0) {
        const unsigned t = atomicAdd(counter, 1u);
        *flag_smem = (t == gridDim.x - 1) ? 1 : 0;
    }
    consumers_sync();
    const bool last = *flag_smem != 0;
    if (last) __threadfence();
    return last;
}

// Every stage starts by waiting for the previous stage of all CTAs. Whatever does not depend on activations (the
// stage descriptor, index arithmetic, zeroing of partial sums, RMSNorm gains) is done before this wait.
__device__ __forceinline__ void stage_begin(const PassParams& p, int s, unsigned extra = 0u) {
    if (s > 0) grid_wait(p, p.bar_base + (unsigned)s * gridDim.x + extra);
    trace_mark(p, s, 1);
}

// LM head: (largest logit, its lowest index, second-largest logit) of two disjoint index sets combined
__device__ __forceinline__ void top2_merge(float& v, int& i, float& s, float ov, int oi, float os) {
    s = fmaxf(fminf(v, ov), fmaxf(s, os));
    if (ov > v || (ov == v && oi < i)) {
        v = ov;
        i = oi;
    }
}

// ============================================================================================ tagged handoff
// One-row passes (decode, draft) spend a third of their time between weight streams,
// and most of that in round trips to L2: a stage's last output is stored, a fence and an atomic arrive at the grid
// barrier, every CTA polls the barrier word, and only then loads the activations. Here the activations carry their
// own "ready" mark instead: every 4-byte value (one fp32 of the hidden state, or two bf16 of the attention / SwiGLU
// output) is stored together with a 4-byte tag as ONE 8-byte word (8-byte scalar stores are single-copy atomic), the
// tag naming the pass and the stage that wrote it. A consumer simply loads the words it needs and repeats the load
// until every tag is the one it expects: one round trip after the slowest producer's store, no fence, no barrier.
// A buffer is only overwritten by a stage that itself needed ALL outputs of a later stage than every reader's, so no
// reader can still be waiting for the old contents (same ordering a barrier would give, carried by the data).
// The attention stage takes part: W_qkv's epilogue leaves q and this pass's k and v as tagged words (one bf16 each), a
// (head, chunk) item leaves its partial result as tagged words, and the group that took a head's last chunk merges the
// head once all items of its CTA are done. q, k, v and the partial results of a layer are overwritten by the next
// layer's stages, which a CTA only reaches through W_o's stage, i.e. after every head's merged output (and with it
// every read of q, k, v and of the partial results) exists.
__device__ __forceinline__ void ll_store(uint2* dst, uint32_t data, uint32_t tag) {
    const unsigned long long v = ((unsigned long long)tag << 32) | (unsigned long long)data;
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(dst), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long ll_load1(const uint2* src) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(src) : "memory");
    return v;
}
__device__ __forceinline__ void ll_load2(const uint2* src, unsigned long long& a, unsigned long long& b) {  // 16-byte aligned
    asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(a), "=l"(b) : "l"(src) : "memory");
}
__device__ __forceinline__ bool ll_ready(unsigned long long v, uint32_t tag) { return (uint32_t)(v >> 32) == tag; }
// after a load that found a stale tag: go on waiting? (bounded like every other wait of the kernel)
__device__ __forceinline__ bool ll_keep_waiting(const PassParams& p, unsigned& spins, long long& t0, int stage) {
    if (spins == 0) t0 = clock64();
    if ((++spins & 31u) != 0) return true;
    volatile int* err = p.err;
    if (*err != kErrNone) return false;
    if (clock64() - t0 > p.wait_cycles) {
        if (atomicCAS(p.err, kErrNone, kErrGridWait) == kErrNone) {
            p.err[1] = stage, p.err[2] = -1, p.err[3] = -1, p.err[4] = blockIdx.x, p.err[5] = threadIdx.x, p.err[6] = 77, p.err[7] = 0;
        }
        return false;
    }
    return true;
}

// ============================================================================================ GEMV stage
// RMSNorm of M whole rows into the activation window (two or more rows; rows of at most 12 x 480 elements), for most
// row counts a function of its own so that its registers are its own: the rows are taken in batches of up to six, all loads of a
// batch in flight together, and what was loaded for the statistics is normalised from registers, so a batch costs one
// memory round trip. The arithmetic of a row is the one of the other paths: thread t adds the squares of its chunks
// t, t + 480, t + 960 element by element, lanes by butterfly, warps in index order.
template <int M>
__device__ __forceinline__ void norm_rows_body(const float* xf, const __nv_bfloat16* gain, int n_in, int wlen, int xstride, float eps,
                                               __nv_bfloat16* xs, float* red) {
    constexpr int kBatches = (M + 5) / 6, kRB = (M + kBatches - 1) / kBatches;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint2 gv[3];
#pragma unroll
    for (int c = 0; c < 3; ++c) {
        const int i = (tid + c * kPassConsumers) * 4;
        gv[c] = make_uint2(0u, 0u);
        if (i < n_in) gv[c] = *reinterpret_cast<const uint2*>(gain + i);
    }
#pragma unroll
    for (int m0 = 0; m0 < M; m0 += kRB) {
        float4 v[kRB][3];
#pragma unroll
        for (int u = 0; u < kRB; ++u)
#pragma unroll
            for (int c = 0; c < 3; ++c) {
                const int i = (tid + c * kPassConsumers) * 4;
                v[u][c] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (m0 + u < M && i < n_in) v[u][c] = __ldcg(reinterpret_cast<const float4*>(xf + (size_t)(m0 + u) * n_in + i));
            }
#pragma unroll
        for (int u = 0; u < kRB; ++u)
            if (m0 + u < M) {
                float s = 0.f;
#pragma unroll
                for (int c = 0; c < 3; ++c) {
                    const int i = (tid + c * kPassConsumers) * 4;
                    if (i < n_in) {
                        s = fmaf(v[u][c].x, v[u][c].x, s);
                        s = fmaf(v[u][c].y, v[u][c].y, s);
                        s = fmaf(v[u][c].z, v[u][c].z, s);
                        s = fmaf(v[u][c].w, v[u][c].w, s);
                    }
                }
                s = warp_sum(s);
                if (lane == 0) red[warp * (kPassMaxRows * 4) + m0 + u] = s;
            }
        bar_sync(1, kPassConsumers);
#pragma unroll
        for (int u = 0; u < kRB; ++u)
            if (m0 + u < M) {
                const int m = m0 + u;
                float s = 0.f;
#pragma unroll
                for (int w = 0; w < kPassConsumerWarps; ++w) s += red[w * (kPassMaxRows * 4) + m];
                const float inv = 1.0f / sqrtf(s / (float)n_in + eps);
#pragma unroll
                for (int c = 0; c < 3; ++c) {
                    const int i = (tid + c * kPassConsumers) * 4;
                    if (i < wlen) {
                        uint2 o = make_uint2(0u, 0u);
                        if (i < n_in) {
                            const float g0 = bf_lo(gv[c].x), g1 = bf_hi(gv[c].x), g2 = bf_lo(gv[c].y), g3 = bf_hi(gv[c].y);
                            __nv_bfloat162 lo = __floats2bfloat162_rn(v[u][c].x * inv * g0, v[u][c].y * inv * g1);
                            __nv_bfloat162 hi = __floats2bfloat162_rn(v[u][c].z * inv * g2, v[u][c].w * inv * g3);
                            o.x = *reinterpret_cast<uint32_t*>(&lo);
                            o.y = *reinterpret_cast<uint32_t*>(&hi);
                        }
                        *reinterpret_cast<uint2*>(xs + (size_t)m * xstride + i) = o;
                    }
                }
            }
    }
    for (int i = kPassConsumers * 12 + tid * 4; i < wlen; i += kPassConsumers * 4)  // zero padding past 5760
        for (int m = 0; m < M; ++m) *reinterpret_cast<uint2*>(xs + (size_t)m * xstride + i) = make_uint2(0u, 0u);
}

// Called as a function by most row counts; with five and six rows the call itself (measured) costs more than the
// registers it frees.
template <int M>
__device__ __noinline__ void norm_rows_call(const float* xf, const __nv_bfloat16* gain, int n_in, int wlen, int xstride, float eps,
                                            __nv_bfloat16* xs, float* red) {
    norm_rows_body<M>(xf, gain, n_in, wlen, xstride, eps, xs, red);
}
template <int M>
__device__ __forceinline__ void norm_rows_into_window(const float* xf, const __nv_bfloat16* gain, int n_in, int wlen, int xstride, float eps,
                                                      __nv_bfloat16* xs, float* red) {
    if constexpr (M == 5 || M == 6) norm_rows_body<M>(xf, gain, n_in, wlen, xstride, eps, xs, red);
    else norm_rows_call<M>(xf, gain, n_in, wlen, xstride, eps, xs, red);
}

// Epilogues of a GEMV stage with three or more activation rows, as functions of their own (their registers are their
// own; everything they need comes as scalar arguments, so nothing is re-read from the parameter block or the stage
// table). The (weight row or pair, activation row) items of the CTA are spread over all consumer threads instead of
// giving a thread all M rows of its pair. Every item is computed exactly as the one-row path computes it, and the
// sums that cross threads keep that path's shape (the cosine sums of activation row m: the lanes of a warp hold 32
// consecutive weight rows and are added by the same butterfly, the warps' sums are added in ascending order of the
// weight rows), so row m of an M-row pass stays bit-identical to a one-row pass. pre0 / pre1: what the first item of
// the thread (W_qkv: rotary factors) or of the warp (residual stages: old hidden state) needs from global memory,
// requested by the caller ahead of the weight stream.
__device__ __forceinline__ float psum_total(const float* psum, int idx, int S, int copy_stride) {
    float v = psum[idx];  // the copies of a partial sum (warp sets that shared a group) in the order 0, 1, ...
    for (int k = 1; k < S; ++k) v += psum[(size_t)k * copy_stride + idx];
    return v;
}

// residual add + cosine sums: item (m, j) = activation row m, weight rows 32 j .. 32 j + 31 of this CTA, one warp each
template <int M>
__device__ __noinline__ void epi_resid_rows(float* out, const float* psum, float* red, float* partials_dst, int n_rows, int pair0, int np,
                                            int S, float pre0) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int copy_stride = np * 2 * M;
    const int W = (np * 2 + 31) >> 5;
    for (int it = warp; it < M * W; it += kPassConsumerWarps) {
        const int m = it / W, j = it - m * W, e = j * 32 + lane, row = 2 * pair0 + e;
        float sxy = 0.f, sxx = 0.f, syy = 0.f;
        if (e < np * 2 && row < n_rows) {
            const float xv = (it == warp) ? pre0 : __ldcg(out + (size_t)m * n_rows + row);
            const float y = xv + psum_total(psum, e * M + m, S, copy_stride);
            out[(size_t)m * n_rows + row] = y;
            sxy = fmaf(xv, y, 0.f);
            sxx = fmaf(xv, xv, 0.f);
            syy = fmaf(y, y, 0.f);
        }
        sxy = warp_sum(sxy);
        sxx = warp_sum(sxx);
        syy = warp_sum(syy);
        if (lane == 0) red[it * 4 + 0] = sxy, red[it * 4 + 1] = sxx, red[it * 4 + 2] = syy;
    }
    bar_sync(1, kPassConsumers);
    if (tid < M * 3) {
        const int m = tid / 3, q = tid - m * 3;
        float tot = 0.f;
        for (int j = 0; j < W; ++j) tot += red[(m * W + j) * 4 + q];
        partials_dst[m * 4 + q] = tot;
    }
}

// W_qkv: rotary embedding of the q and k pairs, bf16 rounding, q to its buffer and k, v to the cache rows pos0 + m
template <int M>
__device__ __noinline__ void epi_qkv_rows(const float* psum, int pair0, int np, int S, int pos0, int d_model, int kv_dim, int head_dim,
                                          const float* rope_cos, const float* rope_sin, __nv_bfloat16* q, __nv_bfloat16* kc,
                                          __nv_bfloat16* vc, float pre0, float pre1) {
    const int tid = threadIdx.x;
    const int copy_stride = np * 2 * M;
    const int half = head_dim >> 1, nq = d_model >> 1, nk = kv_dim >> 1;
    for (int it = tid; it < np * M; it += kPassConsumers) {
        const int m = it / np, pl = it - m * np, pair = pair0 + pl;
        const int base = pair < nq ? 0 : (pair < nq + nk ? d_model : d_model + kv_dim);
        const int pp = pair < nq ? pair : (pair < nq + nk ? pair - nq : pair - nq - nk);
        const int head = pp / half, jr = pp - head * half;
        const int ra = base + head * head_dim + jr, rb = ra + half;
        float va = psum_total(psum, (pl * 2 + 0) * M + m, S, copy_stride), vb = psum_total(psum, (pl * 2 + 1) * M + m, S, copy_stride);
        const int pos = pos0 + m;
        if (ra < d_model + kv_dim) {  // q or k: rotate the pair (j, j + head_dim/2) by pos * theta_j
            const float c = (it == tid) ? pre0 : rope_cos[(size_t)pos * half + jr];
            const float sn = (it == tid) ? pre1 : rope_sin[(size_t)pos * half + jr];
            const float r0 = __fmaf_rn(va, c, -__fmul_rn(vb, sn));
            const float r1 = __fmaf_rn(vb, c, __fmul_rn(va, sn));
            va = r0;
            vb = r1;
        }
        const __nv_bfloat16 ha = __float2bfloat16_rn(va), hb = __float2bfloat16_rn(vb);
        if (ra < d_model) {
            q[(size_t)m * d_model + ra] = ha;
            q[(size_t)m * d_model + rb] = hb;
        } else if (ra < d_model + kv_dim) {
            kc[(size_t)pos * kv_dim + (ra - d_model)] = ha;
            kc[(size_t)pos * kv_dim + (rb - d_model)] = hb;
        } else {
            vc[(size_t)pos * kv_dim + (ra - d_model - kv_dim)] = ha;
            vc[(size_t)pos * kv_dim + (rb - d_model - kv_dim)] = hb;
        }
    }
}

// W_gu: SwiGLU of every (pair, row), bf16 rounding
template <int M>
__device__ __noinline__ void epi_gateup_rows(const float* psum, int pair0, int np, int S, __nv_bfloat16* t_out, int t_stride) {
    const int copy_stride = np * 2 * M;
    for (int it = threadIdx.x; it < np * M; it += kPassConsumers) {
        const int m = it / np, pl = it - m * np;
        const float va = psum_total(psum, (pl * 2 + 0) * M + m, S, copy_stride), vb = psum_total(psum, (pl * 2 + 1) * M + m, S, copy_stride);
        const float t = va / (1.0f + expf(-va)) * vb;
        t_out[(size_t)m * t_stride + (pair0 + pl)] = __float2bfloat16_rn(t);
    }
}

// LM head: the warps are dealt to the activation rows (warp w serves rows w mod G, w mod G + G, ...); a row's (largest
// logit, its lowest index, second-largest logit) does not depend on the order of the comparisons. lmp: this CTA's
// block of the per-CTA results.
template <int M>
__device__ __noinline__ void epi_lmhead_rows(const float* psum, float* red, int pair0, int np, int S, int n_rows, float* logits_out, float* lmp) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int copy_stride = np * 2 * M;
    constexpr int G = M < kPassConsumerWarps ? M : kPassConsumerWarps;
    const int g = warp % G, wi = warp / G, nw = (kPassConsumerWarps - g + G - 1) / G;
    for (int m = g; m < M; m += G) {
        float bv = -INFINITY, sv = -INFINITY;
        int bi = INT_MAX;
        for (int pl = wi * 32 + lane; pl < np; pl += nw * 32) {
            const int ra = 2 * (pair0 + pl), rb = ra + 1;
            const bool has_b = rb < n_rows;
            const float va = psum_total(psum, (pl * 2 + 0) * M + m, S, copy_stride), vb = psum_total(psum, (pl * 2 + 1) * M + m, S, copy_stride);
            if (logits_out) {
                logits_out[(size_t)m * n_rows + ra] = va;
                if (has_b) logits_out[(size_t)m * n_rows + rb] = vb;
            }
            if (va > bv) {  // rows come in ascending order: an equal logit keeps the lower index
                sv = bv, bv = va, bi = ra;
            } else {
                sv = fmaxf(sv, va);
            }
            if (has_b) {
                if (vb > bv) {
                    sv = bv, bv = vb, bi = rb;
                } else {
                    sv = fmaxf(sv, vb);
                }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            const float os = __shfl_xor_sync(0xffffffffu, sv, o);
            top2_merge(bv, bi, sv, ov, oi, os);
        }
        if (lane == 0) {
            red[warp * (kPassMaxRows * 4) + m * 4 + 0] = bv;
            red[warp * (kPassMaxRows * 4) + m * 4 + 1] = __int_as_float(bi);
            red[warp * (kPassMaxRows * 4) + m * 4 + 2] = sv;
        }
    }
    bar_sync(1, kPassConsumers);
    if (tid < M) {
        float v = -INFINITY, sc = -INFINITY;
        int i = INT_MAX;
        for (int w = tid % G; w < kPassConsumerWarps; w += G)
            top2_merge(v, i, sc, red[w * (kPassMaxRows * 4) + tid * 4 + 0], __float_as_int(red[w * (kPassMaxRows * 4) + tid * 4 + 1]),
                       red[w * (kPassMaxRows * 4) + tid * 4 + 2]);
        lmp[tid * 4 + 0] = v;
        lmp[tid * 4 + 1] = __int_as_float(i);
        lmp[tid * 4 + 2] = sc;
    }
}

template <int M, bool LL>
__device__ void gemv_stage(const PassParams& p, const StageDesc& st, const PassSmem& sm, uint32_t& gi, int stage) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int type = st.type;
    const bool norm = (type == kStQkv || type == kStGateUp || type == kStLmHead);
    const int n_in = st.n_in, n_rows = st.n_rows;
    // this CTA's share of the matrix (computed once per launch: the split costs three integer divisions)
    const int pair0 = sm.split[type * 4 + 0], np = sm.split[type * 4 + 1];
    const int n_seg = (n_in + kSegK - 1) / kSegK;
    const int n_oct = sm.split[type * 4 + 2];  // groups of 16 rows (8 pairs; the last group may hold fewer)
    const int wseg = pass_wseg(M, p.xs_bytes);
    const int xstride = wseg * kSegK + kXsPad;  // bf16 elements per activation row in the window
    __nv_bfloat16* xs = reinterpret_cast<__nv_bfloat16*>(sm.reg_a);
    float* red = sm.red;
    float* psum = sm.psum;

    const float* xf = p.x;
    const __nv_bfloat16* xb = (type == kStOproj) ? p.a : p.t;
    constexpr bool kLLCap = LL;
    constexpr bool ll = LL;                                       // activations come and go through the tagged buffers
    const uint32_t tag_x = p.pass_tag + (uint32_t)st.src_stage;   // tag of the hidden state this stage reads
    const uint32_t tag_in = p.pass_tag + (uint32_t)(stage - 1);   // tag of the attention / SwiGLU output (previous stage)
    const uint32_t tag_out = p.pass_tag + (uint32_t)stage;        // tag of what this stage writes
    unsigned ll_spins = 0;
    long long ll_t0 = 0;
    // Fewer groups than warps (the d x d matrices leave ~28 rows to a CTA): several warps share a group, warp set ks
    // taking the segments congruent to ks modulo S and summing into its own copy of the partial sums; the copies are
    // added in the epilogue in the order ks = 0, 1, ... (a fixed order that depends on the matrix shape only).
    const int S = sm.split[type * 4 + 3];
    const int copy_stride = np * 2 * M;
    // A warp's first item of the stage stores its sums, later items add: the partial sums need no zeroing (only when a
    // row has fewer segments than warp sets, i.e. some copies would never be written, they are zeroed and all items add)
    const bool store_first = n_seg >= S;
    if (!store_first)
        for (int i = tid; i < S * copy_stride; i += kPassConsumers) psum[i] = 0.f;
    constexpr bool kKeepX = (M == 1);
    const bool keep = kKeepX && norm && n_in <= kPassConsumers * 12;
    uint2 gpre[3] = {make_uint2(0u, 0u), make_uint2(0u, 0u), make_uint2(0u, 0u)};  // this thread's RMSNorm gains
    const bool short_rows = norm && n_in <= kPassConsumers * 12;  // a thread owns at most three 4-element chunks of a row
    if (short_rows) {
#pragma unroll
        for (int c = 0; c < 3; ++c) {
            const int i = (tid + c * kPassConsumers) * 4;
            if (i < n_in) gpre[c] = *reinterpret_cast<const uint2*>(st.gain + i);
        }
    }
    // One or two rows: what the epilogue will need from global memory is requested ahead of the weight stream
    // (the rotary factors of this thread's pair before the barrier, the old hidden state of its row after it),
    // so the epilogue does not wait for a memory round trip.
    constexpr bool kSpreadEpi = (M >= 3);  // measured: spreading the epilogue's items over the threads pays from three rows on (two rows: no difference)
    constexpr bool kPre = (M <= 2);
    float pre[kPre ? 2 * M : 1];
    float pre0 = 0.f, pre1 = 0.f;  // spread epilogue: what the first item of this thread / warp needs (see the epi_*_rows functions)
    if (kSpreadEpi && type == kStQkv && tid < np * M) {
        const int m = tid / np;
        int ra, rb;
        stage_pair_rows(type, p, pair0 + (tid - m * np), ra, rb);
        if (ra < p.d_model + p.kv_dim) {
            const int half = p.head_dim >> 1, jr = p.hd_shift ? (ra & (p.head_dim - 1)) : ra % p.head_dim;
            pre0 = p.rope_cos[(size_t)(p.pos0 + m) * half + jr];
            pre1 = p.rope_sin[(size_t)(p.pos0 + m) * half + jr];
        }
    }
    if (kPre && type == kStQkv && tid < np) {
        int ra, rb;
        stage_pair_rows(type, p, pair0 + tid, ra, rb);
        if (ra < p.d_model + p.kv_dim) {
            const int half = p.head_dim >> 1, jr = p.hd_shift ? (ra & (p.head_dim - 1)) : ra % p.head_dim;
#pragma unroll
            for (int m = 0; m < (kPre ? M : 0); ++m) {
                pre[m] = p.rope_cos[(size_t)(p.pos0 + m) * half + jr];
                pre[M + m] = p.rope_sin[(size_t)(p.pos0 + m) * half + jr];
            }
        }
    }
    if (ll) trace_mark(p, stage, 1);  // no barrier: the loads below wait for exactly the words they need
    else stage_begin(p, stage);
    if (kSpreadEpi && (type == kStOproj || type == kStDown)) {
        const int W = (np * 2 + 31) >> 5;
        if (warp < M * W) {
            const int m = warp / W, e = (warp - m * W) * 32 + lane;
            if (e < np * 2 && 2 * pair0 + e < n_rows) pre0 = __ldcg(p.x + (size_t)m * n_rows + 2 * pair0 + e);
        }
    }
    if (kPre && (type == kStOproj || type == kStDown) && tid < np * 2 && 2 * pair0 + tid < n_rows) {
        if (ll) {
            unsigned long long raw[kPre ? M : 1] = {};
            bool ok;
            do {
                ok = true;
#pragma unroll
                for (int m = 0; m < (kPre ? M : 0); ++m) raw[m] = ll_load1(p.xl + (size_t)m * n_rows + 2 * pair0 + tid);
#pragma unroll
                for (int m = 0; m < (kPre ? M : 0); ++m) ok = ok && ll_ready(raw[m], tag_x);
            } while (!ok && ll_keep_waiting(p, ll_spins, ll_t0, stage));
#pragma unroll
            for (int m = 0; m < (kPre ? M : 0); ++m) pre[m] = __uint_as_float((uint32_t)raw[m]);
        } else {
#pragma unroll
            for (int m = 0; m < (kPre ? M : 0); ++m) pre[m] = __ldcg(p.x + (size_t)m * n_rows + 2 * pair0 + tid);
        }
    }

    // ---- RMSNorm statistics (same arithmetic for every row count). With one row the hidden state read here stays in
    //      registers for the window fill below (one L2 round trip less per stage); two and more rows whose window
    //      holds them whole take norm_rows_into_window() instead.
    float4 xr[kKeepX ? M : 1][3];
    float inv[M];
    constexpr bool kFusedNorm = (M >= 2);
    const bool fused = kFusedNorm && short_rows && n_seg <= wseg;  // whole rows in one window: statistics and fill in one go below
    if (norm && !fused) {
        float ssq[M];  // this thread's share of every row's sum of squares; per row the additions run in index order
#pragma unroll
        for (int m = 0; m < M; ++m) ssq[m] = 0.f;
        if (keep) {
            if (ll) {
                // all of this thread's words of all rows in flight together; then only the 16-byte halves whose tags are
                // still stale are loaded again, with a growing pause in between (a CTA that is early would otherwise
                // re-read 32 KB per row and round and crowd the other CTAs' weight streams out of L2's ports)
                unsigned long long raw[kKeepX ? M : 1][3][4] = {};
                unsigned stale = 0u;  // bit (m * 3 + c) * 2 + h
#pragma unroll
                for (int m = 0; m < (kKeepX ? M : 0); ++m)
#pragma unroll
                    for (int c = 0; c < 3; ++c)
                        if ((tid + c * kPassConsumers) * 4 < n_in) stale |= 3u << ((m * 3 + c) * 2);
                for (;;) {
#pragma unroll
                    for (int m = 0; m < (kKeepX ? M : 0); ++m)
#pragma unroll
                        for (int c = 0; c < 3; ++c)
#pragma unroll
                            for (int h = 0; h < 2; ++h)
                                if (stale & (1u << ((m * 3 + c) * 2 + h)))
                                    ll_load2(p.xl + (size_t)m * n_in + (tid + c * kPassConsumers) * 4 + 2 * h, raw[m][c][2 * h], raw[m][c][2 * h + 1]);
#pragma unroll
                    for (int m = 0; m < (kKeepX ? M : 0); ++m)
#pragma unroll
                        for (int c = 0; c < 3; ++c)
#pragma unroll
                            for (int h = 0; h < 2; ++h)
                                if ((stale & (1u << ((m * 3 + c) * 2 + h))) && ll_ready(raw[m][c][2 * h], tag_x) && ll_ready(raw[m][c][2 * h + 1], tag_x))
                                    stale &= ~(1u << ((m * 3 + c) * 2 + h));
                    if (stale == 0u || !ll_keep_waiting(p, ll_spins, ll_t0, stage)) break;
                    __nanosleep(ll_spins < 4 ? 100u : 300u);
                }
#pragma unroll
                for (int m = 0; m < (kKeepX ? M : 0); ++m)
#pragma unroll
                    for (int c = 0; c < 3; ++c)
                        xr[m][c] = make_float4(__uint_as_float((uint32_t)raw[m][c][0]), __uint_as_float((uint32_t)raw[m][c][1]),
                                               __uint_as_float((uint32_t)raw[m][c][2]), __uint_as_float((uint32_t)raw[m][c][3]));
            }
#pragma unroll
            for (int m = 0; m < M; ++m) {
#pragma unroll
                for (int c = 0; c < 3; ++c) {
                    const int i = (tid + c * kPassConsumers) * 4;
                    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (ll) v = xr[kKeepX ? m : 0][c];
                    else if (i < n_in) v = __ldcg(reinterpret_cast<const float4*>(xf + (size_t)m * n_in + i));
                    xr[kKeepX ? m : 0][c] = v;
                    if (i < n_in) {
                        float s = ssq[m];
                        s = fmaf(v.x, v.x, s);
                        s = fmaf(v.y, v.y, s);
                        s = fmaf(v.z, v.z, s);
                        s = fmaf(v.w, v.w, s);
                        ssq[m] = s;
                    }
                }
            }
        } else {
            // long rows: the loads of up to four rows are in flight together (one memory round trip per four rows and stride)
            for (int i = tid * 4; i < n_in; i += kPassConsumers * 4) {
#pragma unroll
                for (int m0 = 0; m0 < M; m0 += 4) {
                    float4 v[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        if (m0 + u < M) v[u] = __ldcg(reinterpret_cast<const float4*>(xf + (size_t)(m0 + u) * n_in + i));
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        if (m0 + u < M) {
                            float s = ssq[m0 + u];
                            s = fmaf(v[u].x, v[u].x, s);
                            s = fmaf(v[u].y, v[u].y, s);
                            s = fmaf(v[u].z, v[u].z, s);
                            s = fmaf(v[u].w, v[u].w, s);
                            ssq[m0 + u] = s;
                        }
                }
            }
        }
#pragma unroll
        for (int m = 0; m < M; ++m) {
            const float s = warp_sum(ssq[m]);
            if (lane == 0) red[warp * (kPassMaxRows * 4) + m] = s;
        }
        consumers_sync();
#pragma unroll
        for (int m = 0; m < M; ++m) {
            float s = 0.f;
#pragma unroll
            for (int w = 0; w < kPassConsumerWarps; ++w) s += red[w * (kPassMaxRows * 4) + m];
            inv[m] = 1.0f / sqrtf(s / (float)n_in + p.eps);
        }
    }
    trace_mark(p, stage, 6);

    long long cyc_wait = 0, cyc_work = 0;  // when tracing: cycles this warp spent waiting for slots / working on them
    // ---- stream the slab window by window
    const int g8 = lane >> 2, q4 = lane & 3;  // tensor-core fragment coordinates of this lane
    for (int w0 = 0; w0 < n_seg; w0 += wseg) {
        const int ws = min(wseg, n_seg - w0);
        const int k0 = w0 * kSegK;
        const int wlen = ws * kSegK;  // inputs in this window, including the zero padding past n_in
        consumers_sync();  // previous window fully consumed; psum zeroed; red free
        if (fused) {
            norm_rows_into_window<M>(xf, st.gain, n_in, wlen, xstride, p.eps, xs, red);
        } else if (keep) {  // a single window (n_in <= 5760): normalise the rows held in registers
#pragma unroll
            for (int c = 0; c < 3; ++c) {
                const int i = (tid + c * kPassConsumers) * 4;
                if (i < wlen) {
                    const bool in = i < n_in;
                    const uint2 gv = gpre[c];
                    const float g0 = bf_lo(gv.x), g1 = bf_hi(gv.x), g2 = bf_lo(gv.y), g3 = bf_hi(gv.y);
#pragma unroll
                    for (int m = 0; m < M; ++m) {
                        uint2 o = make_uint2(0u, 0u);
                        if (in) {
                            const float4 v = xr[kKeepX ? m : 0][c];
                            __nv_bfloat162 lo = __floats2bfloat162_rn(v.x * inv[m] * g0, v.y * inv[m] * g1);
                            __nv_bfloat162 hi = __floats2bfloat162_rn(v.z * inv[m] * g2, v.w * inv[m] * g3);
                            o.x = *reinterpret_cast<uint32_t*>(&lo);
                            o.y = *reinterpret_cast<uint32_t*>(&hi);
                        }
                        *reinterpret_cast<uint2*>(xs + (size_t)m * xstride + i) = o;
                    }
                }
            }
            for (int i = kPassConsumers * 12 + tid * 4; i < wlen; i += kPassConsumers * 4)  // zero padding past 5760
                for (int m = 0; m < M; ++m) *reinterpret_cast<uint2*>(xs + (size_t)m * xstride + i) = make_uint2(0u, 0u);
        } else if (norm) {
            for (int i = tid * 4; i < wlen; i += kPassConsumers * 4) {
                const bool in = k0 + i < n_in;
                uint2 gv = make_uint2(0u, 0u);
                if (in) gv = *reinterpret_cast<const uint2*>(st.gain + k0 + i);
                const float g0 = bf_lo(gv.x), g1 = bf_hi(gv.x), g2 = bf_lo(gv.y), g3 = bf_hi(gv.y);
#pragma unroll
                for (int m0 = 0; m0 < M; m0 += 4) {
                    float4 v[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        if (m0 + u < M && in) v[u] = __ldcg(reinterpret_cast<const float4*>(xf + (size_t)(m0 + u) * n_in + k0 + i));
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        if (m0 + u < M) {
                            const int m = m0 + u;
                            uint2 o = make_uint2(0u, 0u);
                            if (in) {
                                __nv_bfloat162 lo = __floats2bfloat162_rn(v[u].x * inv[m] * g0, v[u].y * inv[m] * g1);
                                __nv_bfloat162 hi = __floats2bfloat162_rn(v[u].z * inv[m] * g2, v[u].w * inv[m] * g3);
                                o.x = *reinterpret_cast<uint32_t*>(&lo);
                                o.y = *reinterpret_cast<uint32_t*>(&hi);
                            }
                            *reinterpret_cast<uint2*>(xs + (size_t)m * xstride + i) = o;
                        }
                }
            }
        } else if (ll) {
            // bf16 inputs as tagged words (two bf16 each): the window holds whole rows; two 8-element chunks per row and
            // thread in flight together, repeated until every tag is the expected one
            const uint2* src = (type == kStOproj) ? p.al : p.tl;
            for (int i0 = tid * 8; i0 < wlen; i0 += 2 * kPassConsumers * 8) {
                unsigned long long raw[kLLCap ? M : 1][2][4] = {};
                unsigned stale = 0u;  // bit (m * 2 + u) * 2 + h
#pragma unroll
                for (int m = 0; m < (kLLCap ? M : 0); ++m)
#pragma unroll
                    for (int u = 0; u < 2; ++u)
                        if (i0 + u * kPassConsumers * 8 < n_in) stale |= 3u << ((m * 2 + u) * 2);
                for (;;) {
#pragma unroll
                    for (int m = 0; m < (kLLCap ? M : 0); ++m)
#pragma unroll
                        for (int u = 0; u < 2; ++u)
#pragma unroll
                            for (int h = 0; h < 2; ++h)
                                if (stale & (1u << ((m * 2 + u) * 2 + h)))
                                    ll_load2(src + (((size_t)m * n_in + i0 + u * kPassConsumers * 8) >> 1) + 2 * h, raw[m][u][2 * h], raw[m][u][2 * h + 1]);
#pragma unroll
                    for (int m = 0; m < (kLLCap ? M : 0); ++m)
#pragma unroll
                        for (int u = 0; u < 2; ++u)
#pragma unroll
                            for (int h = 0; h < 2; ++h)
                                if ((stale & (1u << ((m * 2 + u) * 2 + h))) && ll_ready(raw[m][u][2 * h], tag_in) && ll_ready(raw[m][u][2 * h + 1], tag_in))
                                    stale &= ~(1u << ((m * 2 + u) * 2 + h));
                    if (stale == 0u || !ll_keep_waiting(p, ll_spins, ll_t0, stage)) break;
                    __nanosleep(ll_spins < 4 ? 100u : 300u);
                }
#pragma unroll
                for (int m = 0; m < (kLLCap ? M : 0); ++m)
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const int i = i0 + u * kPassConsumers * 8;
                        if (i < wlen) {
                            uint4 v = make_uint4(0u, 0u, 0u, 0u);
                            if (i < n_in) v = make_uint4((uint32_t)raw[m][u][0], (uint32_t)raw[m][u][1], (uint32_t)raw[m][u][2], (uint32_t)raw[m][u][3]);
                            *reinterpret_cast<uint4*>(xs + (size_t)m * xstride + i) = v;
                        }
                    }
            }
        } else {
            for (int i = tid * 8; i < wlen; i += kPassConsumers * 8) {
                const bool in = k0 + i < n_in;
#pragma unroll
                for (int m = 0; m < M; ++m) {
                    uint4 v = make_uint4(0u, 0u, 0u, 0u);
                    if (in) v = __ldcg(reinterpret_cast<const uint4*>(xb + (size_t)m * n_in + k0 + i));
                    *reinterpret_cast<uint4*>(xs + (size_t)m * xstride + i) = v;
                }
            }
        }
        consumers_sync();

        if (w0 == 0) trace_mark(p, stage, 7);
        // Ring order is segment-major: consecutive items are different groups, i.e. different warps. One item is up to
        // 16 weight rows x 256 inputs, stored as column blocks of 32 inputs ([block][row][64 bytes]); lane (g8, q4)
        // owns inputs 32*block + 8*q4 .. +7 of rows g8 and g8 + 8. Two m16n8k16 steps per block: the weights are the
        // 16-row A operand, the activation rows the 8 columns of the B operand (columns >= M are zero), so every
        // step covers 16 weight rows and nothing of the tile is wasted on padding rows.
        const __nv_bfloat16* xa = xs + (size_t)min(g8, M - 1) * xstride + q4 * 8;
        const __nv_bfloat16* xb2 = xs + (size_t)min(g8 + 8, M - 1) * xstride + q4 * 8;
        const int ks = (S > 1) ? warp / n_oct : 0;                 // which copy of the partial sums this warp adds into
        const int o_first = (S > 1) ? ((ks < S) ? warp - ks * n_oct : n_oct) : warp;
        const int o_step = (S > 1) ? n_oct : kPassConsumerWarps;  // S > 1: exactly one group per warp
        float* psum_w = psum + (size_t)ks * copy_stride;
        // this warp set's segments of the window: ks, ks + S, ... (one remainder per window instead of one per segment)
        int seg_first = w0;
        if (S > 1) {
            const int r = w0 % S;
            seg_first = w0 + (ks >= r ? ks - r : ks + S - r);
        }
        for (int seg = seg_first; seg < w0 + ws; seg += S) {
            const int sg = seg - w0;
            for (int o = o_first; o < n_oct; o += o_step) {
                const uint32_t g = gi + (uint32_t)(seg * n_oct + o);
                const int rows = 2 * min(kGrpPairs, np - kGrpPairs * o);
                const long long tw0 = p.trace ? clock64() : 0;
                const int slot = ring_wait_full(p, sm, g, stage, M * 1000 + seg);
                const long long tw1 = p.trace ? clock64() : 0;
                const unsigned char* sl = sm.ring + (size_t)slot * kSlotBytes + g8 * 64 + q4 * 16;
                const int blk = rows * 64;
                const int nblk = min(kSegBlocks, ((n_in + 31) >> 5) - seg * kSegBlocks);
                // Four independent accumulators (column block parity x half of the block), added in a fixed order;
                // acc2 holds activation rows 8..15 (row passes of a prompt with more than 8 rows).
                float acc[4][4], acc2[M > 8 ? 4 : 1][4];
#pragma unroll
                for (int a = 0; a < 4; ++a) acc[a][0] = acc[a][1] = acc[a][2] = acc[a][3] = 0.f;
#pragma unroll
                for (int a = 0; a < (M > 8 ? 4 : 1); ++a) acc2[a][0] = acc2[a][1] = acc2[a][2] = acc2[a][3] = 0.f;
                // Operands of four column blocks in registers, then 8 steps; twice per full item. Lanes whose weight row lies
                // beyond the item's rows, or whose activation row beyond M, read whatever follows in the slot / the last
                // activation row: every output element depends on its own weight row and activation row only, and the
                // outputs of such rows are never stored. Only column blocks past the end of a ragged last segment must
                // contribute nothing and are replaced by zeros.
                if (nblk == kSegBlocks) {
#pragma unroll
                    for (int h = 0; h < kSegBlocks / 4; ++h) {
                        uint4 wlo[4], whi[4], xv[4], xv2[M > 8 ? 4 : 1];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            wlo[j] = *reinterpret_cast<const uint4*>(sl + (h * 4 + j) * blk);
                            whi[j] = *reinterpret_cast<const uint4*>(sl + (h * 4 + j) * blk + 8 * 64);
                            xv[j] = *reinterpret_cast<const uint4*>(xa + sg * kSegK + (h * 4 + j) * 32);
                            if (M > 8) xv2[j] = *reinterpret_cast<const uint4*>(xb2 + sg * kSegK + (h * 4 + j) * 32);
                        }
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            mma_bf16_16816(acc[(j & 1) * 2 + 0], wlo[j].x, whi[j].x, wlo[j].y, whi[j].y, xv[j].x, xv[j].y);
                            mma_bf16_16816(acc[(j & 1) * 2 + 1], wlo[j].z, whi[j].z, wlo[j].w, whi[j].w, xv[j].z, xv[j].w);
                            if (M > 8) {
                                mma_bf16_16816(acc2[(j & 1) * 2 + 0], wlo[j].x, whi[j].x, wlo[j].y, whi[j].y, xv2[j].x, xv2[j].y);
                                mma_bf16_16816(acc2[(j & 1) * 2 + 1], wlo[j].z, whi[j].z, wlo[j].w, whi[j].w, xv2[j].z, xv2[j].w);
                            }
                        }
                    }
                } else {
#pragma unroll 1
                    for (int h = 0; h * 4 < nblk; ++h) {
                        uint4 wlo[4], whi[4], xv[4], xv2[M > 8 ? 4 : 1];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const bool inb = h * 4 + j < nblk;
                            wlo[j] = inb ? *reinterpret_cast<const uint4*>(sl + (h * 4 + j) * blk) : make_uint4(0u, 0u, 0u, 0u);
                            whi[j] = inb ? *reinterpret_cast<const uint4*>(sl + (h * 4 + j) * blk + 8 * 64) : make_uint4(0u, 0u, 0u, 0u);
                            xv[j] = *reinterpret_cast<const uint4*>(xa + sg * kSegK + (h * 4 + j) * 32);
                            if (M > 8) xv2[j] = *reinterpret_cast<const uint4*>(xb2 + sg * kSegK + (h * 4 + j) * 32);
                        }
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            mma_bf16_16816(acc[(j & 1) * 2 + 0], wlo[j].x, whi[j].x, wlo[j].y, whi[j].y, xv[j].x, xv[j].y);
                            mma_bf16_16816(acc[(j & 1) * 2 + 1], wlo[j].z, whi[j].z, wlo[j].w, whi[j].w, xv[j].z, xv[j].w);
                            if (M > 8) {
                                mma_bf16_16816(acc2[(j & 1) * 2 + 0], wlo[j].x, whi[j].x, wlo[j].y, whi[j].y, xv2[j].x, xv2[j].y);
                                mma_bf16_16816(acc2[(j & 1) * 2 + 1], wlo[j].z, whi[j].z, wlo[j].w, whi[j].w, xv2[j].z, xv2[j].w);
                            }
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) ring_release(p, sm, g);
                // c[0], c[1]: weight row g8 of the group, activation rows 2*q4 and 2*q4 + 1; c[2], c[3]: weight row g8 + 8.
                // Local weight row 16*o + r is row (r & 1) of local pair 8*o + r/2. Segments are added in ascending
                // order, always by this lane.
#pragma unroll
                for (int hr = 0; hr < 2; ++hr) {
                    const int wr = g8 + 8 * hr;
                    if (wr < rows) {
                        float* dst = psum_w + (size_t)(kGrpRows * o + wr) * M;
                        const bool first = store_first && seg == ((S > 1) ? ks : 0);
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int mm = 2 * q4 + e;
                            if (mm < M) {
                                const float v = (acc[0][2 * hr + e] + acc[2][2 * hr + e]) + (acc[1][2 * hr + e] + acc[3][2 * hr + e]);
                                dst[mm] = first ? v : dst[mm] + v;
                            }
                            if (M > 8 && mm + 8 < M) {
                                const float v = (acc2[0][2 * hr + e] + acc2[2][2 * hr + e]) + (acc2[1][2 * hr + e] + acc2[3][2 * hr + e]);
                                dst[mm + 8] = first ? v : dst[mm + 8] + v;
                            }
                        }
                    }
                }
                if (p.trace) {
                    cyc_wait += tw1 - tw0;
                    cyc_work += clock64() - tw1;
                }
            }
        }
    }
    gi += (uint32_t)(n_oct * n_seg);
    consumers_sync();
    trace_mark(p, stage, 2);
    if (p.trace && tid == 0) {
        p.trace[((size_t)stage * kTraceEntries + 4) * gridDim.x + blockIdx.x] = cyc_wait;
        p.trace[((size_t)stage * kTraceEntries + 5) * gridDim.x + blockIdx.x] = cyc_work;
    }

    if constexpr (!kSpreadEpi) {
    // ---- epilogue of a pass of one or two rows: thread t owns pairs t, t+480, ... of this CTA and all M rows of them
    float s_loc[M][3];
    float best_v[M], sec_v[M];
    int best_i[M];
#pragma unroll
    for (int m = 0; m < M; ++m) {
        s_loc[m][0] = s_loc[m][1] = s_loc[m][2] = 0.f;
        best_v[m] = sec_v[m] = -INFINITY;
        best_i[m] = INT_MAX;
    }
    const bool resid = (type == kStOproj || type == kStDown);
    if (resid) {
        // residual add: one thread per weight row, the M loads of the old hidden state issued together
        float* out = p.x;
        for (int e = tid; e < np * 2; e += kPassConsumers) {
            const int row = 2 * pair0 + e;
            if (row >= n_rows) continue;
            float xv[M];
#pragma unroll
            for (int m = 0; m < M; ++m) {
                if (kPre && e == tid) {
                    xv[m] = pre[kPre ? m : 0];
                } else if (ll) {  // (a CTA with more rows than threads: not on the benchmark shapes)
                    unsigned long long raw;
                    do raw = ll_load1(p.xl + (size_t)m * n_rows + row);
                    while (!ll_ready(raw, tag_x) && ll_keep_waiting(p, ll_spins, ll_t0, stage));
                    xv[m] = __uint_as_float((uint32_t)raw);
                } else {
                    xv[m] = __ldcg(out + (size_t)m * n_rows + row);
                }
            }
#pragma unroll
            for (int m = 0; m < M; ++m) {
                float v = psum[e * M + m];
                for (int k = 1; k < S; ++k) v += psum[(size_t)k * copy_stride + e * M + m];
                const float y = xv[m] + v;
                if (ll) ll_store(p.xl + (size_t)m * n_rows + row, __float_as_uint(y), tag_out);
                else out[(size_t)m * n_rows + row] = y;
                s_loc[m][0] = fmaf(xv[m], y, s_loc[m][0]);
                s_loc[m][1] = fmaf(xv[m], xv[m], s_loc[m][1]);
                s_loc[m][2] = fmaf(y, y, s_loc[m][2]);
            }
        }
    }
    if (ll && type == kStGateUp) {
        // pair0 and np are even: outputs pair0 + 2j and pair0 + 2j + 1 form one tagged word
        for (int pj = tid; 2 * pj < np; pj += kPassConsumers) {
#pragma unroll
            for (int m = 0; m < M; ++m) {
                uint32_t word = 0u;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int pl = 2 * pj + h;
                    float va = psum[(pl * 2 + 0) * M + m], vb = psum[(pl * 2 + 1) * M + m];
                    for (int k = 1; k < S; ++k) {
                        va += psum[(size_t)k * copy_stride + (pl * 2 + 0) * M + m];
                        vb += psum[(size_t)k * copy_stride + (pl * 2 + 1) * M + m];
                    }
                    const float t = va / (1.0f + expf(-va)) * vb;
                    word |= (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(t)) << (16 * h);
                }
                ll_store(p.tl + (((size_t)m * (n_rows >> 1) + pair0) >> 1) + pj, word, tag_out);
            }
        }
    }
    for (int pl = (resid || (ll && type == kStGateUp)) ? np : tid; pl < np; pl += kPassConsumers) {
        int ra, rb;
        stage_pair_rows(type, p, pair0 + pl, ra, rb);
        const bool has_b = rb < n_rows;
        // rotary factors of all rows first: the stores below may alias them as far as the compiler knows, and one
        // memory round trip per row would add up
        float rc[M], rs[M];
        if (type == kStQkv && ra < p.d_model + p.kv_dim) {
            const int half = p.head_dim >> 1, jr = p.hd_shift ? (ra & (p.head_dim - 1)) : ra % p.head_dim;
#pragma unroll
            for (int m = 0; m < M; ++m) {
                rc[m] = (kPre && pl == tid) ? pre[kPre ? m : 0] : p.rope_cos[(size_t)(p.pos0 + m) * half + jr];
                rs[m] = (kPre && pl == tid) ? pre[kPre ? M + m : 0] : p.rope_sin[(size_t)(p.pos0 + m) * half + jr];
            }
        }
#pragma unroll
        for (int m = 0; m < M; ++m) {
            float va = psum[(pl * 2 + 0) * M + m], vb = psum[(pl * 2 + 1) * M + m];
            for (int k = 1; k < S; ++k) {
                va += psum[(size_t)k * copy_stride + (pl * 2 + 0) * M + m];
                vb += psum[(size_t)k * copy_stride + (pl * 2 + 1) * M + m];
            }
            if (type == kStGateUp) {
                const float t = va / (1.0f + expf(-va)) * vb;
                p.t[(size_t)m * (n_rows >> 1) + (pair0 + pl)] = __float2bfloat16_rn(t);
            } else if (type == kStQkv) {
                const int pos = p.pos0 + m;
                if (ra < p.d_model + p.kv_dim) {  // q or k: rotate the pair (j, j + head_dim/2) by pos * theta_j
                    // explicit roundings: the same arithmetic whatever the row count the kernel was compiled for
                    const float c = rc[m], s = rs[m];
                    const float r0 = __fmaf_rn(va, c, -__fmul_rn(vb, s));
                    const float r1 = __fmaf_rn(vb, c, __fmul_rn(va, s));
                    va = r0;
                    vb = r1;
                }
                const __nv_bfloat16 ha = __float2bfloat16_rn(va), hb = __float2bfloat16_rn(vb);
                if (ll) {  // the attention stage of this pass takes q, k, v from tagged words (k, v also go to the cache)
                    uint2* dst = ra < p.d_model ? p.ql : (ra < p.d_model + p.kv_dim ? p.kl : p.vl);
                    const int off = ra < p.d_model ? 0 : (ra < p.d_model + p.kv_dim ? p.d_model : p.d_model + p.kv_dim);
                    ll_store(dst + (ra - off), (uint32_t)__bfloat16_as_ushort(ha), tag_out);
                    ll_store(dst + (rb - off), (uint32_t)__bfloat16_as_ushort(hb), tag_out);
                }
                if (ra < p.d_model) {
                    if (!ll) {
                        p.q[(size_t)m * p.d_model + ra] = ha;
                        p.q[(size_t)m * p.d_model + rb] = hb;
                    }
                } else if (ra < p.d_model + p.kv_dim) {
                    st.k_cache[(size_t)pos * p.kv_dim + (ra - p.d_model)] = ha;
                    st.k_cache[(size_t)pos * p.kv_dim + (rb - p.d_model)] = hb;
                } else {
                    st.v_cache[(size_t)pos * p.kv_dim + (ra - p.d_model - p.kv_dim)] = ha;
                    st.v_cache[(size_t)pos * p.kv_dim + (rb - p.d_model - p.kv_dim)] = hb;
                }
            } else {  // LM head
                if (p.logits_out) {
                    p.logits_out[(size_t)m * n_rows + ra] = va;
                    if (has_b) p.logits_out[(size_t)m * n_rows + rb] = vb;
                }
                if (va > best_v[m]) {  // rows come in ascending order: an equal logit keeps the lower index
                    sec_v[m] = best_v[m];
                    best_v[m] = va;
                    best_i[m] = ra;
                } else {
                    sec_v[m] = fmaxf(sec_v[m], va);
                }
                if (has_b) {
                    if (vb > best_v[m]) {
                        sec_v[m] = best_v[m];
                        best_v[m] = vb;
                        best_i[m] = rb;
                    } else {
                        sec_v[m] = fmaxf(sec_v[m], vb);
                    }
                }
            }
        }
    }

    if (type == kStOproj || type == kStDown) {
        // cosine similarity of the hidden state before and after this sublayer: warp-shuffle partial dot and
        // norm products, one block-level finish; the per-CTA partials are combined by the finish stage of the pass
#pragma unroll
        for (int m = 0; m < M; ++m)
#pragma unroll
            for (int j = 0; j < 3; ++j) {
                const float v = warp_sum(s_loc[m][j]);
                if (lane == 0) red[warp * (kPassMaxRows * 4) + m * 4 + j] = v;
            }
        consumers_sync();
        if (tid < M * 3) {
            const int m = tid / 3, j = tid - m * 3;
            float tot = 0.f;
#pragma unroll
            for (int w = 0; w < kPassConsumerWarps; ++w) tot += red[w * (kPassMaxRows * 4) + m * 4 + j];
            p.partials[(((size_t)st.resid_slot * gridDim.x + blockIdx.x) * kPassMaxRows + m) * 4 + j] = tot;
        }
    } else if (type == kStLmHead) {
#pragma unroll
        for (int m = 0; m < M; ++m) {
            float v = best_v[m], sc = sec_v[m];
            int i = best_i[m];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, v, o);
                const int oi = __shfl_xor_sync(0xffffffffu, i, o);
                const float os = __shfl_xor_sync(0xffffffffu, sc, o);
                top2_merge(v, i, sc, ov, oi, os);
            }
            if (lane == 0) {
                red[warp * (kPassMaxRows * 4) + m * 4 + 0] = v;
                red[warp * (kPassMaxRows * 4) + m * 4 + 1] = __int_as_float(i);
                red[warp * (kPassMaxRows * 4) + m * 4 + 2] = sc;
            }
        }
        consumers_sync();
        if (tid < M) {
            float v = -INFINITY, sc = -INFINITY;
            int i = INT_MAX;
            for (int w = 0; w < kPassConsumerWarps; ++w)
                top2_merge(v, i, sc, red[w * (kPassMaxRows * 4) + tid * 4 + 0], __float_as_int(red[w * (kPassMaxRows * 4) + tid * 4 + 1]),
                           red[w * (kPassMaxRows * 4) + tid * 4 + 2]);
            float* lmp = p.partials + (size_t)p.n_resid * gridDim.x * kPassMaxRows * 4;
            lmp[((size_t)blockIdx.x * kPassMaxRows + tid) * 4 + 0] = v;
            lmp[((size_t)blockIdx.x * kPassMaxRows + tid) * 4 + 1] = __int_as_float(i);
            lmp[((size_t)blockIdx.x * kPassMaxRows + tid) * 4 + 2] = sc;
        }
    }
    } else {
        if (type == kStOproj || type == kStDown)
            epi_resid_rows<M>(p.x, psum, red, p.partials + ((size_t)st.resid_slot * gridDim.x + blockIdx.x) * kPassMaxRows * 4, n_rows, pair0, np, S,
                              pre0);
        else if (type == kStQkv)
            epi_qkv_rows<M>(psum, pair0, np, S, p.pos0, p.d_model, p.kv_dim, p.head_dim, p.rope_cos, p.rope_sin, p.q, st.k_cache, st.v_cache, pre0,
                            pre1);
        else if (type == kStGateUp)
            epi_gateup_rows<M>(psum, pair0, np, S, p.t, n_rows >> 1);
        else
            epi_lmhead_rows<M>(psum, red, pair0, np, S, n_rows, p.logits_out,
                               p.partials + ((size_t)p.n_resid * gridDim.x + blockIdx.x) * kPassMaxRows * 4);
    }
    if (type == kStLmHead) {
        if (last_cta_consumers(p.fin_counter, sm.flag)) {
            int* g = reinterpret_cast<int*>(red);
            for (int m = warp; m < M; m += kPassConsumerWarps) {  // a warp per row: lanes scan the per-CTA partials, then a butterfly; ties -> lowest index
                float v = -INFINITY, sc = -INFINITY;
                int i = INT_MAX;
                const float* lmp = p.partials + (size_t)p.n_resid * gridDim.x * kPassMaxRows * 4;
                for (unsigned b = lane; b < gridDim.x; b += 32) {
                    const float4 o4 = __ldcg(reinterpret_cast<const float4*>(lmp + ((size_t)b * kPassMaxRows + m) * 4));
                    top2_merge(v, i, sc, o4.x, __float_as_int(o4.y), o4.z);
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    const float ov = __shfl_xor_sync(0xffffffffu, v, o);
                    const int oi = __shfl_xor_sync(0xffffffffu, i, o);
                    const float os = __shfl_xor_sync(0xffffffffu, sc, o);
                    top2_merge(v, i, sc, ov, oi, os);
                }
                if (lane == 0) {
                    if (i == INT_MAX) i = 0;
                    p.argmax_out[m] = i;
                    if (p.margin_out) p.margin_out[m] = v - sc;
                    g[m] = i;
                }
            }
            consumers_sync();
            if (tid == 0) {
                if (p.accept_out && p.row_tokens) {
                    // greedy verification (Section 1): drafted token j+1 is accepted while it equals M's argmax of row j
                    int a = 0;
                    while (a < M - 1 && p.row_tokens[a + 1] == g[a]) ++a;
                    p.accept_out[0] = a;
                    for (int j = 0; j < a; ++j) p.accept_out[1 + j] = p.row_tokens[j + 1];
                    p.accept_out[1 + a] = g[a];
                }
                *p.fin_counter = 0u;
            }
        }
    }
}

// ============================================================================================ finish stage
// Cosine similarities of all residual stages of the pass (summand of C_l, Section 3.2). Residual stage r is
// finished by CTA r mod gridDim.x: one warp per activation row adds the per-CTA partials b = lane, lane+32, ...
// in order, then an xor butterfly, all in double precision (fixed order, independent of the row count).
template <int M>
__device__ void finish_stage(const PassParams& p, const PassSmem& sm) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int r = blockIdx.x; r < p.n_resid; r += gridDim.x) {
        const float* part = p.partials + (size_t)r * gridDim.x * kPassMaxRows * 4;
        const ResidOut out = p.resid[r];
        for (int m = warp; m < M; m += kPassConsumerWarps) {
            double sxy = 0, sxx = 0, syy = 0;
            for (unsigned b = lane; b < gridDim.x; b += 32) {
                sxy += (double)__ldcg(part + ((size_t)b * kPassMaxRows + m) * 4 + 0);
                sxx += (double)__ldcg(part + ((size_t)b * kPassMaxRows + m) * 4 + 1);
                syy += (double)__ldcg(part + ((size_t)b * kPassMaxRows + m) * 4 + 2);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                sxy += __shfl_xor_sync(0xffffffffu, sxy, o);
                sxx += __shfl_xor_sync(0xffffffffu, sxx, o);
                syy += __shfl_xor_sync(0xffffffffu, syy, o);
            }
            if (lane == 0) {
                const double c = sxy / fmax(sqrt(sxx) * sqrt(syy), 1e-30);
                out.cos_out[m] = (float)c;
                sm.red[m] = (float)c;
            }
        }
        consumers_sync();
        if (tid == 0 && p.acc_sim && out.sumcos) {  // rows are added in order: chunked prefill equals one-shot prefill
            double acc = *out.sumcos;
            for (int m = 0; m < M; ++m) acc += (double)sm.red[m];
            *out.sumcos = acc;
        }
        consumers_sync();
    }
}

// ============================================================================================ attention stage
// Byte offset of (key row r of the 128-key tile, 16-byte chunk c of the head) inside the tile's ring slots.
struct TileAddr {
    int nhb, row_bytes, swz;
    __device__ __forceinline__ void locate(int r, int c, int& slot_in_tile, int& off) const {
        const int rg = r / kBoxKeys, rr = r % kBoxKeys;
        const int hb = (nhb > 1) ? (c >> 3) : 0;
        const int cc = (nhb > 1) ? (c & 7) : c;
        slot_in_tile = rg * nhb + hb;
        off = rr * row_bytes + ((swz ? (cc ^ (rr & 7)) : cc) << 4);
    }
};

template <int M, bool LL>
__device__ void attn_stage(const PassParams& p, const StageDesc& st, const PassSmem& sm, uint32_t& gi, int stage) {
    const int tid = threadIdx.x, warp = tid >> 5;
    const int hd = p.head_dim;
    const int nhb = hd > 64 ? hd / 64 : 1;
    const int box_cols = hd > 64 ? 64 : hd;
    const int tile_slots = (kAttnChunk / kBoxKeys) * nhb;
    int n_chunks, first;
    const int n_local = attn_local_items(p, M, n_chunks, first);
    const uint32_t gi0 = gi;
    gi += (uint32_t)(n_local * 2 * tile_slots);
    if (LL) trace_mark(p, stage, 1);  // tagged handoff: every item waits for exactly the words it needs
    else stage_begin(p, stage);      // all consumer warps, also those without attention work
    const uint32_t tag_in = p.pass_tag + (uint32_t)(stage - 1), tag_out = p.pass_tag + (uint32_t)stage;  // W_qkv's stage precedes this one
    unsigned ll_spins = 0;
    long long ll_t0 = 0;
    const int grp = warp >> 2;
    if (grp >= p.attn_groups) return;

    
    const int gt = tid & 127, glane = gt & 31, gwarp = gt >> 5;
    const int bar_id = 2 + grp;
    const int group = p.n_heads / p.n_kv_heads;
    const int vec_per_row = hd / 8;
    TileAddr ta{nhb, box_cols * 2, (box_cols * 2 == 128) ? 1 : 0};

    // per-group scratch in region A
    const size_t scratch_bytes = ((size_t)M * hd * 4 + (size_t)M * kAttnChunk * 4 + 4 * kPassMaxRows * 4 + 16 + 15) & ~(size_t)15;
    unsigned char* base = sm.reg_a + (size_t)grp * scratch_bytes;
    float* qs = reinterpret_cast<float*>(base);   // [M][hd]
    float* Ps = qs + M * hd;                       // [M][128]
    float* red = Ps + M * kAttnChunk;              // [4][kPassMaxRows]
    int* flag = reinterpret_cast<int*>(red + 4 * kPassMaxRows);

    int q_head = -1;   // head whose queries are in qs
    unsigned run_cnt = 0;  // chunks of the current head finished by this group and not yet reported
    for (int j = grp; j < n_local; j += p.attn_groups) {
        const int idx = first + j;
        const int kvh = idx / n_chunks, chunk = idx - kvh * n_chunks;
        const int key0 = chunk * kAttnChunk;
        const int last_pos = p.pos0 + M - 1;
        const int n_valid = min(kAttnChunk, last_pos + 1 - key0);
        const uint32_t gk = gi0 + (uint32_t)(j * 2 * tile_slots), gv = gk + tile_slots;
        auto slot_ptr = [&](uint32_t g) -> unsigned char* {
            int slot;
            uint32_t gen;
            ring_locate(p, g, slot, gen);
            return sm.ring + (size_t)slot * kSlotBytes;
        };

        // ---- K tile: wait for the boxes, then overwrite the rows this pass has just written (the producer may
        //      have copied the tile before the QKV stage of this pass stored them)
        constexpr int kQPerThread = (M * 256 + 127) / 128;  // head_dim <= 256
        unsigned short qreg[kQPerThread];
#pragma unroll
        for (int u = 0; u < kQPerThread; ++u) {  // the first head's queries are requested before waiting for the tile
            const int i = gt + u * 128;
            const int m = i / hd, e = i - m * hd;
            qreg[u] = (!LL && i < M * hd && q_head != kvh * group) ? __ldcg(reinterpret_cast<const unsigned short*>(p.q) + (size_t)m * p.d_model + (size_t)(kvh * group) * hd + e) : 0;
        }
        // tagged handoff (one row): first look at this thread's words of q and of the fresh k and v; stale ones are asked for again where they are used
        constexpr int kLLPer = LL ? 2 : 1;  // head_dim <= 256: at most two elements per thread
        unsigned long long qraw[kLLPer] = {}, kraw[kLLPer] = {}, vraw[kLLPer] = {};
        const bool has_fresh = LL && key0 <= p.pos0 && p.pos0 < key0 + kAttnChunk;
        if (LL) {
#pragma unroll
            for (int u = 0; u < kLLPer; ++u) {
                const int e = gt + u * 128;
                if (e < hd) {
                    if (q_head != kvh * group) qraw[u] = ll_load1(p.ql + (size_t)(kvh * group) * hd + e);
                    if (has_fresh) kraw[u] = ll_load1(p.kl + (size_t)kvh * hd + e), vraw[u] = ll_load1(p.vl + (size_t)kvh * hd + e);
                }
            }
        }
        const int fresh0 = max(p.pos0, key0), fresh1 = min(last_pos, key0 + kAttnChunk - 1);
        const int n_fresh = fresh1 - fresh0 + 1;
        // one or two rows: the fresh V rows are requested here too, so patching the V tile later costs no round trip
        constexpr bool kVEarly = (M <= 2);
        constexpr int kVPre = kVEarly ? (M * 32 + 127) / 128 : 1;  // head_dim <= 256: at most 32 vectors per row
        uint4 vpre[kVPre];
        if (kVEarly && !LL) {
#pragma unroll
            for (int u = 0; u < kVPre; ++u) {
                const int i = gt + u * 128;
                vpre[u] = make_uint4(0u, 0u, 0u, 0u);
                if (i < n_fresh * vec_per_row) {
                    const int fr = i / vec_per_row, c = i - fr * vec_per_row;
                    vpre[u] = __ldcg(reinterpret_cast<const uint4*>(st.v_cache + (size_t)(fresh0 + fr) * p.kv_dim + (size_t)kvh * hd + c * 8));
                }
            }
        }
        for (int t = 0; t < tile_slots; ++t) ring_wait_full(p, sm, gk + t, stage, M * 1000 + j);
        if (LL) {
            if (has_fresh) {  // this pass's key (element by element from the tagged words) over whatever the producer copied
#pragma unroll
                for (int u = 0; u < kLLPer; ++u) {
                    const int e = gt + u * 128;
                    if (e < hd) {
                        while (!ll_ready(kraw[u], tag_in) && ll_keep_waiting(p, ll_spins, ll_t0, stage)) kraw[u] = ll_load1(p.kl + (size_t)kvh * hd + e);
                        int sit, off;
                        ta.locate(p.pos0 - key0, e >> 3, sit, off);
                        *reinterpret_cast<unsigned short*>(slot_ptr(gk + sit) + off + (e & 7) * 2) = (unsigned short)kraw[u];
                    }
                }
            }
        } else if (n_fresh > 0) {
            for (int i = gt; i < n_fresh * vec_per_row; i += 128) {
                const int fr = i / vec_per_row, c = i - fr * vec_per_row;
                const int r = fresh0 + fr - key0;
                int sit, off;
                ta.locate(r, c, sit, off);
                *reinterpret_cast<uint4*>(slot_ptr(gk + sit) + off) =
                    __ldcg(reinterpret_cast<const uint4*>(st.k_cache + (size_t)(fresh0 + fr) * p.kv_dim + (size_t)kvh * hd + c * 8));
            }
        }
        for (int g = 0; g < group; ++g) {
            const int head = kvh * group + g;
            bar_sync(bar_id, 128);  // patched tile visible; previous head's Ps / qs consumed
            if (LL) {
                if (q_head != head) {
#pragma unroll
                    for (int u = 0; u < kLLPer; ++u) {
                        const int e = gt + u * 128;
                        if (e < hd) {
                            if (g > 0) qraw[u] = ll_load1(p.ql + (size_t)head * hd + e);
                            while (!ll_ready(qraw[u], tag_in) && ll_keep_waiting(p, ll_spins, ll_t0, stage)) qraw[u] = ll_load1(p.ql + (size_t)head * hd + e);
                            qs[e] = __uint_as_float((uint32_t)qraw[u] << 16);
                        }
                    }
                }
            } else if (g == 0) {
                if (q_head != head) {
#pragma unroll
                    for (int u = 0; u < kQPerThread; ++u)
                        if (gt + u * 128 < M * hd) qs[gt + u * 128] = __uint_as_float((uint32_t)qreg[u] << 16);
                }
            } else {
                for (int i = gt; i < M * hd; i += 128) {
                    const int m = i / hd, e = i - m * hd;
                    qs[i] = __uint_as_float((uint32_t)__ldcg(reinterpret_cast<const unsigned short*>(p.q) + (size_t)m * p.d_model + (size_t)head * hd + e) << 16);
                }
            }
            q_head = head;
            bar_sync(bar_id, 128);

            if (j == 0 && g == 0) trace_mark(p, stage, 2);  // attention timeline: 2 = inputs staged, 4 = softmax done, 5 = P V done, 6 = ticket taken / value tile released, 7 = merged
            // ---- scores: thread t owns key key0 + t. Four independent partial sums per row (16-byte chunk parity x half
            //      of the chunk) keep the chains of dependent FMAs short; they are added in a fixed order.
            float sc[M];
            {
                float s4[M][4];
#pragma unroll
                for (int m = 0; m < M; ++m) s4[m][0] = s4[m][1] = s4[m][2] = s4[m][3] = 0.f;
                const int rg = gt / kBoxKeys, rr = gt % kBoxKeys;
                const int chunks_per_box = box_cols / 8;  // even: head_dim >= 16
                for (int hb = 0; hb < nhb; ++hb) {
                    const unsigned char* krow = slot_ptr(gk + rg * nhb + hb) + rr * ta.row_bytes;
                    for (int cc0 = 0; cc0 < chunks_per_box; cc0 += 2) {
#pragma unroll
                        for (int par = 0; par < 2; ++par) {
                            const int cc = cc0 + par, c = hb * 8 + cc;
                            const uint4 kv = *reinterpret_cast<const uint4*>(krow + ((ta.swz ? (cc ^ (rr & 7)) : cc) << 4));
                            const float kf[8] = {bf_lo(kv.x), bf_hi(kv.x), bf_lo(kv.y), bf_hi(kv.y),
                                                 bf_lo(kv.z), bf_hi(kv.z), bf_lo(kv.w), bf_hi(kv.w)};
#pragma unroll
                            for (int m = 0; m < M; ++m) {
                                const float4 q0 = *reinterpret_cast<const float4*>(qs + m * hd + c * 8);
                                const float4 q1 = *reinterpret_cast<const float4*>(qs + m * hd + c * 8 + 4);
                                float a0 = s4[m][2 * par], a1 = s4[m][2 * par + 1];
                                a0 = fmaf(q0.x, kf[0], a0);
                                a1 = fmaf(q1.x, kf[4], a1);
                                a0 = fmaf(q0.y, kf[1], a0);
                                a1 = fmaf(q1.y, kf[5], a1);
                                a0 = fmaf(q0.z, kf[2], a0);
                                a1 = fmaf(q1.z, kf[6], a1);
                                a0 = fmaf(q0.w, kf[3], a0);
                                a1 = fmaf(q1.w, kf[7], a1);
                                s4[m][2 * par] = a0, s4[m][2 * par + 1] = a1;
                            }
                        }
                    }
                }
#pragma unroll
                for (int m = 0; m < M; ++m) sc[m] = (s4[m][0] + s4[m][1]) + (s4[m][2] + s4[m][3]);
            }
            // ---- chunk-local softmax statistics; the row at position pos0+m sees keys <= pos0+m
            const int key = key0 + gt;
            float cmax[M];
#pragma unroll
            for (int m = 0; m < M; ++m) {
                const bool ok = key <= p.pos0 + m;
                sc[m] = ok ? sc[m] * p.attn_scale : -INFINITY;
                const float v = warp_max(sc[m]);
                if (glane == 0) red[gwarp * kPassMaxRows + m] = v;
            }
            bar_sync(bar_id, 128);
            if (g == group - 1) {  // K tile no longer needed: hand its slots back to the producer
                if (gt == 0) {
                    fence_proxy_async_smem();
                    for (int t = 0; t < tile_slots; ++t) ring_release(p, sm, gk + t);
                }
            }
#pragma unroll
            for (int m = 0; m < M; ++m)
                cmax[m] = fmaxf(fmaxf(red[0 * kPassMaxRows + m], red[1 * kPassMaxRows + m]),
                                fmaxf(red[2 * kPassMaxRows + m], red[3 * kPassMaxRows + m]));
            bar_sync(bar_id, 128);
#pragma unroll
            for (int m = 0; m < M; ++m) {
                const float pe = (sc[m] == -INFINITY) ? 0.f : expf(sc[m] - cmax[m]);
                Ps[m * kAttnChunk + gt] = pe;
                const float v = warp_sum(pe);
                if (glane == 0) red[gwarp * kPassMaxRows + m] = v;
            }
            if (g == 0) {  // V tile: wait and patch once per item
                for (int t = 0; t < tile_slots; ++t) ring_wait_full(p, sm, gv + t, stage, M * 1000 + 500 + j);
                if (LL) {
                    if (has_fresh) {
#pragma unroll
                        for (int u = 0; u < kLLPer; ++u) {
                            const int e = gt + u * 128;
                            if (e < hd) {
                                while (!ll_ready(vraw[u], tag_in) && ll_keep_waiting(p, ll_spins, ll_t0, stage)) vraw[u] = ll_load1(p.vl + (size_t)kvh * hd + e);
                                int sit, off;
                                ta.locate(p.pos0 - key0, e >> 3, sit, off);
                                *reinterpret_cast<unsigned short*>(slot_ptr(gv + sit) + off + (e & 7) * 2) = (unsigned short)vraw[u];
                            }
                        }
                    }
                } else if (kVEarly) {
#pragma unroll
                    for (int u = 0; u < kVPre; ++u) {
                        const int i = gt + u * 128;
                        if (i < n_fresh * vec_per_row) {
                            const int fr = i / vec_per_row, c = i - fr * vec_per_row;
                            int sit, off;
                            ta.locate(fresh0 + fr - key0, c, sit, off);
                            *reinterpret_cast<uint4*>(slot_ptr(gv + sit) + off) = vpre[u];
                        }
                    }
                } else if (n_fresh > 0) {
                    for (int i = gt; i < n_fresh * vec_per_row; i += 128) {
                        const int fr = i / vec_per_row, c = i - fr * vec_per_row;
                        const int r = fresh0 + fr - key0;
                        int sit, off;
                        ta.locate(r, c, sit, off);
                        *reinterpret_cast<uint4*>(slot_ptr(gv + sit) + off) =
                            __ldcg(reinterpret_cast<const uint4*>(st.v_cache + (size_t)(fresh0 + fr) * p.kv_dim + (size_t)kvh * hd + c * 8));
                    }
                }
            }
            bar_sync(bar_id, 128);
            if (gt < M) {
                const float l = ((red[0 * kPassMaxRows + gt] + red[1 * kPassMaxRows + gt]) + red[2 * kPassMaxRows + gt]) + red[3 * kPassMaxRows + gt];
                if (LL) ll_store(p.pl_ml + ((size_t)head * p.chunk_stride + chunk) * 2 + 1, __float_as_uint(l), tag_out);
                else p.part_ml[(((size_t)head * p.chunk_stride + chunk) * kPassMaxRows + gt) * 2 + 1] = l;
            }
            if (gt == 0) {
#pragma unroll
                for (int m = 0; m < M; ++m) {
                    if (LL) ll_store(p.pl_ml + ((size_t)head * p.chunk_stride + chunk) * 2 + 0, __float_as_uint(cmax[m]), tag_out);
                    else p.part_ml[(((size_t)head * p.chunk_stride + chunk) * kPassMaxRows + m) * 2 + 0] = cmax[m];
                }
            }
            if (j == 0 && g == 0) trace_mark(p, stage, 4);
            // ---- P V: thread (c, kg) owns the 8 output dimensions of 16-byte chunk c for the keys kg, kg + 8, ... (one
            //      16-byte read per key); the eight key groups of a chunk sit in neighbouring lanes and are added by an
            //      xor butterfly. Up to six rows share one sweep over the keys (more rows: two or more sweeps).
            //      Probabilities past n_valid are zero and the tile rows behind them hold finite cache contents.
            {
                constexpr int kRowBatch = M <= 6 ? M : (M <= 12 ? (M + 1) / 2 : 4);
                const int kg = gt & 7;
                const int n_steps = (n_valid + 7) >> 3;  // keys kg + 8 i, i < n_steps
                for (int c0 = 0; c0 < (hd >> 3); c0 += 16) {  // every lane runs the loop (the butterfly below is warp-wide)
                    const bool active = c0 + (gt >> 3) < (hd >> 3);
                    const int c = active ? c0 + (gt >> 3) : 0;
                    const int hb = (nhb > 1) ? (c >> 3) : 0, cc = (nhb > 1) ? (c & 7) : c;
                    const int coff = (ta.swz ? (cc ^ kg) : cc) << 4;  // key & 7 == kg for every key of this thread
#pragma unroll 1
                    for (int m0 = 0; m0 < M; m0 += kRowBatch) {
                        float acc[kRowBatch][8];
#pragma unroll
                        for (int u = 0; u < kRowBatch; ++u)
#pragma unroll
                            for (int d8 = 0; d8 < 8; ++d8) acc[u][d8] = 0.f;
                        for (int i = 0; i < n_steps; ++i) {
                            const int key = kg + 8 * i;
                            const unsigned char* vrow = slot_ptr(gv + (key / kBoxKeys) * nhb + hb) + (key % kBoxKeys) * ta.row_bytes + coff;
                            const uint4 vv = *reinterpret_cast<const uint4*>(vrow);
                            const float vf[8] = {bf_lo(vv.x), bf_hi(vv.x), bf_lo(vv.y), bf_hi(vv.y), bf_lo(vv.z), bf_hi(vv.z), bf_lo(vv.w), bf_hi(vv.w)};
#pragma unroll
                            for (int u = 0; u < kRowBatch; ++u)
                                if (m0 + u < M) {
                                    const float pw = Ps[(m0 + u) * kAttnChunk + key];
#pragma unroll
                                    for (int d8 = 0; d8 < 8; ++d8) acc[u][d8] = fmaf(pw, vf[d8], acc[u][d8]);
                                }
                        }
#pragma unroll
                        for (int u = 0; u < kRowBatch; ++u)
                            if (m0 + u < M) {
#pragma unroll
                                for (int d8 = 0; d8 < 8; ++d8) {
                                    float v = acc[u][d8];
                                    v += __shfl_xor_sync(0xffffffffu, v, 1);
                                    v += __shfl_xor_sync(0xffffffffu, v, 2);
                                    v += __shfl_xor_sync(0xffffffffu, v, 4);
                                    acc[u][d8] = v;
                                }
                                if (kg == 0 && active) {
                                    if (LL) {
                                        uint2* dst = p.pl_acc + ((size_t)head * p.chunk_stride + chunk) * hd + c * 8;
#pragma unroll
                                        for (int d8 = 0; d8 < 8; ++d8) ll_store(dst + d8, __float_as_uint(acc[u][d8]), tag_out);
                                    } else {
                                        float* dst = p.part_acc + (((size_t)head * p.chunk_stride + chunk) * kPassMaxRows + m0 + u) * hd + c * 8;
                                        reinterpret_cast<float4*>(dst)[0] = make_float4(acc[u][0], acc[u][1], acc[u][2], acc[u][3]);
                                        reinterpret_cast<float4*>(dst)[1] = make_float4(acc[u][4], acc[u][5], acc[u][6], acc[u][7]);
                                    }
                                }
                            }
                    }
                }
            }
        }
        if (j == 0) trace_mark(p, stage, 5);
        // ---- release the V tile. Finished chunks are reported once per run of chunks of the same head; the group
        //      whose report completes the head merges its chunks in order.
        ++run_cnt;
        const int jn = j + p.attn_groups;
        const bool report = (jn >= n_local) || ((first + jn) / n_chunks != kvh);
        bar_sync(bar_id, 128);
        if (LL) {
            // Tagged handoff: no ticket (the heads are merged in a second sweep below)
            if (gt == 0) {
                fence_proxy_async_smem();
                for (int t = 0; t < tile_slots; ++t) ring_release(p, sm, gv + t);
            }
            if (j == 0) trace_mark(p, stage, 6);
            continue;
        }
        if (gt == 0) {
            fence_proxy_async_smem();
            for (int t = 0; t < tile_slots; ++t) ring_release(p, sm, gv + t);
            if (report) {
                // release: the group's partial results (ordered before this thread by the barrier above) are visible
                // to whoever reads the count; acquire: so are those of the groups that reported earlier
                unsigned tk;
                asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(tk) : "l"(p.attn_counters + kvh), "r"(run_cnt) : "memory");
                *flag = (tk + run_cnt == (unsigned)n_chunks) ? 1 : 0;
            } else {
                *flag = 0;
            }
        }
        if (report) run_cnt = 0;
        bar_sync(bar_id, 128);
        if (j == 0) trace_mark(p, stage, 6);
        if (*flag) {
            if (gt == 0) p.attn_counters[kvh] = 0u;
            // warp w of the group merges rows w, w+4, ...; a lane owns four neighbouring output dimensions. The chunks
            // are merged in ascending order, eight loads of a batch in flight together; explicit roundings keep the
            // arithmetic identical in every instantiation of the kernel.
            for (int g = 0; g < group; ++g) {
                const int head = kvh * group + g;
                for (int e4 = glane * 4; e4 < hd; e4 += 128) {
                    for (int m = gwarp; m < M; m += 4) {
                        const int nc = (p.pos0 + m) / kAttnChunk + 1;
                        float mx = -INFINITY, l = 0.f, acc[4] = {0.f, 0.f, 0.f, 0.f};
                        for (int c0 = 0; c0 < nc; c0 += 8) {
                            float2 ml[8];
                            float4 pa[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                const int c = min(c0 + i, nc - 1);
                                const size_t b = ((size_t)head * p.chunk_stride + c) * kPassMaxRows + m;
                                ml[i] = __ldcg(reinterpret_cast<const float2*>(p.part_ml + b * 2));
                                pa[i] = __ldcg(reinterpret_cast<const float4*>(p.part_acc + b * hd + e4));
                            }
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                if (c0 + i < nc) {
                                    const float mn = fmaxf(mx, ml[i].x);
                                    const float s_old = expf(mx - mn), s_new = expf(ml[i].x - mn);
                                    acc[0] = __fmaf_rn(acc[0], s_old, __fmul_rn(pa[i].x, s_new));
                                    acc[1] = __fmaf_rn(acc[1], s_old, __fmul_rn(pa[i].y, s_new));
                                    acc[2] = __fmaf_rn(acc[2], s_old, __fmul_rn(pa[i].z, s_new));
                                    acc[3] = __fmaf_rn(acc[3], s_old, __fmul_rn(pa[i].w, s_new));
                                    l = __fmaf_rn(l, s_old, __fmul_rn(ml[i].y, s_new));
                                    mx = mn;
                                }
                            }
                        }
                        const __nv_bfloat162 o01 = __floats2bfloat162_rn(__fdiv_rn(acc[0], l), __fdiv_rn(acc[1], l));
                        const __nv_bfloat162 o23 = __floats2bfloat162_rn(__fdiv_rn(acc[2], l), __fdiv_rn(acc[3], l));
                        uint2 o;
                        o.x = *reinterpret_cast<const uint32_t*>(&o01);
                        o.y = *reinterpret_cast<const uint32_t*>(&o23);
                        if (LL) {
                            uint2* dst = p.al + (((size_t)m * p.d_model + (size_t)head * hd + e4) >> 1);
                            ll_store(dst, o.x, p.pass_tag + (uint32_t)stage);
                            ll_store(dst + 1, o.y, p.pass_tag + (uint32_t)stage);
                        } else {
                            *reinterpret_cast<uint2*>(p.a + (size_t)m * p.d_model + (size_t)head * hd + e4) = o;
                        }
                    }
                }
            }
        }
        if (j == 0) trace_mark(p, stage, 7);
    }
    if (LL) {
        // Tagged handoff, second sweep: the group that took a head's last chunk (the one with this pass's key) merges the
        // head, after ALL its items: it asks for the chunks' partial results until their tags are this stage's. Nobody who
        // produces a partial result ever waits for a merge, so the wait ends; merging inside the first sweep would hold
        // this CTA's later items (and through the ring its other groups) behind chunks that other CTAs reach last.
        for (int j = grp; j < n_local; j += p.attn_groups) {
            const int idx = first + j;
            const int kvh = idx / n_chunks, chunk = idx - kvh * n_chunks;
            if (chunk != n_chunks - 1) continue;
            for (int g = 0; g < group; ++g) {
                const int head = kvh * group + g;
                for (int e0 = 0; e0 < hd; e0 += 128) {  // one output dimension per thread (every lane runs the loop: shuffle below)
                    const int e = e0 + gt;
                    const bool act = e < hd;
                    float mx = -INFINITY, l = 0.f, acc = 0.f;
                    // Lane i of every warp fetches (maximum, sum of weights) of chunk c0 + i, 32 chunks per memory round trip,
                    // and hands them round by shuffle; every thread fetches its own dimension's sums 16 chunks at a time
                    for (int c0 = 0; c0 < n_chunks; c0 += 32) {
                        unsigned long long rm = 0, rl = 0;
                        bool ml_stale = c0 + glane < n_chunks;
#pragma unroll 1
                        for (int c1 = c0; c1 < c0 + 32 && c1 < n_chunks; c1 += 16) {
                            unsigned long long ra[16] = {};
                            unsigned stale = 0u;
#pragma unroll
                            for (int i = 0; i < 16; ++i)
                                if (act && c1 + i < n_chunks) stale |= 1u << i;
                            for (;;) {
                                if (ml_stale) ll_load2(p.pl_ml + ((size_t)head * p.chunk_stride + c0 + glane) * 2, rm, rl);
#pragma unroll
                                for (int i = 0; i < 16; ++i)
                                    if (stale & (1u << i)) ra[i] = ll_load1(p.pl_acc + ((size_t)head * p.chunk_stride + c1 + i) * hd + e);
                                if (ml_stale && ll_ready(rm, tag_out) && ll_ready(rl, tag_out)) ml_stale = false;
#pragma unroll
                                for (int i = 0; i < 16; ++i)
                                    if ((stale & (1u << i)) && ll_ready(ra[i], tag_out)) stale &= ~(1u << i);
                                if ((stale == 0u && !ml_stale) || !ll_keep_waiting(p, ll_spins, ll_t0, stage)) break;
                                __nanosleep(100u);
                            }
                            __syncwarp();
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                if (c1 + i < n_chunks) {  // (uniform) same arithmetic as the merge of the other instantiations
                                    const float cm = __uint_as_float(__shfl_sync(0xffffffffu, (uint32_t)rm, (c1 - c0) + i));
                                    const float cl = __uint_as_float(__shfl_sync(0xffffffffu, (uint32_t)rl, (c1 - c0) + i));
                                    const float mn = fmaxf(mx, cm);
                                    const float s_old = expf(mx - mn), s_new = expf(cm - mn);
                                    acc = __fmaf_rn(acc, s_old, __fmul_rn(__uint_as_float((uint32_t)ra[i]), s_new));
                                    l = __fmaf_rn(l, s_old, __fmul_rn(cl, s_new));
                                    mx = mn;
                                }
                            }
                        }
                    }
                    const uint32_t ob = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(__fdiv_rn(acc, l)));
                    const uint32_t up = __shfl_down_sync(0xffffffffu, ob, 1);
                    if (act && (gt & 1) == 0) ll_store(p.al + (((size_t)head * hd + e) >> 1), ob | (up << 16), tag_out);
                }
            }
        }
        if (grp == 0) trace_mark(p, stage, 7);
    }
}

// ============================================================================================ the kernel
template <int M, bool LL>
__global__ void __launch_bounds__(kPassThreads, 1) pass_kernel(const __grid_constant__ PassParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* base = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    PassSmem sm;
    sm.ring = base;
    sm.full = reinterpret_cast<uint64_t*>(base + p.off_bars);
    sm.empty = sm.full + p.ns;
    sm.red = reinterpret_cast<float*>(base + p.off_misc);
    sm.flag = reinterpret_cast<int*>(sm.red + 16 * kPassMaxRows * 4);
    sm.consumed = reinterpret_cast<volatile unsigned*>(sm.flag + 8);
    int* split = reinterpret_cast<int*>(const_cast<unsigned*>(sm.consumed) + 64);
    sm.split = split;
    sm.psum = reinterpret_cast<float*>(base + p.off_psum);
    sm.reg_a = base + p.off_reg_a;

    if (threadIdx.x == 0) {
        for (int i = 0; i < p.ns; ++i) {
            mbar_init(&sm.full[i], 1);
            mbar_init(&sm.empty[i], 1);
            sm.consumed[i] = 0u;
        }
        mbar_fence_init();
    }
    if (threadIdx.x >= 32 && threadIdx.x < 40) {  // split table: rows of the matrix of every stage type
        const int type = threadIdx.x - 32;
        const int n_rows = type == kStQkv ? p.d_model + 2 * p.kv_dim
                         : (type == kStOproj || type == kStDown) ? p.d_model
                         : type == kStGateUp ? 2 * p.d_ffn
                         : type == kStLmHead ? p.vocab : 0;
        int pair0 = 0, np = 0;
        if (n_rows > 0) cta_pairs(n_rows, type, pair0, np);
        const int n_oct = (np + kGrpPairs - 1) / kGrpPairs;
        // fewer groups than warps: several warp sets share a group (see gemv_stage)
        split[type * 4 + 0] = pair0, split[type * 4 + 1] = np, split[type * 4 + 2] = n_oct;
        split[type * 4 + 3] = (n_oct > 0 && n_oct < 8) ? kPassConsumerWarps / n_oct : 1;
    }
    __syncthreads();

    if (threadIdx.x >= kPassConsumers) {
        pass_producer<M>(p, sm);
        return;
    }

    uint32_t gi = 0;
    if (p.trace && threadIdx.x == 0) {  // which SM runs this CTA (entry 4 of the embedding stage, which streams nothing)
        unsigned smid;
        asm volatile("mov.u32 %0, %smid;" : "=r"(smid));
        p.trace[((size_t)0 * kTraceEntries + 4) * gridDim.x + blockIdx.x] = smid;
    }
    for (int s = 0; s < p.n_stages; ++s) {
        trace_mark(p, s, 0);
        const StageDesc st = p.stages[s];  // static: read before waiting for the previous stage
        const int next_type = (s + 1 < p.n_stages) ? p.stages[s + 1].type : -1;  // (read now: at the end of the stage it would be a round trip)
        // the next descriptor is requested now so that reading it at the next stage boundary hits L1
        if (threadIdx.x < 2 && s + 1 < p.n_stages)
            asm volatile("prefetch.global.L1 [%0];" ::"l"(reinterpret_cast<const char*>(p.stages + s + 1) + threadIdx.x * 64));
        if (p.trace && threadIdx.x == 0) p.trace[((size_t)s * kTraceEntries + 11) * gridDim.x + blockIdx.x] = st.type >= 0 ? global_ns() : 0;  // descriptor read
        if (st.type == kStEmbed) {
            stage_begin(p, s);
            const int d = p.d_model;
            for (int i = blockIdx.x * kPassConsumers + threadIdx.x; i < M * d; i += gridDim.x * kPassConsumers) {
                const int m = i / d, e = i - m * d;
                int t = __ldcg(p.tokens + m);
                t = min(max(t, 0), p.vocab - 1);
                const float v = __bfloat162float(p.embed[(size_t)t * d + e]);
                if (LL) ll_store(p.xl + i, __float_as_uint(v), p.pass_tag);
                else p.x[i] = v;
            }
        } else if (st.type == kStFinish) {
            stage_begin(p, s, p.bar_extra_last);  // (test hook: extra arrivals that never come)
            finish_stage<M>(p, sm);
        } else if (st.type == kStAttn) {
            attn_stage<M, LL>(p, st, sm, gi, s);
        } else {
            gemv_stage<M, LL>(p, st, sm, gi, s);
        }
        trace_mark(p, s, 3);
        // With the tagged handoff only the finish stage still waits at the grid barrier: the arrival in front of it
        // publishes everything this CTA has written so far, the others just count.
        bool release = true;
        if (LL && next_type >= 0) release = (next_type == kStFinish);
        grid_arrive(p, release);
    }
}

}  // namespace asd
