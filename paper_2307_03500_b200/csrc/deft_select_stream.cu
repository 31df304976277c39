// Layer-wise top-k selection (Algorithm 5) in ONE pass over the call's part of the vector: the kernel for
// large calls whose layers were selected from before on the same workspace (a training loop).
//
// Every layer comes with a remembered cut (predict_cut in deft_select_dev.cuh).  One CTA of 512 threads
// per SM; the call's tiles are dealt to the CTAs in stripes.  Whole tiles arrive through a ring of
// bulk copies in shared memory (or, in the kernel's other form, by plain loads); a warp takes a tile into
// registers, tests it against the cut (one floating-point test per 16-byte load, the exact test only
// where that one passes) and moves the entries at or above the cut, in index order, into the CTA's shared
// memory.  At the end of its read the CTA copies what it staged into the layers' regions of the staging
// area (one atomic per CTA and layer reserves the room) and writes (first entry, entries) per tile.
// With `prestaged` the accumulate pass has done all of this already and the kernel starts here:
//
// Behind a grid barrier every layer is finished by one CTA (largest first, from a queue): if at least k
// entries were staged, the k largest of the layer are among them; a histogram of fine bins counted from
// the cut gives the bin of the k-th largest, the few entries of that bin are ranked among themselves,
// and the selected entries are written in ascending index (value, int64 index; equal keys: lowest indices
// first) from the tile table: per-tile counts, a prefix over the layer's tiles, an ordered write.
// Behind a second barrier the whole grid clears the selected entries in the vector, and the layers that
// could not be finished (fewer than k staged entries, far too many, no usable cut, too dense, k too
// large for one CTA) go through the five steps (deft_select_steps.cuh) inside the same launch.
// The result never depends on the cuts.
//
// Layers of at most kDirectElems elements are handed out from a counter; one CTA loads each whole.
//
// Determinism: staging order inside a CTA and the order of the CTAs' chunks in a layer's region depend
// on timing, but every output position is a function of counts and of the tile an entry came from.
#include "deft_select_steps.cuh"

namespace cg = cooperative_groups;

namespace deft {
namespace {

constexpr uint32_t kStreamRes = kSmMainBytes / 8;   // staged entries a CTA keeps in shared memory
constexpr uint32_t kFloodFactor = 8;                 // a CTA stops staging beyond this multiple of what its layers should stage
constexpr uint32_t kTileGlobal = 0xffffffffu;       // TileTable::first of a tile whose entries went straight to global memory
static_assert(kBins1 * 4 <= kSmAuxBytes, "the finishing CTA's histograms live in the aux region");

// staged entry in a layer's region: .x = value bits, .y = offset in tile | tile within the layer << 11
__device__ __forceinline__ uint32_t region_y(uint32_t off, uint32_t tile_in_layer) { return off | (tile_in_layer << 11); }

// Appends layer j of the call to the retry list (one thread).  The layer gets a place in the list, a
// run of tiles and a staging region of its own (a multiple of kTile entries from the call's base).
__device__ __noinline__ void push_retry(const SelParams& p, int j) {
    const uint32_t tiles = (uint32_t)(p.desc[j + 1].tile_first - p.desc[j].tile_first);
    const unsigned long long old = atomicAdd(&p.retry->packed, (1ull << 32) | (unsigned long long)tiles);
    const uint32_t pos = (uint32_t)(old >> 32), tf = (uint32_t)old;
    LayerDesc d = p.desc[j];
    d.tile_first = (int32_t)tf;
    d.elem_off = p.retry_elem_base + (int64_t)tf * kTile;
    p.retry_desc[pos] = d;
    // the list's end marker: whoever appends the next layer writes the same number there again
    p.retry_desc[pos + 1].tile_first = (int32_t)(tf + tiles);
}

// ---------------------------------------------------------------------------------
// the finishing CTA
// ---------------------------------------------------------------------------------
// Code that runs once per layer and CTA is bound by instruction fetch and by round trips to L2, not by
// arithmetic (an instruction that is not in the SM's instruction cache costs several nanoseconds):
// what follows is written for few instructions and few dependent loads — plain loops, little
// unrolling, the layer's entries and its tile table fetched together.
//
// Which staged entries are selected is settled in two steps.  A histogram with bins of 2^kFineShift
// keys counted from the cut (1/4096 octave over one octave; the first-level buckets are 1/16, and the staged keys crowd
// into the few buckets right above the cut) gives the bin `a` of the k-th largest key: everything in a
// higher bin is selected, nothing in a lower one.  The few entries of bin a (the candidates) are ranked
// among themselves by (key descending, index ascending); the first k - (entries above bin a) of them
// are selected and get a flag in their entry.  No threshold key is ever needed.
constexpr int kFineShift = 11;
constexpr int kFineBins = kBins1;   // the top bin takes everything beyond
constexpr uint32_t kCandMax = 1024; // candidates that can be ranked; a layer with more goes to the retry list
constexpr uint32_t kSelFlag = 0x80000000u;   // in an entry's .y: a candidate that is selected
static_assert(kCandMax * 12 <= kSmAuxBytes && kFineShift <= kFinePosShift && kSelWarps == 16 &&
              DEFT_MAX_LAYER_ELEMS / kTile < (1 << 20),
              "candidates live in the aux region; bit 31 of .y is free; a warp id fits four bits");

__device__ __forceinline__ uint32_t fine_bin(uint32_t key, uint32_t cut) {
    const uint32_t b = (key - cut) >> kFineShift;
    return b < (uint32_t)kFineBins - 1u ? b : (uint32_t)kFineBins - 1u;
}

// A layer's staged entries: the first kStreamRes in shared memory, the rest in the layer's region
// (read through L1: regions start on 128-byte boundaries, a region is complete before its finishing CTA
// reads it, and no SM reads a region at any other time).
struct Staged {
    uint2* src;
    uint2* res;
    uint32_t S;
};
__device__ __forceinline__ uint2 staged_get(const Staged& f, uint32_t pos) {
    return pos < kStreamRes ? f.res[pos] : f.src[pos];
}

// CTA-wide pass over the staged entries in no particular order: f(entry, position).  The part that lives in
// global memory is read four entries per thread at a time (one round trip per four instead of one each).
template <typename F>
__device__ __forceinline__ void for_each_entry(const Staged& f, F fn) {
    const uint32_t nres = f.S < kStreamRes ? f.S : kStreamRes;
    for (uint32_t pos = threadIdx.x; pos < nres; pos += kSelThreads) fn(f.res[pos], pos);
    for (uint32_t p0 = kStreamRes + threadIdx.x; p0 < f.S; p0 += 4 * kSelThreads) {
        uint2 ent[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t pos = p0 + u * kSelThreads;
            ent[u] = pos < f.S ? f.src[pos] : make_uint2(0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t pos = p0 + u * kSelThreads;
            if (pos < f.S) fn(ent[u], pos);
        }
    }
}

// Diagnostic lap timer of the finishing CTA: adds the nanoseconds since the previous lap to timing[slot].
struct Lap {
    unsigned long long* timing;
    unsigned long long t0;
    __device__ __forceinline__ void start(unsigned long long* tm) {
        timing = tm;
        if (timing && threadIdx.x == 0) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    }
    __device__ __forceinline__ void lap(int slot) {
        if (timing && threadIdx.x == 0) {
            unsigned long long t;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
            atomicAdd(timing + slot, t - t0);
            t0 = t;
        }
    }
};

// One layer, finished by the CTA that completed its last tile.  c: local layer; S: entries staged for
// the layer by all CTAs; flooded: some CTA stopped staging.
__device__ __noinline__ bool finish_layer(const SelParams& p, LayerTable* lt, int c, uint32_t S, uint32_t flooded,
                                          TileTable* tt, unsigned char* smem) {
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kSmMisc);
    uint32_t* scratch = misc + kMScratch;
    uint32_t* out3 = misc + kMOut3;
    uint32_t* h = reinterpret_cast<uint32_t*>(smem + kSmAux);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int lid = lt->lid[c];
    const uint32_t k = lt->k[c], k_safe = safe_rank(k), cut = lt->sthr[c];
    Lap lap;
    lap.start(p.timing);
    LayerHint* hp = p.hint + lid;
    // (far more staged than selected: one CTA would take longer over them than the grid takes to read the
    // layer again)
    if (S < k || flooded || (unsigned long long)S > 6ull * k + 8192ull) {
        // the cut was too high (fewer than k entries reached the staging area) or far too low (a CTA
        // stopped staging): the layer goes to the retry list; a cut that was too high lowers the next ones
        if (tid == 0) {
            atomicAdd(p.spec_ctl + 5, 1u);
            push_retry(p, lt->j[c]);
        }
        return false;
    }
    Staged f;
    f.S = S;
    f.src = p.staging + lt->elem_off[c];
    f.res = reinterpret_cast<uint2*>(smem + kSmMain);
    const int tf = lt->tf[c], tn = lt->tfe[c] - tf;
    const uint2* tab = p.runge + tf;
    const int np0 = tn < kMaxLocalTiles ? tn : kMaxLocalTiles;
    // the entries and (the first pass of) the tile table are fetched together
    {
        const uint32_t nres = S < kStreamRes ? S : kStreamRes;
        // (two entries per load: regions start on 128-byte boundaries and have slack behind them)
        const uint4* src2 = reinterpret_cast<const uint4*>(f.src);
        uint4* res2 = reinterpret_cast<uint4*>(f.res);
#pragma unroll 8
        for (uint32_t pos = tid; pos < (nres + 1u) / 2u; pos += kSelThreads) res2[pos] = src2[pos];
#pragma unroll 4
        for (int t = tid; t < np0; t += kSelThreads) tt->first[t] = __ldcg(tab + t).x;
    }
    for (int i = tid; i < kFineBins; i += kSelThreads) h[i] = 0;
    if (tid == 0) misc[kMFlag] = 0u;   // candidates collected
    __syncthreads();
    lap.lap(20);
    for_each_entry(f, [&](const uint2 ent, uint32_t) { atomicAdd(&h[fine_bin(key_of(ent.x), cut)], 1u); });
    __syncthreads();
    lap.lap(21);
    block_scan_select(h, kFineBins, false, k, k_safe, scratch, out3);
    const uint32_t a = out3[0], krem = k - out3[1], a_safe = out3[2];
    const uint32_t C = h[a];
    __syncthreads();
    lap.lap(22);
    if (C > kCandMax) {
        // many equal or nearly equal keys around the k-th largest: not this routine's business
        if (tid == 0) {
            atomicAdd(p.spec_ctl + 5, 1u);
            push_retry(p, lt->j[c]);
        }
        return false;
    }
    if (tid == kSelThreads - 1) {   // (not thread 0: the loads it waits for are off the CTA's critical path this way)
        // what the next call starts from: the first-level bucket of the k_safe-th key if that many were
        // staged, else the bucket below this call's cut
        const double norm = p.desc[lt->j[c]].norm;
        if (S >= k_safe) {
            hint_update(hp, (cut >> kFinePosShift) + (a_safe >> (kFinePosShift - kFineShift)), true, 0, k, norm);
        } else {
            const uint32_t cutp = cut >> kFinePosShift;
            hint_update(hp, cutp > 0u ? cutp - 1u : 0u, false, 0, k, norm);
        }
        atomicAdd(p.spec_ctl + 4, 1u);
        atomicAdd(p.spec_ctl + 9, S);
    }
    // the candidates: (key, index order) as one 64-bit word that sorts the way the selection wants
    // (larger key first, then lower index: .y grows with the index and bit 31 of it is free), and
    // where the entry lives; the histogram's room is free now
    unsigned long long* cword = reinterpret_cast<unsigned long long*>(h);
    uint32_t* cpos = h + 2 * kCandMax;
    for_each_entry(f, [&](const uint2 ent, uint32_t pos) {
        if (fine_bin(key_of(ent.x), cut) == a) {
            const uint32_t i = atomicAdd(misc + kMFlag, 1u);
            cword[i] = ((unsigned long long)key_of(ent.x) << 32) | (0x7fffffffu - ent.y);
            cpos[i] = pos;
        }
    });
    __syncthreads();
    for (uint32_t i = tid; i < C; i += kSelThreads) {
        const unsigned long long mine = cword[i];
        uint32_t before = 0;
#pragma unroll 8
        for (uint32_t j = 0; j < C; ++j) before += cword[j] > mine ? 1u : 0u;
        if (before < krem) {
            const uint32_t pos = cpos[i];
            if (pos < kStreamRes) f.res[pos].y |= kSelFlag; else f.src[pos].y |= kSelFlag;
        }
    }
    __syncthreads();
    stamp(p, 10);
    lap.lap(23);
    if (p.timing && tid == 0) { atomicMax(p.timing + 14, (unsigned long long)S); atomicAdd(p.timing + 15, (unsigned long long)S); atomicMax(p.timing + 13, (unsigned long long)C); atomicMax(p.timing + 12, ((unsigned long long)S << 32) | ((unsigned long long)lid << 20) | (k < 0xfffffu ? k : 0xfffffu)); }
    // The ordered write.  An entry's place in the output is (selected entries of the layer's earlier tiles) +
    // (selected entries before it in its own tile).  A tile's entries are consecutive in the region, so the
    // second term is a difference of running counts along the region: two passes over the entries, each
    // warp over a contiguous range of them (32 consecutive entries per step: coalesced, and a ballot gives
    // the running count).  Pass 1 counts the selected entries per tile and notes the running count at
    // every tile's first entry; a prefix over the tiles and over the warps' totals; pass 2 writes.
    // Up to kMaxLocalTiles tiles of the layer per round.
    float* const val = p.val;
    int64_t* const idx = p.idx;
    const int64_t cap = p.out_cap;
    const int64_t tile0 = lt->start[c] / kTile;
    const int64_t out_off = lt->out_off[c];
    // Each warp walks two ranges: its share of the entries held in shared memory, then its share of
    // those left in the region (reading those costs a round trip to L2 per batch: they are spread over
    // all warps instead of falling to the last few).  2 * kSelWarps ranges in region order.
    uint32_t* wtot = misc + kMWarpCnt;   // per range: selected entries, then their exclusive prefix
    const uint32_t n_sm = S < kStreamRes ? S : kStreamRes;
    uint32_t w_lo_[2], w_hi_[2];
#pragma unroll
    for (int part = 0; part < 2; ++part) {
        const uint32_t p0 = part ? n_sm : 0u, p1 = part ? S : n_sm;
        const uint32_t per = ((p1 - p0 + kSelWarps - 1) / kSelWarps + 127u) & ~127u;
        w_lo_[part] = p0 + (uint32_t)warp * per < p1 ? p0 + (uint32_t)warp * per : p1;
        w_hi_[part] = w_lo_[part] + per < p1 ? w_lo_[part] + per : p1;
    }
    uint32_t base = 0;
    for (int tp = 0; tp < tn; tp += kMaxLocalTiles) {
        const int np = tn - tp < kMaxLocalTiles ? tn - tp : kMaxLocalTiles;
        if (tp > 0) {
#pragma unroll 4
            for (int t = tid; t < np; t += kSelThreads) tt->first[t] = __ldcg(tab + tp + t).x;
        }
        for (int t = tid; t < np; t += kSelThreads) tt->ge[t] = 0u;
        __syncthreads();
        // pass 1
        for (int part = 0; part < 2; ++part) {
        const uint32_t w_hi = part ? w_hi_[1] : w_hi_[0];
        const uint32_t vw = (uint32_t)(part * kSelWarps + warp);
        uint32_t run = 0;
        for (uint32_t p4 = part ? w_lo_[1] : w_lo_[0]; p4 < w_hi; p4 += 128) {   // four steps' entries are fetched together
            uint2 e4[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint32_t pos = p4 + u * 32 + lane;
                e4[u] = pos < w_hi ? staged_get(f, pos) : make_uint2(0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint32_t pos = p4 + u * 32 + lane;
                const bool valid = pos < w_hi;
                const uint2 ent = e4[u];
                const uint32_t t = ((ent.y & ~kSelFlag) >> 11) - (uint32_t)tp;   // tile within this round (or out of it)
                const bool here = valid && t < (uint32_t)np;
                const bool sel = here && ((fine_bin(key_of(ent.x), cut) > a) || (ent.y & kSelFlag));
                const unsigned ball = __ballot_sync(0xffffffffu, sel);
                if (here && tt->first[t] == pos) tt->first[t] = 0x80000000u | (vw << 26) | (run + __popc(ball & ((1u << lane) - 1u)));
                // a tile's entries are neighbours: the first lane of every run of equal tiles adds the run's count
                const uint32_t tkey = here ? t : 0xffffffffu;
                const uint32_t tprev = __shfl_up_sync(0xffffffffu, tkey, 1);
                const bool starts = lane == 0 || tkey != tprev;
                const unsigned sb = __ballot_sync(0xffffffffu, starts);
                if (starts && here) {
                    const unsigned above = sb & ~((2u << lane) - 1u);   // (2u << 31 == 0: nothing above lane 31)
                    const unsigned upto = above ? ((1u << (__ffs((int)above) - 1)) - 1u) : 0xffffffffu;
                    const uint32_t cnt = __popc(ball & upto & ~((1u << lane) - 1u));
                    if (cnt) atomicAdd(&tt->ge[t], cnt);
                }
                run += __popc(ball);
            }
        }
        if (lane == 0) wtot[vw] = run;
        }
        __syncthreads();
        lap.lap(24);
        if (warp == 0) {
            const uint32_t x = wtot[lane];
            wtot[lane] = warp_incl_scan(x, lane) - x;
        }
        // exclusive prefix of the tiles' counts: each thread a run of consecutive tiles
        const int m = (np + kSelThreads - 1) / kSelThreads;
        const int lo = tid * m < np ? tid * m : np, hi = lo + m < np ? lo + m : np;
        uint32_t mine = 0;
        for (int t = lo; t < hi; ++t) mine += tt->ge[t];
        uint32_t total;
        uint32_t before = base + block_excl_scan(mine, scratch, total);
        for (int t = lo; t < hi; ++t) {
            const uint32_t g = tt->ge[t];
            tt->ge[t] = before;
            before += g;
        }
        __syncthreads();
        lap.lap(25);
        // pass 2
        for (int part = 0; part < 2; ++part) {
        const uint32_t w_hi = part ? w_hi_[1] : w_hi_[0];
        uint32_t run = wtot[part * kSelWarps + warp];
        for (uint32_t p4 = part ? w_lo_[1] : w_lo_[0]; p4 < w_hi; p4 += 128) {
            uint2 e4[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint32_t pos = p4 + u * 32 + lane;
                e4[u] = pos < w_hi ? staged_get(f, pos) : make_uint2(0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
            const uint32_t pos = p4 + u * 32 + lane;
            const bool valid = pos < w_hi;
            const uint2 ent = e4[u];
            const uint32_t t = ((ent.y & ~kSelFlag) >> 11) - (uint32_t)tp;
            const bool here = valid && t < (uint32_t)np;
            const bool sel = here && ((fine_bin(key_of(ent.x), cut) > a) || (ent.y & kSelFlag));
            const unsigned ball = __ballot_sync(0xffffffffu, sel);
            if (sel) {
                const uint32_t mark = tt->first[t];   // where the tile's first entry stood: warp, running count
                const uint32_t at_first = wtot[(mark >> 26) & 31u] + (mark & 0x3ffffffu);
                const int64_t o = out_off + tt->ge[t] + (run + __popc(ball & ((1u << lane) - 1u)) - at_first);
                const int64_t elem = (tile0 + tp + t) * kTile + (int64_t)y_off(ent.y);
                if (o < cap) {
                    val[o] = __uint_as_float(ent.x);
                    idx[o] = elem;
                }
            }
            run += __popc(ball);
            }
        }
        }
        base += total;
        __syncthreads();   // the tables are rewritten by the next round
        lap.lap(26);
    }
    if (p.timing && tid == 0) atomicAdd(p.timing + 28, 1ull);
    return true;
}

// Out of line: the rare path must not cost the kernel's main loop registers.
__device__ __noinline__ void retry_steps(const SelParams& q, unsigned char* smem, cg::grid_group& grid) {
    five_steps(q, smem, grid);
}

// Tiles are dealt out to the CTAs in stripes of kStripe consecutive tiles, round-robin: every CTA gets an
// even sample of every layer of the call, so the layers whose entries crowd (large k_l / size_l) are
// everybody's business, and so is the second look at a layer whose cut failed.
constexpr int kStripe = 16;

// ---- the read through a ring of bulk copies (the kernel's second form) ----
// Instead of every warp loading its tile into registers and waiting for it, the CTA keeps
// kRingStages whole tiles in flight as bulk copies (cp.async.bulk, completion counted on an mbarrier
// per stage) into a ring in shared memory.  Tiles are handed to the warps in ascending order from a
// counter, so tile number n of the CTA always uses stage n % kRingStages; the warp that has taken
// tile n out of its stage (into registers) starts the copy of tile n + kRingStages into it.  Only whole
// tiles of layers with a cut go through the ring; for any other tile the stage's barrier just gets an
// arrival, so that every use of a stage is one phase of its barrier.  A parity wait can only tell a
// phase from its neighbour, so a warp first waits until its use of the stage has been started (a
// sequence word per stage, written after the copy is issued) and only then for the phase to complete.
// The ring takes its room from the shared-memory staging area, which keeps kRingRes entries during the read.
constexpr int kRingStages = 16;
constexpr uint32_t kTileBytes = kTile * 4;
// During the read the kernel's tile table (StreamTiles) sits in the second half of the tile-table area;
// the first half, the aux area and the main area are one stretch of shared memory for the staged entries and the ring.
struct StreamTiles {                 // per local tile of the CTA, see TileTable
    uint32_t first[kStreamLocalTiles];
    uint32_t ge[kStreamLocalTiles];
    uint16_t n[kStreamLocalTiles];
};
constexpr int kSmStreamTiles = kSmTile + kSmTileBytes - (int)sizeof(StreamTiles);
constexpr uint32_t kRingRes = (uint32_t)(kSmStreamTiles - kSmMain - kRingStages * (int)kTileBytes) / 8;
constexpr int kMRingBar = 164;    // misc words, two per stage: the stages' mbarriers
constexpr int kMRingDead = 162;   // misc word: a wait on the ring gave up; the CTA reads with plain loads from then on
constexpr int kMRingSeq = 200;    // misc words, one per stage: uses of the stage started so far
static_assert(kSmAux == kSmMain + kSmMainBytes && kSmTile == kSmAux + kSmAuxBytes && kSmStreamTiles % 128 == 0 &&
              kRingRes >= 4096 && (kRingRes * 8) % 128 == 0 && kMRingBar + 2 * kRingStages <= kMRingSeq && kMRingSeq + kRingStages <= 256 && kMRingBar % 2 == 0 &&
              kMWarpCnt + 32 <= kMRingDead, "ring: room, alignment, misc words");

__device__ __forceinline__ uint32_t smem_addr(const void* ptr) { return (uint32_t)__cvta_generic_to_shared(ptr); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded: a copy that has not landed after this many polls (seconds) never will.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    for (int i = 0; i < (1 << 22); ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(dst_smem)), "l"(src), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}

static_assert(kStreamLocalTiles % kStripe == 0 && kTfCache * 2 <= kSmSuperBytes, "stripes; the layer map lives in the super-tile area");

template <bool kRing>
__global__ void __launch_bounds__(kSelThreads, 1) k_select_stream(const SelParams p_in, const int has_streamed) {
    extern __shared__ __align__(16) unsigned char smem[];
    cg::grid_group grid = cg::this_grid();
    SelParams& p = params_in_smem(p_in, smem);
    if (p.timing && threadIdx.x == 0 && blockIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        p.timing[0] = t;
    }
    LayerTable* lt = reinterpret_cast<LayerTable*>(smem + kSmLayer);
    TileTable* tt = reinterpret_cast<TileTable*>(smem + kSmTile);                  // the finishing CTA's
    StreamTiles* rt = reinterpret_cast<StreamTiles*>(smem + kSmStreamTiles);       // the read's
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kSmMisc);
    uint32_t* wbase = reinterpret_cast<uint32_t*>(smem + kSmWBase);
    uint2* res = reinterpret_cast<uint2*>(smem + kSmMain);
    int* tfc = reinterpret_cast<int*>(smem + kSmTf);                    // first tile of every layer of the call (+ end)
    uint16_t* jmap = reinterpret_cast<uint16_t*>(smem + kSmSuper);      // layer of the call -> local (streamed) layer
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.x, G = gridDim.x;
    for (int i = threadIdx.x; i <= p.n_my; i += kSelThreads) tfc[i] = p.desc[i].tile_first;
    for (int i = threadIdx.x; i < p.n_my; i += kSelThreads) jmap[i] = 0xffffu;
    CtaRange r;
    r.il = 0; r.q0tab = nullptr; r.nsuper = 0;
    r.q0 = 0; r.q1 = p.tiles; r.nloc = 0;
    r.jA = 0; r.jB = p.n_my - 1;
    const int nl = build_layer_table(p, r, lt, misc + kMScratch, true, kErrUnit / 4, true);   // every streamed layer of the call
    const int nstripe = (p.tiles + kStripe - 1) / kStripe;
    // (prestaged: the accumulate pass has staged the call's entries and filled the tile table: nothing to read)
    const int nloc = p.prestaged ? 0 : (b < nstripe ? (nstripe - b + G - 1) / G : 0) * kStripe;
    if (threadIdx.x == 0) { misc[kMCursor] = 0; misc[kMTileCtr] = 0; misc[kMBudget] = 4096u; }
    constexpr uint32_t kReadRes = kRing ? kRingRes : kStreamRes;   // staged entries the CTA keeps in shared memory during the read
    uint64_t* const bars = reinterpret_cast<uint64_t*>(misc + kMRingBar);
    unsigned char* const ring = smem + kSmMain + kRingRes * 8;
    if (kRing && threadIdx.x == 0) {
        misc[kMRingDead] = 0u;
        for (int sg = 0; sg < kRingStages; ++sg) { mbar_init(bars + sg, 1); misc[kMRingSeq + sg] = 0u; }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // Starts the use of its stage by local tile lq (one thread): the copy of a whole tile of a layer with a cut, else an arrival.
    auto ring_issue = [&](int lq) {
        const int q = kStripe * (b + (lq / kStripe) * G) + lq % kStripe;
        const int sg = lq % kRingStages;
        uint64_t* bar = bars + sg;
        bool copied = false;
        const uint32_t m = rt->first[lq];   // the tile's layer (filled in before the read starts)
        if (m != 0xffffu) {
            const TileSpan ts = tile_span(lt->start[m], lt->end[m], lt->tf[m], q);
            if (ts.s == 0 && ts.e == kTile) {
                mbar_expect_tx(bar, kTileBytes);
                bulk_load(ring + (size_t)sg * kTileBytes, p.acc + ts.lo, kTileBytes, bar);
                copied = true;
            }
        }
        if (!copied) mbar_arrive(bar);
        __threadfence_block();
        *reinterpret_cast<volatile uint32_t*>(misc + kMRingSeq + sg) = (uint32_t)(lq / kRingStages) + 1u;
    };
    __syncthreads();
    for (int c = threadIdx.x; c < nl; c += kSelThreads) {
        jmap[lt->j[c]] = (uint16_t)c;
        lt->v0[c] = 0u;   // entries of the layer this CTA keeps in shared memory
        if (lt->sthr[c] == 0xffffffffu) {
            // no usable cut: the layer goes to the retry list (one CTA says so)
            if (c % G == b) {
                push_retry(p, lt->j[c]);
                atomicAdd(p.spec_ctl + 6, 1u);
            }
            continue;
        }
        // what the CTA may stage: a multiple of what its share of the layer's tiles should hold if the entries
        // down to the rank behind the cut were spread evenly.  A cut that turns out far too low must not
        // flood the staging area: past the budget the CTA stops reading, and the layers it skips tiles of
        // go to the retry list.
        const int64_t size = lt->end[c] - lt->start[c];
        const uint64_t per_tile = ((uint64_t)safe_rank(lt->k[c]) * kTile + size - 1) / size;
        const uint64_t want = ((uint64_t)(lt->tfe[c] - lt->tf[c]) / G + 1) * per_tile * kFloodFactor;
        atomicAdd(&misc[kMBudget], (uint32_t)(want < 0x3fffffffull ? want : 0x3fffffffull));
    }
    __syncthreads();
    stamp(p, 8);
    const uint32_t budget = misc[kMBudget] < 0x7fffffffu ? misc[kMBudget] : 0x7fffffffu;
    // which layer (of those with a cut) every tile of the CTA belongs to: looked up once, here; the tile's
    // slot in the table is rewritten when the tile has been read
    for (int lq = threadIdx.x; lq < nloc; lq += kSelThreads) {
        const int q = kStripe * (b + (lq / kStripe) * G) + lq % kStripe;
        uint32_t m = 0xffffu;
        if (q < p.tiles) {
            m = jmap[layer_of_tile_sh(tfc, p.n_my, q)];
            if (m != 0xffffu && lt->sthr[m] == 0xffffffffu) m = 0xffffu;
        }
        rt->first[lq] = m;
    }
    __syncthreads();
    if (kRing && (int)threadIdx.x < kRingStages && (int)threadIdx.x < nloc) ring_issue((int)threadIdx.x);

    // ---- the read: every tile of the CTA once ----
    for (int lq = grab_tile(misc + kMTileCtr, lane); lq < nloc; lq = grab_tile(misc + kMTileCtr, lane)) {
        const int q = kStripe * (b + (lq / kStripe) * G) + lq % kStripe;
        uint32_t first = 0, n = 0, off = 0;
        const uint32_t m = rt->first[lq];
        const int cl = m != 0xffffu ? (int)m : -1;
        TileSpan ts;
        ts.lo = 0; ts.s = 0; ts.e = 0;
        if (cl >= 0) ts = tile_span(lt->start[cl], lt->end[cl], lt->tf[cl], q);
        TileRegs t;
        uint32_t vm[2], keep[2];
        bool have = false;   // the tile is in registers already (it came through the ring)
        if (kRing) {
            const bool dead = *reinterpret_cast<volatile uint32_t*>(misc + kMRingDead) != 0u;
            bool landed = false;
            if (!dead) {
                const uint32_t use = (uint32_t)(lq / kRingStages);
                const volatile uint32_t* seq = misc + kMRingSeq + lq % kRingStages;
                bool started = false;
                for (int i = 0; i < (1 << 24) && !started; ++i) started = *seq > use;
                landed = started && mbar_wait(bars + lq % kRingStages, use & 1u);
            }
            if (!dead && !landed) {   // never expected: remember it, and read the rest of the CTA's tiles the plain way
                if (lane == 0) { misc[kMRingDead] = 1u; atomicAdd(p.spec_ctl + 8, 1u); }
            }
            if (landed && cl >= 0 && ts.s == 0 && ts.e == kTile) {
                const uint4* st4 = reinterpret_cast<const uint4*>(ring + (size_t)(lq % kRingStages) * kTileBytes) + lane;
#pragma unroll
                for (int i = 0; i < 16; ++i) t.v[i] = st4[i * 32];
                vm[0] = vm[1] = 0xffffffffu;
                have = true;
            }
            __syncwarp();
            if (landed && lane == 0 && lq + kRingStages < nloc) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the stage's reads come before the copy that refills it
                ring_issue(lq + kRingStages);
            }
        }
        if (cl >= 0 && *reinterpret_cast<volatile uint32_t*>(misc + kMCursor) > budget) {
            if (lane == 0) atomicOr(&p.state[lt->lid[cl]].spec_bad, 1u);
        } else if (cl >= 0) {
            if (!have) load_tile(p.acc, ts, lane, t, vm);
            if (mark_tile(t, vm, lt->sthr[cl], keep)) {
                // room in the CTA's shared memory, or, when that is full, straight in the layer's region
                const bool single = marks_single(keep[0], keep[1]);   // uniform over the warp
                MarkScan ms;
                if (single) n = count_single(keep[0], keep[1]);
                else { ms = scan_marks(keep[0], keep[1], lane); n = ms.n; }
                if (lane == 0) first = atomicAdd(misc + kMCursor, n);
                first = __shfl_sync(0xffffffffu, first, 0);
                uint2* dst = res;
                uint32_t ytag = pack_y(0u, (uint32_t)cl, 0u);
                const bool to_global = first + n > kReadRes;
                if (lane == 0) off = to_global ? atomicAdd(&p.state[lt->lid[cl]].cursor, n) : atomicAdd(&lt->v0[cl], n);
                off = __shfl_sync(0xffffffffu, off, 0);
                if (to_global) {
                    dst = p.staging + lt->elem_off[cl];
                    ytag = region_y(0u, (uint32_t)(q - lt->tf[cl]));
                    if (lane == 0) p.runge[q] = make_uint2(off, n);
                    first = off;
                }
                auto put = [&](uint32_t pos, uint32_t bits, uint32_t o) { dst[pos] = make_uint2(bits, ytag | o); };
                if (single) write_single(t, keep[0], keep[1], first, lane, put);
                else write_scanned(reinterpret_cast<const uint32_t*>(p.acc + ts.lo), keep[0], keep[1], ms, first,
                                   wbase + 16 * warp, lane, put);
                if (to_global) { first = kTileGlobal; n = 0; }
            }
        }
        if (lane == 0) { rt->first[lq] = first; rt->n[lq] = (uint16_t)n; rt->ge[lq] = off; }
    }
    __syncthreads();
    stamp(p, 1);

    // ---- hand the staged entries to the layers' regions ----
    // room in every layer's region for what this CTA holds of it; then one thread per tile copies
    for (int c = threadIdx.x; c < nl; c += kSelThreads) {
        const uint32_t nc = lt->v0[c];
        lt->v1[c] = nc ? atomicAdd(&p.state[lt->lid[c]].cursor, nc) : 0u;
    }
    __syncthreads();
    for (int lq = threadIdx.x; lq < nloc; lq += kSelThreads) {
        const int q = kStripe * (b + (lq / kStripe) * G) + lq % kStripe;
        const uint32_t n = rt->n[lq], first = rt->first[lq];
        if (q >= p.tiles || first == kTileGlobal) continue;
        if (n == 0) { p.runge[q] = make_uint2(0u, 0u); continue; }
        const int cl = (int)y_layer(res[first].y);
        const uint32_t g = lt->v1[cl] + rt->ge[lq];
        p.runge[q] = make_uint2(g, n);
        uint2* dst = p.staging + lt->elem_off[cl] + g;
        const uint32_t yt = region_y(0u, (uint32_t)(q - lt->tf[cl]));
        for (uint32_t e = 0; e < n; ++e) {
            const uint2 ent = res[first + e];
            dst[e] = make_uint2(ent.x, yt | y_off(ent.y));
        }
    }
    stamp(p, 2);

    // ---- small layers, handed out one at a time (the counter is cleared with the plan upload) ----
    // With streamed layers in the call they wait until the CTA has nothing left to finish: most CTAs
    // have time on their hands then, while the largest layers are still being finished.
    auto small_layers = [&]() {
        uint32_t* next = &p.state[p.desc[0].layer_id].pad[0];
        for (;;) {
            __syncthreads();
            if (threadIdx.x == 0) misc[kMTileCtr] = atomicAdd(next, 1u);
            __syncthreads();
            const int j = (int)misc[kMTileCtr];
            if (j >= p.n_my) break;
            if (is_direct(p, j)) resolve_direct(p, j, smem);   // uniform over the CTA
        }
    };
    if (!has_streamed) {   // uniform over the grid: small layers only
        small_layers();
        return;
    }

    // ---- every layer's entries are in its region: the layers are finished one per CTA, round-robin ----
    if (!p.prestaged) {   // uniform over the grid
        __threadfence();
        grid.sync();
    }
    // largest first (a layer's cost grows with what was staged for it): the order is worked out by
    // every CTA for itself; CTA b starts with the b-th largest, the rest are taken from a counter
    // (cleared with the plan upload) as CTAs become free
    for (int c = threadIdx.x; c < nl; c += kSelThreads)
        lt->v0[c] = lt->sthr[c] == 0xffffffffu ? 0u : __ldcg(&p.state[lt->lid[c]].cursor);
    __syncthreads();
    for (int c = threadIdx.x; c < nl; c += kSelThreads) {
        const uint32_t s = lt->v0[c];
        int before = 0;
        for (int o = 0; o < nl; ++o) {
            const uint32_t so = lt->v0[o];
            before += (so > s || (so == s && o < c)) ? 1 : 0;
        }
        lt->v1[before] = (uint32_t)c;
    }
    __syncthreads();
    {
        uint32_t* next = &p.state[p.desc[0].layer_id].pad[1];
        int slot = b;
        while (slot < nl) {
            const int c = (int)lt->v1[slot];
            bool done = false;
            if (lt->sthr[c] != 0xffffffffu) {
                const uint32_t flooded = __ldcg(&p.state[lt->lid[c]].spec_bad);
                done = finish_layer(p, lt, c, lt->v0[c], flooded, tt, smem);
            }
            if (!done && p.acc_rw) {
                // the layer is on the retry list: its part of the index output must not be mistaken for
                // selected entries by the pass that clears them
                const int64_t o0 = lt->out_off[c];
                for (int64_t i = threadIdx.x; i < (int64_t)lt->k[c]; i += kSelThreads)
                    if (o0 + i < p.out_cap) p.idx[o0 + i] = -1;
            }
            __syncthreads();
            if (threadIdx.x == 0) misc[kMTileCtr] = (uint32_t)G + atomicAdd(next, 1u);
            __syncthreads();
            slot = (int)misc[kMTileCtr];
        }
    }
    stamp(p, 5);
    small_layers();
    stamp(p, 6);

    // ---- what is left over: the five steps on the retry list, by the whole grid ----
    __threadfence();
    grid.sync();
    // The selected entries are cleared in the accumulator by the whole grid (one SM gets through about
    // one scattered 4-byte store per clock: a large layer's would hold its finishing CTA up for
    // microseconds).  Small layers and the retry list clear their own.
    if (p.acc_rw) {
        const int64_t n_out = p.out_total < p.out_cap ? p.out_total : p.out_cap;
        const int64_t step = (int64_t)G * kSelThreads;
        for (int64_t i0 = (int64_t)b * kSelThreads + threadIdx.x; i0 < n_out; i0 += 4 * step) {
            int64_t at[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) at[u] = i0 + u * step < n_out ? __ldcg(p.idx + i0 + u * step) : -1;
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (at[u] >= 0) p.acc_rw[at[u]] = 0.0f;
        }
    }
    stamp(p, 3);
    const unsigned long long packed = __ldcg(&p.retry->packed);
    if ((packed >> 32) == 0ull) return;   // uniform over the grid
    __syncthreads();
    if (threadIdx.x == 0) {   // the parameters in shared memory now describe the retry list
        p.from_retry = 1;
        p.n_my = (int32_t)(packed >> 32);
        p.tiles = (int32_t)(uint32_t)packed;
        p.desc = p.retry_desc;
    }
    __syncthreads();
    retry_steps(p, smem, grid);
}

}  // namespace

deft_status launch_select_stream(const SelParams& p, bool has_streamed, bool ring, cudaStream_t stream) {
    static thread_local int attr_dev = -1;
    int dev = 0;
    DEFT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != attr_dev) {
        DEFT_CUDA_TRY(cudaFuncSetAttribute(k_select_stream<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
        DEFT_CUDA_TRY(cudaFuncSetAttribute(k_select_stream<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
        attr_dev = dev;
    }
    SelParams args = p;
    int hs = has_streamed ? 1 : 0;
    void* kargs[] = {&args, &hs};
    void* fn = ring ? reinterpret_cast<void*>(k_select_stream<true>) : reinterpret_cast<void*>(k_select_stream<false>);
    DEFT_CUDA_TRY(cudaLaunchCooperativeKernel(fn, dim3(p.grid), dim3(kSelThreads), kargs, kSmemBytes, stream));
    return DEFT_OK;
}

}  // namespace deft
