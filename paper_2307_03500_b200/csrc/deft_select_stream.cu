// Layer-wise top-k selection for one worker (Algorithm 5) in ONE pass over the worker's part of the
// vector, without grid-wide barriers: the kernel for calls whose layers were selected from before on
// the same workspace (a training loop).
//
// Every layer comes with a remembered cut: the first-level bucket (key bits 30..19) in which the
// previous call found a key some way below the layer's k-th largest, moved by the change of the
// layer's norm (predict_cut).  One CTA of 512 threads per SM owns a contiguous run of the call's
// tiles.  A warp holds a whole tile in registers, tests it against the cut (one floating-point
// test per 16-byte load, the exact test only where that one passes) and moves the entries at or
// above the cut, in index order, into the CTA's shared memory.  At the end of its run the CTA
// copies what it staged into the layer's region of the staging area (one atomic per CTA and layer
// reserves the room) and publishes (first entry, entries) for each of its tiles.
//
// The CTA that completes a layer's last tile (a ticket per layer) finishes the layer on its own while
// the others are still reading: if at least k entries were staged, the k largest of the layer are
// among them, so a three-level radix select over the staged entries (shared memory) gives the exact
// threshold key T and the number of entries equal to T to take; the per-tile counts, a prefix over
// the layer's tiles and the ordered write (value, int64 index; ascending index, equal keys: lowest
// indices first; optionally clearing the selected entries of the vector) follow from the published
// tile table.  The result never depends on the cut: a layer with fewer than k staged entries, or
// without a usable cut, or too dense to speculate on, is appended to a retry list, and the five-step
// kernel (deft_select.cu), launched right behind this one, selects exactly those layers with its two
// reads (it returns at once when the list is empty).
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
// keys counted from the cut (1/256 octave; the first-level buckets are 1/16, and the staged keys crowd
// into the few buckets right above the cut) gives the bin `a` of the k-th largest key: everything in a
// higher bin is selected, nothing in a lower one.  The few entries of bin a (the candidates) are ranked
// among themselves by (key descending, index ascending); the first k - (entries above bin a) of them
// are selected and get a flag in their entry.  No threshold key is ever needed.
constexpr int kFineShift = 15;
constexpr int kFineBins = kBins1;   // the top bin takes everything beyond
constexpr uint32_t kCandMax = 1024; // candidates that can be ranked; a layer with more goes to the retry list
constexpr uint32_t kBigMax = 1024;  // tiles per pass that can wait for a warp
constexpr uint32_t kSelFlag = 0x80000000u;   // in an entry's .y: a candidate that is selected
static_assert(kBigMax * 16 <= kSmAuxBytes && kCandMax * 12 <= kSmAuxBytes && kShift1 > kFineShift &&
              DEFT_MAX_LAYER_ELEMS / kTile < (1 << 20),
              "candidates and the list of tiles waiting for a warp live in the aux region; bit 31 of .y is free");

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
__device__ __noinline__ void finish_layer(const SelParams& p, LayerTable* lt, int c, uint32_t S, uint32_t flooded,
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
    if (S < k || flooded) {
        // the cut was too high (fewer than k entries reached the staging area) or far too low (a CTA
        // stopped staging): the layer goes to the retry list; a cut that was too high lowers the next ones
        if (tid == 0) {
            atomicAdd(p.spec_ctl + 5, 1u);
            push_retry(p, lt->j[c]);
        }
        return;
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
#pragma unroll 4
        for (uint32_t pos = tid; pos < nres; pos += kSelThreads) f.res[pos] = f.src[pos];
#pragma unroll 4
        for (int t = tid; t < np0; t += kSelThreads) {
            const uint2 fn = __ldcg(tab + t);
            tt->first[t] = fn.x;
            tt->n[t] = (uint16_t)fn.y;
        }
    }
    for (int i = tid; i < kFineBins; i += kSelThreads) h[i] = 0;
    if (tid == 0) { misc[kMBudget] = 0u; misc[kMFlag] = 0u; }   // tiles listed for the warps; candidates collected
    __syncthreads();
    lap.lap(20);
    for (uint32_t pos = tid; pos < S; pos += kSelThreads) atomicAdd(&h[fine_bin(key_of(staged_get(f, pos).x), cut)], 1u);
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
        return;
    }
    if (tid == 0) {
        // what the next call starts from: the first-level bucket of the k_safe-th key if that many were
        // staged, else the bucket below this call's cut
        const double norm = p.desc[lt->j[c]].norm;
        if (S >= k_safe) {
            hint_update(hp, (cut + (a_safe << kFineShift)) >> kShift1, true, k, norm);
        } else {
            const uint32_t cutb = cut >> kShift1;
            hint_update(hp, cutb > 0u ? cutb - 1u : 0u, false, k, norm);
        }
        atomicAdd(p.spec_ctl + 4, 1u);
    }
    // the candidates: (key, index order, where the entry lives); the histogram's room is free now
    uint32_t* ckey = h;
    uint32_t* cy = h + kCandMax;
    uint32_t* cpos = h + 2 * kCandMax;
    for (uint32_t pos = tid; pos < S; pos += kSelThreads) {
        const uint2 ent = staged_get(f, pos);
        if (fine_bin(key_of(ent.x), cut) == a) {
            const uint32_t i = atomicAdd(misc + kMFlag, 1u);
            ckey[i] = key_of(ent.x);
            cy[i] = ent.y;
            cpos[i] = pos;
        }
    }
    __syncthreads();
    for (uint32_t i = tid; i < C; i += kSelThreads) {
        const uint32_t key = ckey[i], y = cy[i];
        uint32_t before = 0;
        for (uint32_t j = 0; j < C; ++j) before += (ckey[j] > key) || (ckey[j] == key && cy[j] < y);
        if (before < krem) {
            const uint32_t pos = cpos[i];
            if (pos < kStreamRes) f.res[pos].y = y | kSelFlag; else f.src[pos].y = y | kSelFlag;
        }
    }
    __syncthreads();
    stamp(p, 10);
    lap.lap(23);
    if (p.timing && tid == 0) { atomicMax(p.timing + 14, (unsigned long long)S); atomicAdd(p.timing + 15, (unsigned long long)S); atomicMax(p.timing + 13, (unsigned long long)C); }
    // per-tile counts, prefix over the layer's tiles, ordered write: up to kMaxLocalTiles tiles per pass,
    // each thread a run of consecutive tiles.  A tile with few entries is written by its thread, the
    // others go on a list that the warps work off afterwards.
    float* const val = p.val;
    int64_t* const idx = p.idx;
    float* const acc_rw = p.acc_rw;
    const int64_t cap = p.out_cap;
    const int64_t tile0 = lt->start[c] / kTile;
    const int64_t out_off = lt->out_off[c];
    uint4* big = reinterpret_cast<uint4*>(smem + kSmAux);   // (tile, selected entries before it, -, -)
    uint32_t base = 0;
    for (int tp = 0; tp < tn; tp += kMaxLocalTiles) {
        const int np = tn - tp < kMaxLocalTiles ? tn - tp : kMaxLocalTiles;
        if (tp > 0) {
#pragma unroll 4
            for (int t = tid; t < np; t += kSelThreads) {
                const uint2 fn = __ldcg(tab + tp + t);
                tt->first[t] = fn.x;
                tt->n[t] = (uint16_t)fn.y;
            }
            if (tid == 0) misc[kMBudget] = 0u;
            __syncthreads();
        }
        const int m = (np + kSelThreads - 1) / kSelThreads;
        const int lo = tid * m < np ? tid * m : np, hi = lo + m < np ? lo + m : np;
        uint32_t mine = 0;
        for (int t = lo; t < hi; ++t) {
            const uint32_t first = tt->first[t], n = tt->n[t];
            uint32_t g = 0;
            for (uint32_t e = 0; e < n; ++e) {
                const uint2 ent = staged_get(f, first + e);
                g += (fine_bin(key_of(ent.x), cut) > a) || (ent.y & kSelFlag);
            }
            tt->ge[t] = g;
            mine += g;
        }
        lap.lap(24);
        uint32_t total;
        uint32_t run = base + block_excl_scan(mine, scratch, total);
        lap.lap(25);
        for (int t = lo; t < hi; ++t) {
            const uint32_t first = tt->first[t], n = tt->n[t];
            if (n != 0) {
                uint32_t slot = kBigMax;
                if (n > kThreadEmit) slot = atomicAdd(misc + kMBudget, 1u);
                if (slot < kBigMax) {
                    big[slot] = make_uint4((uint32_t)t, run, 0u, 0u);
                } else {
                    const int64_t lo_elem = (tile0 + tp + t) * kTile;
                    int64_t pos = out_off + run;
                    for (uint32_t e = 0; e < n; ++e) {
                        const uint2 ent = staged_get(f, first + e);
                        if ((fine_bin(key_of(ent.x), cut) > a) || (ent.y & kSelFlag)) {
                            const int64_t elem = lo_elem + (int64_t)y_off(ent.y);
                            if (pos < cap) {
                                val[pos] = __uint_as_float(ent.x);
                                idx[pos] = elem;
                            }
                            if (acc_rw) acc_rw[elem] = 0.0f;
                            ++pos;
                        }
                    }
                }
            }
            run += tt->ge[t];
        }
        __syncthreads();
        lap.lap(26);
        const uint32_t nbig = misc[kMBudget] < kBigMax ? misc[kMBudget] : kBigMax;
        for (uint32_t i = warp; i < nbig; i += kSelWarps) {   // one warp per listed tile, 32 entries per round
            const uint4 it = big[i];
            const uint32_t first = tt->first[it.x], n = tt->n[it.x];
            const int64_t lo_elem = (tile0 + tp + it.x) * kTile;
            int64_t pos = out_off + it.y;
            for (uint32_t e0 = 0; e0 < n; e0 += 32) {
                const bool valid = e0 + lane < n;
                const uint2 ent = valid ? staged_get(f, first + e0 + lane) : make_uint2(0u, 0u);
                const bool sel = valid && ((fine_bin(key_of(ent.x), cut) > a) || (ent.y & kSelFlag));
                const unsigned ball = __ballot_sync(0xffffffffu, sel);
                if (sel) {
                    const int64_t mypos = pos + __popc(ball & ((1u << lane) - 1u));
                    const int64_t elem = lo_elem + (int64_t)y_off(ent.y);
                    if (mypos < cap) {
                        val[mypos] = __uint_as_float(ent.x);
                        idx[mypos] = elem;
                    }
                    if (acc_rw) acc_rw[elem] = 0.0f;
                }
                pos += __popc(ball);
            }
        }
        base += total;
        __syncthreads();   // the tables are rewritten by the next pass
        lap.lap(27);
    }
    if (p.timing && tid == 0) atomicAdd(p.timing + 28, 1ull);
}

// Out of line: the rare path must not cost the kernel's main loop registers.
__device__ __noinline__ void retry_steps(const SelParams& q, unsigned char* smem, cg::grid_group& grid) {
    five_steps(q, smem, grid);
}

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
    TileTable* tt = reinterpret_cast<TileTable*>(smem + kSmTile);
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kSmMisc);
    uint32_t* wbase = reinterpret_cast<uint32_t*>(smem + kSmWBase);
    uint2* res = reinterpret_cast<uint2*>(smem + kSmMain);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const CtaRange r = cta_range(p, reinterpret_cast<int*>(smem + kSmTf));
    const int nl = build_layer_table(p, r, lt, misc + kMScratch, true);
    if (threadIdx.x == 0) { misc[kMCursor] = 0; misc[kMTileCtr] = 0; misc[kMFlag] = 0; misc[kMBudget] = 4096u; }
    __syncthreads();
    // what the CTA may stage: a multiple of what its tiles should hold if every layer's entries down to
    // the rank behind its cut were spread evenly.  A cut that turns out far too low must not flood the
    // staging area: past the budget the CTA stops reading and its layers go to the retry list.
    for (int c = threadIdx.x; c < nl; c += kSelThreads) {
        lt->v0[c] = 0u;   // entries of the layer this CTA stages
        if (lt->sthr[c] == 0xffffffffu) continue;
        const int64_t size = lt->end[c] - lt->start[c];
        const uint64_t per_tile = ((uint64_t)safe_rank(lt->k[c]) * kTile + size - 1) / size;
        const uint64_t want = (uint64_t)own_tiles(p, r, lt, c) * per_tile * kFloodFactor;
        atomicAdd(&misc[kMBudget], (uint32_t)(want < 0x3fffffffull ? want : 0x3fffffffull));
    }
    // layers without a usable cut: the CTA that owns the layer's first tile hands them on
    for (int c = threadIdx.x; c < nl; c += kSelThreads)
        if (lt->sthr[c] == 0xffffffffu && lt->tf[c] >= r.q0 && lt->tf[c] < r.q1) {
            push_retry(p, lt->j[c]);
            atomicAdd(p.spec_ctl + 6, 1u);
        }
    __syncthreads();
    stamp(p, 8);
    const uint32_t budget = misc[kMBudget] < 0x7fffffffu ? misc[kMBudget] : 0x7fffffffu;

    if (nl > 0) {   // uniform over the CTA; a CTA without streamed layers has nothing to read or hand over
        // ---- the read: every tile of the CTA once ----
        {
            int c = 0;
            for (int lq = grab_tile(misc + kMTileCtr, lane); lq < r.nloc; lq = grab_tile(misc + kMTileCtr, lane)) {
                const int q = r.q0 + lq;
                const int cl = tile_layer(lt, nl, q, c);
                uint32_t first = 0, n = 0;
                if (cl >= 0 && lt->sthr[cl] != 0xffffffffu &&
                    *reinterpret_cast<volatile uint32_t*>(misc + kMCursor) > budget) {
                    if (lane == 0) misc[kMFlag] = 1u;
                } else if (cl >= 0 && lt->sthr[cl] != 0xffffffffu) {
                    const TileSpan ts = tile_span(lt->start[cl], lt->end[cl], lt->tf[cl], q);
                    TileRegs t;
                    uint32_t vm[2], keep[2];
                    load_tile(p.acc, ts, lane, t, vm);
                    const bool any_marked = mark_tile(t, vm, lt->sthr[cl], keep);
                    if (any_marked) {
                        // room in the CTA's shared memory, or, when that is full, straight in the layer's region
                        const bool single = marks_single(keep[0], keep[1]);   // uniform over the warp
                        MarkScan ms;
                        if (single) n = count_single(keep[0], keep[1]);
                        else { ms = scan_marks(keep[0], keep[1], lane); n = ms.n; }
                        if (lane == 0) first = atomicAdd(misc + kMCursor, n);
                        first = __shfl_sync(0xffffffffu, first, 0);
                        uint2* dst = res;
                        uint32_t ytag = pack_y(0u, (uint32_t)cl, (uint32_t)lq);
                        const bool to_global = first + n > kStreamRes;
                        if (to_global) {
                            uint32_t g = 0;
                            if (lane == 0) g = atomicAdd(&p.state[lt->lid[cl]].cursor, n);
                            g = __shfl_sync(0xffffffffu, g, 0);
                            dst = p.staging + lt->elem_off[cl];
                            ytag = region_y(0u, (uint32_t)(q - lt->tf[cl]));
                            if (lane == 0) { p.runge[q] = make_uint2(g, n); atomicAdd(&lt->v0[cl], n); }
                            first = g;
                        }
                        auto put = [&](uint32_t pos, uint32_t bits, uint32_t off) { dst[pos] = make_uint2(bits, ytag | off); };
                        if (single) write_single(t, keep[0], keep[1], first, lane, put);
                        else write_scanned(reinterpret_cast<const uint32_t*>(p.acc + ts.lo), keep[0], keep[1], ms, first,
                                           wbase + 16 * warp, lane, put);
                        if (to_global) { first = kTileGlobal; n = 0; }
                    }
                }
                if (lane == 0) { tt->first[lq] = first; tt->n[lq] = (uint16_t)n; }
            }
        }
        __syncthreads();
        stamp(p, 1);

        // ---- hand the staged entries to the layers' regions ----
        // one warp per local layer: room for the CTA's entries of the layer, then where each tile's entries go
        for (int c = warp; c < nl; c += kSelWarps) {
            if (lt->sthr[c] == 0xffffffffu) continue;
            int a, b;
            local_span(r, lt, c, c, a, b);
            uint32_t nc = 0;
            for (int i = a + lane; i < b; i += 32) nc += tt->n[i];
            nc = __reduce_add_sync(0xffffffffu, nc);
            uint32_t run = 0;
            if (lane == 0) lt->v0[c] += nc;   // with the tiles that went straight to the region: the CTA's entries of the layer
            if (lane == 0 && nc != 0) run = atomicAdd(&p.state[lt->lid[c]].cursor, nc);
            run = __shfl_sync(0xffffffffu, run, 0);
            for (int i0 = a; i0 < b; i0 += 32) {
                const int i = i0 + lane;
                const uint32_t n = i < b ? tt->n[i] : 0u;
                const uint32_t incl = warp_incl_scan(n, lane);
                if (i < b && tt->first[i] != kTileGlobal) {
                    tt->ge[i] = run + incl - n;
                    p.runge[r.q0 + i] = make_uint2(run + incl - n, n);
                }
                run += __shfl_sync(0xffffffffu, incl, 31);
            }
        }
        __syncthreads();
        // one thread per tile copies the tile's entries
        for (int lq = threadIdx.x; lq < r.nloc; lq += kSelThreads) {
            const uint32_t n = tt->n[lq];
            if (n == 0) continue;
            const uint32_t first = tt->first[lq], g = tt->ge[lq];
            const int cl = (int)y_layer(res[first].y);
            uint2* dst = p.staging + lt->elem_off[cl] + g;
            const uint32_t yt = region_y(0u, (uint32_t)(r.q0 + lq - lt->tf[cl]));
            for (uint32_t e = 0; e < n; ++e) {
                const uint2 ent = res[first + e];
                dst[e] = make_uint2(ent.x, yt | y_off(ent.y));
            }
        }
        __threadfence();
        __syncthreads();
        stamp(p, 2);
        // per layer, what the CTAs that are through with it add up to: the CTA that completes the layer's last
        // tiles sees every tile accounted for, and with them the layer's entries, and finishes the layer
        for (int c = threadIdx.x; c < nl; c += kSelThreads) {
            uint32_t last = 0u;
            if (lt->sthr[c] != 0xffffffffu) {
                const unsigned long long mine = ((unsigned long long)own_tiles(p, r, lt, c) << 41) |
                                                ((unsigned long long)(misc[kMFlag] ? 1u : 0u) << 31) | lt->v0[c];
                const unsigned long long now = atomicAdd(&p.state[lt->lid[c]].done, mine) + mine;
                if ((uint32_t)(now >> 41) == (uint32_t)(lt->tfe[c] - lt->tf[c])) {
                    last = 1u | ((uint32_t)((now >> 31) & 0x3ffu) != 0u ? 2u : 0u);
                    lt->v0[c] = (uint32_t)now & 0x7fffffffu;
                }
            }
            lt->v1[c] = last;
        }
        __syncthreads();
        int nfin = 0;
        for (int c = 0; c < nl; ++c) {
            if (!lt->v1[c]) continue;   // uniform over the CTA
            __threadfence();
            __syncthreads();
            finish_layer(p, lt, c, lt->v0[c], lt->v1[c] >> 1, tt, smem);
            __syncthreads();
            ++nfin;
        }
        if (p.timing && threadIdx.x == 0) atomicMax(p.timing + 29, (unsigned long long)nfin);
    }
    stamp(p, 5);

    // ---- small layers, handed out one at a time (the counter is cleared with the plan upload) ----
    {
        uint32_t* next = &p.state[p.desc[0].layer_id].pad[0];
        for (;;) {
            __syncthreads();
            if (threadIdx.x == 0) misc[kMTileCtr] = atomicAdd(next, 1u);
            __syncthreads();
            const int j = (int)misc[kMTileCtr];
            if (j >= p.n_my) break;
            if (is_direct(p, j)) resolve_direct(p, j, smem);   // uniform over the CTA
        }
    }
    stamp(p, 6);
    if (!has_streamed) return;   // uniform over the grid: small layers only, nothing can be left over

    // ---- what is left over: the five steps on the retry list, by the whole grid ----
    __threadfence();
    grid.sync();
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

deft_status launch_select_stream(const SelParams& p, bool has_streamed, cudaStream_t stream) {
    static thread_local int attr_dev = -1;
    int dev = 0;
    DEFT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != attr_dev) {
        DEFT_CUDA_TRY(cudaFuncSetAttribute(k_select_stream, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
        attr_dev = dev;
    }
    SelParams args = p;
    int hs = has_streamed ? 1 : 0;
    void* kargs[] = {&args, &hs};
    DEFT_CUDA_TRY(cudaLaunchCooperativeKernel(reinterpret_cast<void*>(k_select_stream), dim3(p.grid), dim3(kSelThreads),
                                              kargs, kSmemBytes, stream));
    return DEFT_OK;
}

}  // namespace deft
