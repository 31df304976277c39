// The five steps of the cooperative selection kernel (see deft_select.cu) as device code: used by
// that kernel and, for the layers it leaves over, by the single-pass kernel (deft_select_stream.cu).
#pragma once
#include <cooperative_groups.h>

#include "deft_select_dev.cuh"

namespace deft {
namespace {

// ---------------------------------------------------------------------------------
// step A: level-1 histograms (kSlots layers at a time) and speculative staging
// ---------------------------------------------------------------------------------
// Marker in LayerState::b1: the layer's speculative cut failed (fewer than k entries at or above it, or a
// CTA stopped staging); the layer's histogram is built from all its elements in a second round of step A.
constexpr uint32_t kB1Failed = 0xffffffffu;

// A layer WITH a speculative cut is not histogrammed element by element: only the entries at or above
// the cut are counted (while they are staged).  The cut is a bucket boundary, so these counts are the
// complete histogram from the cut's bucket upwards, and if they add up to k or more the bucket of the k-th
// largest key and the keys above it follow from them as from the full histogram.  If they do not, the cut
// has failed: the layer's counts are cleared, the layer is marked, and round 1 of this step (run by the
// whole grid only if some layer failed) builds its full histogram.
// round 0: every local layer; round 1: only the layers marked kB1Failed, full histogram, nothing staged.
__device__ __noinline__ void step_read1(const SelParams& p, const CtaRange r, LayerTable* lt, int nl,
                                        TileTable* tt, const Stage st, unsigned char* smem, int round) {
    uint32_t* hist = reinterpret_cast<uint32_t*>(smem + kSmMain);
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kSmMisc);
    uint32_t* wbase = reinterpret_cast<uint32_t*>(smem + kSmWBase);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (round == 0) {
        if (threadIdx.x == 0) { misc[kMCursor] = 0; misc[kMFlag] = 0; misc[kMBudget] = 4096u; }
        __syncthreads();
        // staging budget: a few times what the CTA's tiles are expected to stage (k_l / size_l of its layers)
        for (int c = threadIdx.x; c < nl; c += kSelThreads) {
            const int64_t size = lt->end[c] - lt->start[c];
            const uint64_t per_tile = ((uint64_t)lt->k[c] * kTile + size - 1) / size;   // selected entries per tile, rounded up
            const uint64_t want = (uint64_t)own_tiles(p, r, lt, c) * per_tile * kSpecBudgetFactor;
            atomicAdd(&misc[kMBudget], (uint32_t)(want < 0x3fffffffull ? want : 0x3fffffffull));
            lt->base_gt[c] = 0u;   // round 1 works on this layer
            lt->base_eq[c] = 0u;   // this CTA stopped staging for the layer
        }
    } else {
        for (int c = threadIdx.x; c < nl; c += kSelThreads)
            lt->base_gt[c] = __ldcg(&p.state[lt->lid[c]].b1) == kB1Failed ? 1u : 0u;
    }
    __syncthreads();
    const uint32_t budget = misc[kMBudget] < 0x7fffffffu ? misc[kMBudget] : 0x7fffffffu;
    for (int c0 = 0; c0 < nl; c0 += kSlots) {
        const int ns = nl - c0 < kSlots ? nl - c0 : kSlots;
        if (round == 1) {   // uniform over the CTA: nothing to do for this group of layers
            uint32_t any = 0;
            for (int s = 0; s < ns; ++s) any |= lt->base_gt[c0 + s];
            if (!any) continue;
        }
        for (int i = threadIdx.x; i < ns * kBins1; i += kSelThreads) hist[i] = 0;
        int la, lb;
        local_span(r, lt, c0, c0 + ns - 1, la, lb);
        if (threadIdx.x == 0) misc[kMTileCtr] = (uint32_t)la;
        __syncthreads();
        stamp(p, 8);
        int c = c0;
        for (int lq = grab_tile(misc + kMTileCtr, lane); lq < lb; lq = grab_tile(misc + kMTileCtr, lane)) {
            const int q = local_tile(p, r, lq);
            if (q < 0) continue;
            const int cl = tile_layer(lt, c0 + ns, q, c);
            if (cl < 0) continue;
            uint32_t* h = hist + (cl - c0) * kBins1;
            const uint32_t thr = lt->sthr[cl];
            // round 1 reads only the layers whose cut failed, and those in full; round 0 reads a layer without
            // a cut in full (one place in the code for both: the routine is large)
            if (round == 1 && !lt->base_gt[cl]) continue;
            uint2 fn = make_uint2(0u, 0u);
            if (round == 1 || thr == 0xffffffffu) {   // the full histogram, nothing staged
                const TileSpan ts = tile_span(lt->start[cl], lt->end[cl], lt->tf[cl], q);
                read_tile<true, false>(p.acc, ts, h, 0xffffffffu, st, 0u, misc + kMCursor, wbase + 16 * warp, lane);
                if (round == 1) continue;
            } else if (*reinterpret_cast<volatile uint32_t*>(misc + kMCursor) > budget) {
                // a cut that turns out far too low must not flood the staging area: past the budget the CTA
                // stops staging; the layers it skips tiles of count as failed
                if (lane == 0) {
                    misc[kMFlag] = 1u;
                    lt->base_eq[cl] = 1u;
                    if (p.timing) p.timing[16 + 480 + blockIdx.x] = (1ull << 63) | ((unsigned long long)budget << 32) | (unsigned long long)cl;
                }
            } else {
                const TileSpan ts = tile_span(lt->start[cl], lt->end[cl], lt->tf[cl], q);
                fn = read_tile<false>(p.acc, ts, nullptr, thr, st, pack_y(0u, (uint32_t)cl, (uint32_t)lq), misc + kMCursor,
                                      wbase + 16 * warp, lane, h, kCountStaged);
            }
            if (lane == 0) { tt->first[lq] = fn.x; tt->n[lq] = (uint16_t)fn.y; }
        }
        __syncthreads();
        stamp(p, 9);
        for (int i = threadIdx.x; i < ns * kBins1; i += kSelThreads) {
            const uint32_t cnt = hist[i];
            if (cnt && (round == 0 || lt->base_gt[c0 + i / kBins1]))
                atomicAdd(p.hist1 + (size_t)lt->lid[c0 + i / kBins1] * kBins1 + (i % kBins1), cnt);
        }
        __syncthreads();
        stamp(p, 10);
        // ticket per layer: the CTA that flushes a layer's last tiles sees the complete histogram (round 1
        // counts on from where round 0 ended: twice the layer's tiles)
        if ((int)threadIdx.x < ns) {
            const int cl = c0 + threadIdx.x;
            uint32_t last = 0u;
            if (round == 0 || lt->base_gt[cl]) {
                const uint32_t mine = own_tiles(p, r, lt, cl);
                if (round == 0 && lt->base_eq[cl]) atomicOr(&p.state[lt->lid[cl]].spec_bad, 1u);
                __threadfence();
                const uint32_t old = atomicAdd(&p.state[lt->lid[cl]].ticket1, mine);
                last = (old + mine == (uint32_t)(round + 1) * (uint32_t)(lt->tfe[cl] - lt->tf[cl])) ? 1u : 0u;
            }
            misc[kMLast + threadIdx.x] = last;
        }
        __syncthreads();
        stamp(p, 11);
        for (int s = 0; s < ns; ++s) {
            if (!misc[kMLast + s]) continue;   // uniform over the CTA
            const int cl = c0 + s;
            const int lid = lt->lid[cl];
            __threadfence();
            // besides b1: the bucket of a key some way further down, from which the next call takes its cut
            const uint32_t kk = lt->k[cl], k_safe = safe_rank(kk);
            uint32_t* gh = p.hist1 + (size_t)lid * kBins1;
            block_scan_select(gh, kBins1, true, kk, k_safe, misc + kMScratch, misc + kMOut3);
            const bool spec = round == 0 && lt->sthr[cl] != 0xffffffffu;
            const uint32_t total = misc[kMOut3 + 3];
            const bool failed = spec && (total < kk || __ldcg(&p.state[lid].spec_bad) != 0u);
            if (failed)   // round 1 starts from a clean histogram
                for (int i = threadIdx.x; i < kBins1; i += kSelThreads) gh[i] = 0u;
            if (threadIdx.x == 0) {
                if (round == 0 && !p.from_retry) atomicAdd(p.spec_ctl + (failed ? 5 : (spec ? 4 : 6)), 1u);   // diagnostics
                if (failed) {
                    p.state[lid].b1 = kB1Failed;   // round 1 finds the bucket (and updates what is remembered)
                    atomicAdd(p.spec_ctl + 3, 1u);
                } else {
                    p.state[lid].b1 = misc[kMOut3];
                    p.state[lid].above1 = misc[kMOut3 + 1];
                    // the next call's speculative cut starts from the bucket of the k_safe-th key if the
                    // histogram reaches that far down, else from the bucket below this call's cut
                    const double norm = p.desc[lt->j[cl]].norm;
                    if (!spec || total >= k_safe) {
                        // (known to the bucket: its middle, half a bucket of slack)
                        hint_update(p.hint + lid, misc[kMOut3 + 2] * kErrUnit + kErrUnit / 2, true, kErrUnit / 2, kk, norm);
                    } else {
                        const uint32_t cutp = (lt->sthr[cl] >> kShift1) * kErrUnit;
                        hint_update(p.hint + lid, cutp > 0u ? cutp - 1u : 0u, false, 0, kk, norm);
                    }
                }
            }
            __syncthreads();
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------
// step B: second read where the speculative cut was too high, then level-2 histograms
// ---------------------------------------------------------------------------------
__device__ __noinline__ void step_read2(const SelParams& p, const CtaRange r, LayerTable* lt, int nl,
                                        TileTable* tt, const Stage st, unsigned char* smem) {
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kSmMisc);
    uint32_t* wbase = reinterpret_cast<uint32_t*>(smem + kSmWBase);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0 && p.fixed_thr) misc[kMFlag] = 1u;   // else: set in step A if the CTA ran over its budget
    __syncthreads();
    if (!p.fixed_thr) {
        for (int c = threadIdx.x; c < nl; c += kSelThreads) {
            const LayerState* ls = p.state + lt->lid[c];
            const uint32_t b1 = __ldcg(&ls->b1);
            lt->v0[c] = b1;
            lt->v1[c] = lt->k[c] - __ldcg(&ls->above1);          // krem1
            const uint32_t need_thr = b1 << kShift1;             // key >= need_thr  <=>  bucket >= b1
            if (lt->sthr[c] > need_thr || lt->base_gt[c]) {      // staged too little (or nothing) for this layer, or its cut failed
                if (p.timing && lt->sthr[c] != 0xffffffffu)
                    p.timing[16 + 480 + blockIdx.x] = ((unsigned long long)lt->lid[c] << 40) | ((unsigned long long)lt->k[c] << 24) |
                                                      ((unsigned long long)(lt->sthr[c] >> kShift1) << 12) | b1;
                lt->sthr[c] = need_thr;
                misc[kMFlag] = 1u;
            }
        }
        __syncthreads();
    }
    uint32_t* h2 = reinterpret_cast<uint32_t*>(smem + kSmAux);
    if (misc[kMFlag]) {   // uniform over the CTA: drop what was staged, read the CTA's tiles with the true cuts
        __syncthreads();
        if (threadIdx.x == 0) {
            misc[kMCursor] = 0;
            if (!p.fixed_thr && misc[kMTried]) atomicAdd(p.spec_ctl + 1, 1u);   // a speculative cut failed
        }
        __syncthreads();
        // kH2Slots layers at a time: their level-2 histograms are built in the same pass
        for (int c0 = 0; c0 < nl; c0 += kH2Slots) {
            const int ns = nl - c0 < kH2Slots ? nl - c0 : kH2Slots;
            for (int i = threadIdx.x; i < ns * kBins2; i += kSelThreads) h2[i] = 0;
            int la, lb;
            local_span(r, lt, c0, c0 + ns - 1, la, lb);
            if (threadIdx.x == 0) misc[kMTileCtr] = (uint32_t)la;
            __syncthreads();
            int c = c0;
            for (int lq = grab_tile(misc + kMTileCtr, lane); lq < lb; lq = grab_tile(misc + kMTileCtr, lane)) {
                const int q = local_tile(p, r, lq);
                if (q < 0) continue;
                const int cl = tile_layer(lt, c0 + ns, q, c);
                if (cl < 0) continue;
                const TileSpan ts = tile_span(lt->start[cl], lt->end[cl], lt->tf[cl], q);
                const uint2 fn = read_tile<false>(p.acc, ts, nullptr, lt->sthr[cl], st,
                                                  pack_y(0u, (uint32_t)cl, (uint32_t)lq), misc + kMCursor,
                                                  wbase + 16 * warp, lane,
                                                  p.fixed_thr ? nullptr : h2 + (cl - c0) * kBins2, lt->v0[cl]);
                if (lane == 0) { tt->first[lq] = fn.x; tt->n[lq] = (uint16_t)fn.y; }
            }
            __syncthreads();
            if (!p.fixed_thr) {
                for (int i = threadIdx.x; i < ns * kBins2; i += kSelThreads) {
                    const uint32_t cnt = h2[i];
                    if (cnt) atomicAdd(p.hist2 + (size_t)lt->lid[c0 + i / kBins2] * kBins2 + (i % kBins2), cnt);
                }
                __syncthreads();
            }
        }
        return;
    }
    if (p.fixed_thr) return;
    // level-2 histograms of the staged entries of bucket b1: kH2Slots layers at a time in shared memory
    const uint32_t total = misc[kMCursor];
    for (int c0 = 0; c0 < nl; c0 += kH2Slots) {
        const int ns = nl - c0 < kH2Slots ? nl - c0 : kH2Slots;
        for (int i = threadIdx.x; i < ns * kBins2; i += kSelThreads) h2[i] = 0;
        __syncthreads();
        for_each_staged(st, total, [&](const uint2 ent) {
            const int c = (int)y_layer(ent.y);
            const uint32_t key = key_of(ent.x);
            if (c >= c0 && c < c0 + ns && (key >> kShift1) == lt->v0[c])
                atomicAdd(&h2[(c - c0) * kBins2 + ((key >> kShift2) & (kBins2 - 1))], 1u);
        });
        __syncthreads();
        for (int i = threadIdx.x; i < ns * kBins2; i += kSelThreads) {
            const uint32_t cnt = h2[i];
            if (cnt) atomicAdd(p.hist2 + (size_t)lt->lid[c0 + i / kBins2] * kBins2 + (i % kBins2), cnt);
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------
// step S2: bucket b2 of every local layer, then the level-3 histograms of the staged entries
// ---------------------------------------------------------------------------------
__device__ __forceinline__ void step_hist3(const SelParams& p, LayerTable* lt, int nl, const Stage& st,
                                           unsigned char* smem) {
    const uint32_t* misc = reinterpret_cast<const uint32_t*>(smem + kSmMisc);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t total = misc[kMCursor];
    if (p.timing && threadIdx.x == 0) { atomicMax(p.timing + 14, (unsigned long long)total); atomicAdd(p.timing + 15, (unsigned long long)total); }
    for (int c = warp; c < nl; c += kSelWarps) {   // one warp per layer
        const int lid = lt->lid[c];
        const uint2 s2 = warp_scan_select(p.hist2 + (size_t)lid * kBins2, kBins2 / 32, lt->v1[c]);
        __syncwarp();
        if (lane == 0) {
            lt->v0[c] = (lt->v0[c] << (kShift1 - kShift2)) | s2.x;   // key >> kShift2 of the candidates
            lt->v1[c] = lt->v1[c] - s2.y;                            // krem2
        }
    }
    __syncthreads();
    // level-3 histograms of the staged entries of bucket (b1, b2): kH3Slots layers at a time
    uint32_t* h3 = reinterpret_cast<uint32_t*>(smem + kSmAux);
    for (int c0 = 0; c0 < nl; c0 += kH3Slots) {
        const int ns = nl - c0 < kH3Slots ? nl - c0 : kH3Slots;
        for (int i = threadIdx.x; i < ns * kBins3; i += kSelThreads) h3[i] = 0;
        __syncthreads();
        for_each_staged(st, total, [&](const uint2 ent) {
            const int c = (int)y_layer(ent.y);
            const uint32_t key = key_of(ent.x);
            if (c >= c0 && c < c0 + ns && (key >> kShift2) == lt->v0[c])
                atomicAdd(&h3[(c - c0) * kBins3 + (key & (kBins3 - 1))], 1u);
        });
        __syncthreads();
        for (int i = threadIdx.x; i < ns * kBins3; i += kSelThreads) {
            const uint32_t cnt = h3[i];
            if (cnt) atomicAdd(p.hist3 + (size_t)lt->lid[c0 + i / kBins3] * kBins3 + (i % kBins3), cnt);
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------
// step S3: threshold T of every local layer, counts per tile, totals per (CTA, layer)
// ---------------------------------------------------------------------------------
__device__ __forceinline__ void step_count(const SelParams& p, const CtaRange& r, LayerTable* lt, int nl,
                                           TileTable* tt, const Stage& st, unsigned char* smem) {
    const uint32_t* misc = reinterpret_cast<const uint32_t*>(smem + kSmMisc);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t total = misc[kMCursor];
    if (p.fixed_thr) {
        // the threshold is given: every staged entry is selected, a tile's count is what it staged
        if (threadIdx.x == 0 && nl > 0) { lt->v0[0] = p.thr_key; lt->v1[0] = 0u; }
        for (int i = threadIdx.x; i < r.nloc; i += kSelThreads) tt->ge[i] = local_tile(p, r, i) >= 0 ? tt->n[i] : 0u;
        if (threadIdx.x == 0 && total) atomicAdd(p.count_out, (unsigned long long)total);
        __syncthreads();
    }
    for (int c = warp; c < nl && !p.fixed_thr; c += kSelWarps) {   // one warp per layer
        const uint2 s3 = warp_scan_select(p.hist3 + (size_t)lt->lid[c] * kBins3, kBins3 / 32, lt->v1[c]);
        const uint32_t b3 = s3.x, above3 = s3.y;
        __syncwarp();
        if (lane == 0) {
            lt->v0[c] = (lt->v0[c] << kShift2) | b3;   // T
            lt->v1[c] = lt->v1[c] - above3;            // need
        }
    }
    if (!p.fixed_thr) {
        for (int i = threadIdx.x; i < r.nloc; i += kSelThreads) tt->ge[i] = 0;
        __syncthreads();
        for_each_staged(st, total, [&](const uint2 ent) {
            const uint32_t key = key_of(ent.x), T = lt->v0[y_layer(ent.y)];
            if (key > T) atomicAdd(&tt->ge[y_tile(ent.y)], 1u);
            else if (key == T) atomicAdd(&tt->ge[y_tile(ent.y)], 1u << 16);
        });
        __syncthreads();
    }
    if (r.il) {   // totals per own super-tile, published under the super-tile's id
        for (int m = threadIdx.x; m < r.nloc / kSuper; m += kSelThreads) {
            uint32_t gt = 0, eq = 0;
#pragma unroll
            for (int i = 0; i < kSuper; ++i) { const uint32_t v = tt->ge[m * kSuper + i]; gt += v & 0xffffu; eq += v >> 16; }
            p.runge[blockIdx.x + m * gridDim.x] = make_uint2(gt, eq);
        }
        return;
    }
    for (int c = warp; c < nl; c += kSelWarps) {   // one warp per layer: totals of its tiles here
        int a, b;
        local_span(r, lt, c, c, a, b);
        uint32_t gt = 0, eq = 0;
        for (int i = a + lane; i < b; i += 32) { const uint32_t v = tt->ge[i]; gt += v & 0xffffu; eq += v >> 16; }
        gt = __reduce_add_sync(0xffffffffu, gt);
        eq = __reduce_add_sync(0xffffffffu, eq);
        if (lane == 0) p.runge[blockIdx.x + lt->j[c]] = make_uint2(gt, eq);
    }
}


// ---------------------------------------------------------------------------------
// step S4: totals of the tiles before this CTA's, scan of the own tiles, ordered write
// ---------------------------------------------------------------------------------

__device__ __noinline__ void step_emit(const SelParams& p, const CtaRange r, LayerTable* lt, int nl,
                                       const TileTable* tt, const Stage st, unsigned char* smem) {
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kSmMisc);
    uint32_t* scratch = misc + kMScratch;
    // per local tile: entries above / equal to T that precede the tile in its layer (the histograms' room is free)
    uint32_t* pg = reinterpret_cast<uint32_t*>(smem + kSmMain);
    uint32_t* pe = pg + kMaxLocalTiles;
    static_assert(2 * kMaxLocalTiles * 4 <= kSlots * kBins1 * 4, "tile prefixes fit the histogram slots");
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (nl == 0) return;
    if (r.il) {
        // Prefix at each own super-tile b + mG: the totals of all super-tiles are summed in
        // windows [b + (m-1)G, b + mG) (window 0 = [0, b)), one warp per window, then scanned.
        uint2* sbase = reinterpret_cast<uint2*>(smem + kSmSuper);
        const int nm = r.nloc / kSuper, G = gridDim.x, b = blockIdx.x;
        for (int m = warp; m < nm; m += kSelWarps) {
            const int hi = b + m * G, lo = m ? hi - G : 0;
            uint32_t gt = 0, eq = 0;
            for (int s = lo + lane; s < hi; s += 32) { const uint2 v = __ldcg(p.runge + s); gt += v.x; eq += v.y; }
            gt = __reduce_add_sync(0xffffffffu, gt);
            eq = __reduce_add_sync(0xffffffffu, eq);
            if (lane == 0) sbase[m] = make_uint2(gt, eq);
        }
        __syncthreads();
        {
            const uint2 w = (int)threadIdx.x < nm ? sbase[threadIdx.x] : make_uint2(0u, 0u);
            uint32_t tg, te;
            const uint32_t e_gt = block_excl_scan(w.x, scratch, tg);
            const uint32_t e_eq = block_excl_scan(w.y, scratch, te);
            if ((int)threadIdx.x < nm) sbase[threadIdx.x] = make_uint2(e_gt + w.x, e_eq + w.y);
        }
        __syncthreads();
        for (int t0 = 0; t0 < r.nloc; t0 += kSelThreads) {
            const int i = t0 + (int)threadIdx.x;
            const uint32_t v = i < r.nloc ? tt->ge[i] : 0u;   // counts <= kTile each: 16 of them fit 16 bits
            uint32_t incl = v;
#pragma unroll
            for (int o = 1; o < kSuper; o <<= 1) {
                const uint32_t x = __shfl_up_sync(0xffffffffu, incl, o, kSuper);
                if ((lane & (kSuper - 1)) >= o) incl += x;
            }
            const uint32_t ex = incl - v;
            if (i < r.nloc) {
                const uint2 sb = sbase[i / kSuper];
                pg[i] = sb.x + (ex & 0xffffu);
                pe[i] = sb.y + (ex >> 16);
            }
        }
    } else {
        for (int c = warp; c < nl; c += kSelWarps) {   // one warp per layer: totals of earlier CTAs
            const int j = lt->j[c];
            uint32_t gt = 0, eq = 0;
            for (int b = split_cta_of_tile(p, r, lt->tf[c]) + lane; b < (int)blockIdx.x; b += 32) {
                if (split_q0(p, r, b) < split_q0(p, r, b + 1)) {
                    const uint2 v = __ldcg(p.runge + b + j);
                    gt += v.x;
                    eq += v.y;
                }
            }
            gt = __reduce_add_sync(0xffffffffu, gt);
            eq = __reduce_add_sync(0xffffffffu, eq);
            if (lane == 0) { lt->base_gt[c] = gt; lt->base_eq[c] = eq; }
        }
        __syncthreads();
        for (int c = 0; c < nl; ++c) {
            int ta, tb;
            local_span(r, lt, c, c, ta, tb);
            uint32_t base_gt = lt->base_gt[c], base_eq = lt->base_eq[c];
            for (int t0 = ta; t0 < tb; t0 += kSelThreads) {   // batches of kSelThreads tiles
                const int i = t0 + (int)threadIdx.x;
                const uint32_t v = i < tb ? tt->ge[i] : 0u;
                uint32_t tot_gt, tot_eq;
                const uint32_t e_gt = block_excl_scan(v & 0xffffu, scratch, tot_gt);
                const uint32_t e_eq = block_excl_scan(v >> 16, scratch, tot_eq);
                if (i < tb) {
                    pg[i] = base_gt + e_gt;
                    pe[i] = base_eq + e_eq;
                }
                base_gt += tot_gt;
                base_eq += tot_eq;
            }
        }
    }
    __syncthreads();
    emit_entries(p, r, lt, tt, st, pg, pe, misc[kMCursor]);
}


// ---------------------------------------------------------------------------------
// the five steps for one call.  p: the call's parameters in shared memory (params_in_smem).  p.from_retry: the layer list is what the single-pass kernel left over
// (no speculation, no small layers; the list's counter is cleared once every CTA has read it).
// ---------------------------------------------------------------------------------
__device__ __forceinline__ void five_steps(const SelParams& p, unsigned char* smem, cooperative_groups::grid_group& grid) {
    LayerTable* lt = reinterpret_cast<LayerTable*>(smem + kSmLayer);
    TileTable* tt = reinterpret_cast<TileTable*>(smem + kSmTile);
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kSmMisc);
    CtaRange r = cta_range(p, reinterpret_cast<int*>(smem + kSmTf));
    if (p.weighted)   // contiguous runs of equal estimated cost instead of equal length
        r = weighted_range(p, reinterpret_cast<uint32_t*>(smem + kSmMain), reinterpret_cast<int*>(smem + kSmTf),
                           misc + kMScratch);
    const int nl = build_layer_table(p, r, lt, misc + kMScratch,
                                     !p.fixed_thr && !p.from_retry, kErrUnit);
    Stage st;
    st.res = reinterpret_cast<uint2*>(smem + kSmRes);
    st.spill = spill_base(p, r);
    st.nres = kResident;

    if (!p.fixed_thr) {   // uniform over the grid
        unsigned long long ta0 = 0;
        if (p.timing && threadIdx.x == 0) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ta0));
        step_read1(p, r, lt, nl, tt, st, smem, 0);
        if (p.timing && threadIdx.x == 0) {
            unsigned long long ta1;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ta1));
            p.timing[16 + 800 + blockIdx.x] = ta1 - ta0;
        }
        stamp(p, 1);
        grid.sync();
        if (p.from_retry && blockIdx.x == 0 && threadIdx.x == 0) p.retry->packed = 0ull;   // every CTA has read the list's size
        if (__ldcg(p.spec_ctl + 3) != 0u) {   // uniform over the grid: some speculative cut failed
            step_read1(p, r, lt, nl, tt, st, smem, 1);
            stamp(p, 7);
            grid.sync();
        }
    }
    unsigned long long tb0 = 0;
    if (p.timing && threadIdx.x == 0) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(tb0));
    step_read2(p, r, lt, nl, tt, st, smem);
    if (p.timing && threadIdx.x == 0) {
        unsigned long long tb1;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(tb1));
        p.timing[16 + blockIdx.x] = tb1 - tb0;
        p.timing[16 + 160 + blockIdx.x] = misc[kMCursor];
        p.timing[16 + 320 + blockIdx.x] = (unsigned long long)nl | ((unsigned long long)r.nloc << 16) |
                                          ((unsigned long long)misc[kMFlag] << 32);
    }
    stamp(p, 2);
    if (!p.fixed_thr) {
        grid.sync();
        step_hist3(p, lt, nl, st, smem);
        stamp(p, 3);
    }
    grid.sync();
    step_count(p, r, lt, nl, tt, st, smem);
    stamp(p, 4);
    grid.sync();
    unsigned long long te0 = 0;
    if (p.timing && threadIdx.x == 0) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(te0));
    step_emit(p, r, lt, nl, tt, st, smem);
    __syncthreads();
    if (p.timing && threadIdx.x == 0) {
        unsigned long long te1;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(te1));
        p.timing[16 + 640 + blockIdx.x] = te1 - te0;
    }
    stamp(p, 5);
    __syncthreads();
    if (p.from_retry) return;   // small layers and the speculation counters are the single-pass kernel's business
    if (p.n_my > 2 * (int)gridDim.x) {
        // many layers: the small ones are handed out one at a time (a counter among the per-layer words
        // that the plan upload clears), so that the CTAs that come out of the ordered write first take
        // them and the ones with the most entries do not also finish last here
        uint32_t* next = &p.state[p.desc[0].layer_id].pad[0];
        for (;;) {
            __syncthreads();
            if (threadIdx.x == 0) misc[kMTileCtr] = atomicAdd(next, 1u);
            __syncthreads();
            const int j = (int)misc[kMTileCtr];
            if (j >= p.n_my) break;
            if (is_direct(p, j)) resolve_direct(p, j, smem);   // uniform over the CTA
        }
    } else {
        for (int j = blockIdx.x; j < p.n_my; j += gridDim.x)
            if (is_direct(p, j)) resolve_direct(p, j, smem);   // uniform over the CTA
    }
    stamp(p, 6);
    if (!p.fixed_thr && threadIdx.x == 0) {
        // the last CTA to finish clears the call's counters (kept across calls for diagnostics: [7] = calls
        // in which some cut failed)
        __threadfence();
        if (atomicAdd(p.spec_ctl + 2, 1u) == gridDim.x - 1) {
            if (__ldcg(p.spec_ctl + 3) != 0u) p.spec_ctl[7] += 1u;
            p.spec_ctl[0] = 0u;
            p.spec_ctl[1] = 0u;
            p.spec_ctl[2] = 0u;
            p.spec_ctl[3] = 0u;
        }
    }
}

}  // namespace
}  // namespace deft
