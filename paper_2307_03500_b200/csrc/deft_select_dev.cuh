// Device-side building blocks shared by the two selection kernels (deft_select.cu: the cooperative
// five-step kernel; deft_select_stream.cu: the single-pass kernel): shared-memory carve-up, per-CTA
// layer and tile tables, the work split, the tile reader that keeps a whole tile in registers, the
// ordered staging of marked entries, the ordered write, and the whole-layer path for small layers.
#pragma once
#include "deft_common.cuh"

namespace deft {
namespace {

// Speculative staging (see the head of this file).  The cut a call leaves for the next one is the
// position of the (k + max(k / 8, kSpecSlack))-th largest key: a margin in rank, so that it
// adapts to the tail of the layer's distribution and to k (the k-th largest of a handful moves
// by several buckets from draw to draw, the k-th of a million hardly at all).
constexpr uint32_t kSpecSlack = 48;
constexpr uint32_t kSpecBudgetFactor = 16;   // staging stops at this multiple of the entries the CTA has to select

// shared-memory carve-up (bytes)
constexpr int kSmMain = 0;   // A: kSlots level-1 histograms, then resident entries | direct: keys
constexpr int kSmMainBytes = 128 * 1024;
constexpr int kSmRes = kSmMain + kSlots * kBins1 * 4;   // resident staged entries (live from step A on)
static_assert(kSlots * kBins1 * 4 + kResident * 8 <= kSmMainBytes && kDirectElems * 4 <= kSmMainBytes &&
              3 * (kMaxWeightedLayers + 1) * 4 <= kSmMainBytes, "main region");
constexpr int kSmAux = kSmMain + kSmMainBytes;   // B: level-2 slots | S2: level-3 slots | direct: its histograms
constexpr int kSmAuxBytes = 20 * 1024;
constexpr int kH2Slots = 4, kH3Slots = 8;        // layers whose level-2 / level-3 histograms are built at once
static_assert(kH2Slots * kBins2 * 4 <= kSmAuxBytes && kH3Slots * kBins3 * 4 <= kSmAuxBytes &&
              kDBins1 * 4 + kDBins2 * 4 <= kSmAuxBytes && kDBins2 >= kDBins3, "aux region");
constexpr int kSmTile = kSmAux + kSmAuxBytes;    // per local tile: first entry, entries, counts
constexpr int kSmTileBytes = kMaxLocalTiles * 10;
constexpr int kSmLayer = kSmTile + kSmTileBytes; // per local streamed layer, see LayerTable
constexpr int kSmLayerBytes = kMaxLocalLayers * 72;   // >= sizeof(LayerTable)
constexpr int kSmPref = kSmLayer + kSmLayerBytes;   // prefixes of one batch of tiles in S4
constexpr int kSmPrefBytes = kSelThreads * 8;
constexpr int kSmMisc = kSmPref + kSmPrefBytes;
constexpr int kSmMiscBytes = 1024 + 512;   // scratch words, then the call's parameters (see params_in_smem)
constexpr int kSmTf = kSmMisc + kSmMiscBytes;       // tile_first of the rank's first layers (start-up search)
constexpr int kTfCache = 1024;
constexpr int kSmTfBytes = (kTfCache + 1) * 4 + 12;
constexpr int kSmSuper = (kSmTf + kSmTfBytes + 15) / 16 * 16;   // interleaved split: prefix at each own super-tile
constexpr int kSmSuperBytes = (kMaxLocalTiles / kSuper) * 8;
constexpr int kSmWBase = kSmSuper + kSmSuperBytes;   // staging pass: 16 words per warp
constexpr int kSmWBaseBytes = kSelWarps * 16 * 4;
constexpr int kSmemBytes = kSmWBase + kSmWBaseBytes;
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");

enum MiscOff : int {   // word offsets inside the misc area
    kMScratch = 0,     // 64: block scan scratch
    kMOut3 = 64,       // 4: result of block_scan_select (bucket, keys above, second bucket, keys in all)
    kMLast = 72,       // kSlots: this CTA flushed the layer's last tiles
    kMCursor = 80,     // 1: staged entries of this CTA
    kMFlag = 96,       // 1: this CTA has to read its tiles again
    kMTried = 97,      // 1: at least one layer of this CTA had a speculative cut
    kMBudget = 98,     // entries the CTA may stage speculatively
    kMTileCtr = 99,    // next local tile to hand to a warp
    kMWarpCnt = 128,   // 32: per-warp packed counts (direct layers)
};
static_assert(kMWarpCnt + 32 <= 1024 / 4 && kSlots <= 8 && sizeof(SelParams) <= 512 && sizeof(SelParams) % 4 == 0, "misc area");

// The call's parameters, copied into shared memory once per CTA.  Routines that are kept out of line
// take them by reference; a reference to the kernel's own parameter would make the compiler keep a
// copy in local memory, and with nearly all of L1 given to shared memory and the vector streaming through
// L2, every access to such a copy is a trip to DRAM.  Ends with a barrier.
__device__ __forceinline__ SelParams& params_in_smem(const SelParams& p, unsigned char* smem) {
    uint32_t* dst = reinterpret_cast<uint32_t*>(smem + kSmMisc + 1024);
    const uint32_t* src = reinterpret_cast<const uint32_t*>(&p);
    if (threadIdx.x < sizeof(SelParams) / 4) dst[threadIdx.x] = src[threadIdx.x];
    __syncthreads();
    return *reinterpret_cast<SelParams*>(dst);
}

// Facts about the CTA's streamed layers (shared memory, struct of arrays).
struct LayerTable {
    int j[kMaxLocalLayers];          // position in the rank's layer list
    int lid[kMaxLocalLayers];        // layer id in the model (state / histogram index)
    int tf[kMaxLocalLayers];         // first tile (rank-local tile id)
    int tfe[kMaxLocalLayers];        // one past the last tile
    int64_t start[kMaxLocalLayers];  // first element
    int64_t end[kMaxLocalLayers];
    int64_t out_off[kMaxLocalLayers];
    int64_t elem_off[kMaxLocalLayers];   // first slot of the layer's staging region
    uint32_t k[kMaxLocalLayers];     // entries to select
    uint32_t sthr[kMaxLocalLayers];  // entries with key >= sthr are staged (0xffffffff: none)
    uint32_t v0[kMaxLocalLayers];    // step value: prefix (b1, b2) | T
    uint32_t v1[kMaxLocalLayers];    // step value: krem1 | krem2 | need
    uint32_t base_gt[kMaxLocalLayers];
    uint32_t base_eq[kMaxLocalLayers];
};
static_assert(sizeof(LayerTable) <= kSmLayerBytes, "layer table");

struct TileTable {                   // per local tile (tile q - q0 of the CTA)
    uint32_t first[kMaxLocalTiles];  // first staged entry
    uint32_t ge[kMaxLocalTiles];     // staged entries above T | equal to T << 16
    uint16_t n[kMaxLocalTiles];      // staged entries
};
static_assert(sizeof(TileTable) <= kSmTileBytes && kTile <= 65535, "tile table");

// staged entry: .x = value bits, .y = offset in tile | local layer << 11 | local tile << 19
__device__ __forceinline__ uint32_t pack_y(uint32_t off, uint32_t c, uint32_t lq) { return off | (c << 11) | (lq << 19); }
__device__ __forceinline__ uint32_t y_off(uint32_t y) { return y & 0x7ffu; }
__device__ __forceinline__ uint32_t y_layer(uint32_t y) { return (y >> 11) & 0xffu; }
__device__ __forceinline__ uint32_t y_tile(uint32_t y) { return y >> 19; }
static_assert(kTile == 2048 && kMaxLocalLayers <= 256 && kMaxLocalTiles <= 8192, "entry packing");

__device__ __forceinline__ uint32_t key_of(uint32_t bits) { return bits & 0x7fffffffu; }

__device__ __forceinline__ void stamp(const SelParams& p, int slot) {
    if (p.timing && threadIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        atomicMax(p.timing + slot, t);
    }
}

// Largest j in [0, n_my-1] with desc[j].tile_first <= q.
__device__ __forceinline__ int layer_of_tile(const LayerDesc* __restrict__ desc, int n_my, int q) {
    int lo = 0, hi = n_my - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (desc[mid].tile_first <= q) lo = mid; else hi = mid - 1;
    }
    return lo;
}

struct TileSpan {
    int64_t lo;   // first element of the address-aligned tile
    int s, e;     // offsets [s, e) inside the tile that belong to the layer
};

__device__ __forceinline__ TileSpan tile_span(int64_t start, int64_t end, int tile_first, int q) {
    const int64_t t = start / kTile + (q - tile_first);
    TileSpan r;
    r.lo = t * kTile;
    const int64_t s = start > r.lo ? start : r.lo;
    const int64_t e = end < r.lo + kTile ? end : r.lo + kTile;
    r.s = (int)(s - r.lo);
    r.e = (int)(e - r.lo);
    return r;
}

__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t x = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += x;
    }
    return v;
}

// Sum over lanes >= mine (lane 31 is the top).
__device__ __forceinline__ uint32_t warp_suffix_sum(uint32_t v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t x = __shfl_down_sync(0xffffffffu, v, o);
        if (lane + o < 32) v += x;
    }
    return v;
}

// Exclusive prefix of v over the CTA in thread order; `total` = sum over the CTA.
// scratch: 33 words of shared memory.
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t* scratch, uint32_t& total) {
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t incl = warp_incl_scan(v, lane);
    __syncthreads();   // scratch may still be in use
    if (lane == 31) scratch[w] = incl;
    __syncthreads();
    if (w == 0) {
        const uint32_t x = lane < kSelWarps ? scratch[lane] : 0u;
        const uint32_t xi = warp_incl_scan(x, lane);
        scratch[lane] = xi - x;
        if (lane == 31) scratch[32] = xi;
    }
    __syncthreads();
    total = scratch[32];
    return scratch[w] + incl - v;
}

// The searches below run once per layer and step; they are kept out of line and free of
// unrolled register arrays so that the kernel's straight-line code stays short (at small
// ranks the kernel is bound by latencies, instruction fetch among them).

// CTA-wide: walks a histogram of `bins` bins (bins / kSelThreads consecutive bins per thread;
// bins a multiple of kSelThreads) from its top bin down and finds the bucket that holds the
// k-th largest key.  out[0] = bucket, out[1] = keys strictly above it; if k2 != k also out[2] =
// the bucket of the k2-th largest key; out[3] = keys in the histogram.  `global`: the histogram is in global memory and was
// written by other CTAs (read past L1).
__device__ __noinline__ void block_scan_select(const uint32_t* h, int bins, bool global, uint32_t k, uint32_t k2,
                                               uint32_t* scratch, uint32_t* out) {
    const int per = bins / kSelThreads;
    const int base = bins - per * ((int)threadIdx.x + 1);   // thread order = descending bins
    uint32_t c[8];   // all loads in flight together (per <= 8)
#pragma unroll
    for (int i = 0; i < 8; ++i) c[i] = i < per ? (global ? __ldcg(h + base + i) : h[base + i]) : 0u;
    uint32_t sum = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) sum += c[i];
    uint32_t total;
    const uint32_t excl = block_excl_scan(sum, scratch, total);   // keys in bins above mine
    if (threadIdx.x == 0) { out[0] = 0; out[1] = 0; out[2] = 0; out[3] = total; }
    __syncthreads();
    if (sum != 0 && excl < k && k <= excl + sum) {                // exactly one thread
        uint32_t run = excl;
        bool found = false;
#pragma unroll
        for (int i = 7; i >= 0; --i) {
            if (!found && i < per) {
                if (run + c[i] >= k) { out[0] = (uint32_t)(base + i); out[1] = run; found = true; }
                else run += c[i];
            }
        }
    }
    if (k2 != k && sum != 0 && excl < k2 && k2 <= excl + sum) {   // the bucket of the k2-th largest key (0 if fewer keys)
        uint32_t run = excl;
        bool found = false;
#pragma unroll
        for (int i = 7; i >= 0; --i) {
            if (!found && i < per) {
                if (run + c[i] >= k2) { out[2] = (uint32_t)(base + i); found = true; }
                else run += c[i];
            }
        }
    }
    __syncthreads();
}

// One warp: the same search on a histogram of 32 * per bins in global memory (per a multiple
// of 4, at most 32).  First the lanes' sums (lane l covers bins [per * l, per * (l + 1)), lane 31
// the top), then the bins of the lane that holds the k-th key, one bin per lane.
// Returns (bucket, keys strictly above it).
__device__ __noinline__ uint2 warp_scan_select(const uint32_t* __restrict__ h, int per, uint32_t k) {
    const int lane = threadIdx.x & 31;
    uint32_t sum = 0;
    const uint4* h4 = reinterpret_cast<const uint4*>(h + per * lane);
    uint4 v[8];      // all loads in flight together (per <= 32)
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = 4 * i < per ? __ldcg(h4 + i) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
    for (int i = 0; i < 8; ++i) sum += v[i].x + v[i].y + v[i].z + v[i].w;
    const uint32_t ab = warp_suffix_sum(sum, lane) - sum;   // keys in lanes above mine
    const unsigned hit = __ballot_sync(0xffffffffu, sum != 0 && ab < k && k <= ab + sum);
    if (hit == 0) return make_uint2(0u, 0u);   // k exceeds the histogram total: cannot happen for a valid plan
    const int owner = __ffs(hit) - 1;
    const uint32_t ab_owner = __shfl_sync(0xffffffffu, ab, owner);
    const uint32_t c = lane < per ? __ldcg(h + per * owner + lane) : 0u;
    const uint32_t a = ab_owner + warp_suffix_sum(c, lane) - c;   // keys above this bin
    const unsigned hit2 = __ballot_sync(0xffffffffu, c != 0 && a < k && k <= a + c);
    const int b = __ffs(hit2) - 1;
    return make_uint2((uint32_t)(per * owner + b), __shfl_sync(0xffffffffu, a, b));
}
static_assert(kBins2 % 128 == 0 && kBins3 % 128 == 0 && kBins2 <= 1024 && kBins3 <= 1024 && kBins1 <= 8 * kSelThreads &&
              kBins1 % kSelThreads == 0 && kDBins1 % kSelThreads == 0 && kDBins2 % kSelThreads == 0 &&
              kDBins3 % kSelThreads == 0, "search shapes");

// ---------------------------------------------------------------------------------
// tile workers: one warp holds a whole tile (kTile = 2048 elements) in registers
// ---------------------------------------------------------------------------------
// 16-byte group g of the tile (0..511) is read by lane g % 32 as load g / 32.  Groups that
// do not touch [s, e) are not read; a group that straddles s or e is read whole (the bytes
// outside the layer are inside the same 16-byte aligned group, hence readable) and masked.
struct TileRegs {
    uint4 v[16];
};
static_assert(kTile == 16 * 32 * 4, "16 vector loads per lane");

// Bit c of the result: offset o + c lies in [s, e).
__device__ __forceinline__ uint32_t valid4(int o, int s, int e) {
    const int lo = s - o > 0 ? s - o : 0, hi = e - o < 4 ? e - o : 4;
    return hi > lo ? ((1u << hi) - 1u) & ~((1u << lo) - 1u) : 0u;
}

// vm: bit (4 * (i % 8) + c) of vm[i / 8] = component c of load i belongs to the layer.
// Components outside the layer come back as +0.  The vector is read past L1 (ld.global.cg): the same
// kernels clear selected entries of it on their way out, which the read-only (.nc) path does not allow.
__device__ __forceinline__ void load_tile(const float* acc, const TileSpan& ts, int lane, TileRegs& t,
                                          uint32_t (&vm)[2]) {
    const uint4* p4 = reinterpret_cast<const uint4*>(acc + ts.lo) + lane;
    if (ts.s == 0 && ts.e == kTile) {
#pragma unroll
        for (int i = 0; i < 16; ++i) t.v[i] = __ldcg(p4 + i * 32);
        vm[0] = vm[1] = 0xffffffffu;
    } else {
        vm[0] = vm[1] = 0u;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const uint32_t m = valid4((i * 32 + lane) * 4, ts.s, ts.e);
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (m) v = __ldcg(p4 + i * 32);
            t.v[i] = make_uint4(m & 1u ? v.x : 0u, m & 2u ? v.y : 0u, m & 4u ? v.z : 0u, m & 8u ? v.w : 0u);
            vm[i >> 3] |= m << (4 * (i & 7));
        }
    }
}

// Where a CTA's staged entry number `pos` lives.
struct Stage {
    uint2* res;      // shared memory, nres entries
    uint2* spill;    // global memory: entry pos >= nres is spill[pos - nres]
    uint32_t nres;
};
__device__ __forceinline__ void stage_put(const Stage& st, uint32_t pos, uint2 v) {
    if (pos < st.nres) st.res[pos] = v; else st.spill[pos - st.nres] = v;
}
__device__ __forceinline__ uint2 stage_get(const Stage& st, uint32_t pos) {
    return pos < st.nres ? st.res[pos] : __ldcg(st.spill + (pos - st.nres));
}

// CTA-wide pass over the CTA's staged entries, in no particular order.  The spilled part is
// read in batches of kSpillBatch loads per thread so that the pass is not bound by one
// HBM round trip per entry.
constexpr int kSpillBatch = 8;
constexpr int kEmitBatch = 4;

template <typename F>
__device__ __forceinline__ void for_each_staged(const Stage& st, uint32_t total, F f) {
    const uint32_t nres = total < st.nres ? total : st.nres;
    for (uint32_t pos = threadIdx.x; pos < nres; pos += kSelThreads) f(st.res[pos]);
    if (total <= st.nres) return;
    const uint32_t nsp = total - st.nres;
    for (uint32_t base = 0; base < nsp; base += kSpillBatch * kSelThreads) {
        uint2 ent[kSpillBatch];
#pragma unroll
        for (int u = 0; u < kSpillBatch; ++u) {
            const uint32_t i = base + u * kSelThreads + threadIdx.x;
            ent[u] = i < nsp ? __ldcg(st.spill + i) : make_uint2(0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < kSpillBatch; ++u)
            if (base + u * kSelThreads + threadIdx.x < nsp) f(ent[u]);
    }
}

// Bit c of the result: component c of v has key >= thr.
__device__ __forceinline__ uint32_t keep4(const uint4& v, uint32_t thr) {
    return (key_of(v.x) >= thr ? 1u : 0u) | (key_of(v.y) >= thr ? 2u : 0u) |
           (key_of(v.z) >= thr ? 4u : 0u) | (key_of(v.w) >= thr ? 8u : 0u);
}

__device__ __forceinline__ uint32_t pick4(uint32_t a, uint32_t b, uint32_t c, uint32_t d, int sel) {
    const uint32_t ab = (sel & 1) ? b : a, cd = (sel & 1) ? d : c;
    return (sel & 2) ? cd : ab;
}

// The larger of |a| and |b| up to its sign (which carries no meaning); a NaN operand wins, as it
// does in the order of the magnitude keys.
__device__ __forceinline__ float amax2(float a, float b) {
    float d;
    asm("max.NaN.xorsign.abs.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}

// keep[]: bit (4 * (i % 8) + c) of keep[i / 8] = component c of load i has key >= thr and lies in the
// layer (thr = 0xffffffff: none).  Two levels: one floating-point test of the largest magnitude of a
// 16-byte load rules out almost every load when the cut is high; only the loads that pass get the
// exact integer test per component.  (For floats that are not NaN the order of magnitudes is the
// order of the keys, denormals included; the test is written so that a NaN passes.)
// Returns false, with keep untouched, if no lane of the warp has a load that passes the first test.
__device__ __forceinline__ bool mark_tile(const TileRegs& t, const uint32_t (&vm)[2], uint32_t thr, uint32_t (&keep)[2]) {
    const float thrf = __uint_as_float(thr < 0x7f800000u ? thr : 0x7f800000u);
    uint32_t pass = 0u;   // bit i: load i may hold an entry
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const float m = amax2(amax2(__uint_as_float(t.v[i].x), __uint_as_float(t.v[i].y)),
                              amax2(__uint_as_float(t.v[i].z), __uint_as_float(t.v[i].w)));
        if (!(fabsf(m) < thrf)) pass |= 1u << i;
    }
    if (!__any_sync(0xffffffffu, pass != 0u)) return false;
    keep[0] = keep[1] = 0u;
#pragma unroll
    for (int i = 0; i < 16; ++i)
        if (pass & (1u << i)) keep[i >> 3] |= keep4(t.v[i], thr) << (4 * (i & 7));
    keep[0] &= vm[0];
    keep[1] &= vm[1];
    return __any_sync(0xffffffffu, (keep[0] | keep[1]) != 0u);
}

// ---- moving a tile's marked entries to their places, in index order (load, lane, component) ----
// Nearly always no 16-byte load of any lane holds more than one marked component.  Then where an entry
// goes follows from one ballot per load (the lanes below mine with a mark in the same load, the marks of
// the loads before), and the entry's value is picked out of the registers that hold the tile.  Otherwise
// (dense tiles, runs of equal values) the per-load counts of a lane are packed 8 bits each, four loads
// per word, scanned over the lanes, and the values are read again from the vector in a compact loop
// (the tile has just been loaded: they come from L2).  All of it is inline and small: the loop around
// a tile has to fit the instruction cache, and a call would spill the registers that hold the tile.
struct MarkScan {
    uint32_t excl[4];   // marked components of lower lanes, per load (8 bits each)
    uint32_t mytot;     // lane i < 16: marked components of load i over the warp
    uint32_t incl;      // inclusive scan of mytot over the lanes
    uint32_t n;         // marked components of the tile
};
__device__ __forceinline__ MarkScan scan_marks(uint32_t k0, uint32_t k1, int lane) {
    MarkScan ms;
    uint32_t tot[4];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        const uint32_t kw = (g < 2 ? k0 : k1) >> (16 * (g & 1));
        const uint32_t packed = __popc(kw & 0xfu) | (__popc(kw & 0xf0u) << 8) | (__popc(kw & 0xf00u) << 16) |
                                (__popc(kw & 0xf000u) << 24);
        const uint32_t incl = warp_incl_scan(packed, lane);
        tot[g] = __shfl_sync(0xffffffffu, incl, 31);
        ms.excl[g] = incl - packed;
    }
    ms.mytot = lane < 16 ? (pick4(tot[0], tot[1], tot[2], tot[3], lane >> 2) >> (8 * (lane & 3))) & 0xffu : 0u;
    ms.incl = warp_incl_scan(ms.mytot, lane);
    ms.n = __shfl_sync(0xffffffffu, ms.incl, 31);
    return ms;
}

// True if no load of any lane holds more than one marked component (k0 / k1: the lane's marks).
__device__ __forceinline__ bool marks_single(uint32_t k0, uint32_t k1) {
    // a nibble with two or more bits set: x & (x - 1) != 0 per nibble, for all eight nibbles of a word at once
    const uint32_t m0 = k0 & (((k0 & 0xeeeeeeeeu) >> 1) | ((k0 & 0xccccccccu) >> 2) | ((k0 & 0x88888888u) >> 3));
    const uint32_t m1 = k1 & (((k1 & 0xeeeeeeeeu) >> 1) | ((k1 & 0xccccccccu) >> 2) | ((k1 & 0x88888888u) >> 3));
    return !__any_sync(0xffffffffu, (m0 | m1) != 0u);
}

// Bit 4 * i of the result: load i of the lane (nibble i of k) has a mark.
__device__ __forceinline__ uint32_t marked_loads(uint32_t k) { return (k | (k >> 1) | (k >> 2) | (k >> 3)) & 0x11111111u; }

// Marked components of the tile when marks_single() holds (one per marked load).
__device__ __forceinline__ uint32_t count_single(uint32_t k0, uint32_t k1) {
    return __reduce_add_sync(0xffffffffu, (uint32_t)(__popc(marked_loads(k0)) + __popc(marked_loads(k1))));
}

// marks_single() holds: put(position, value bits, offset in tile) for every marked component; the tile's
// entries take positions first, first + 1, ... in index order.  Loads in which no lane has a mark (most
// of them, when the cut is high) cost a test of a warp-wide mask and nothing else.
template <typename Put>
__device__ __forceinline__ void write_single(const TileRegs& t, uint32_t k0, uint32_t k1, uint32_t first, int lane,
                                             Put put) {
    const uint32_t below = (1u << lane) - 1u;
    const uint32_t u0 = __reduce_or_sync(0xffffffffu, marked_loads(k0)), u1 = __reduce_or_sync(0xffffffffu, marked_loads(k1));
    uint32_t run = first;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        if (((i < 8 ? u0 : u1) >> (4 * (i & 7))) & 1u) {   // uniform over the warp
            const uint32_t nib = ((i < 8 ? k0 : k1) >> (4 * (i & 7))) & 0xfu;
            const uint32_t bal = __ballot_sync(0xffffffffu, nib != 0u);
            if (nib) {
                const uint32_t c = (uint32_t)__ffs((int)nib) - 1u;
                const uint32_t bits = pick4(t.v[i].x, t.v[i].y, t.v[i].z, t.v[i].w, (int)c);
                put(run + (uint32_t)__popc(bal & below), bits, (uint32_t)((i * 32 + lane) * 4) + c);
            }
            run += (uint32_t)__popc(bal);
        }
    }
}

// The general case: positions from the packed scans, values read again from `tile` (the tile's first
// element in the vector).  wbase: 16 words of shared memory private to the warp.
template <typename Put>
__device__ __forceinline__ void write_scanned(const uint32_t* tile, uint32_t k0, uint32_t k1, const MarkScan& ms,
                                              uint32_t first, uint32_t* wbase, int lane, Put put) {
    if (lane < 16) wbase[lane] = first + ms.incl - ms.mytot;   // where load `lane`'s entries start
    __syncwarp();
    unsigned long long m = (unsigned long long)k0 | ((unsigned long long)k1 << 32);
    const unsigned long long all = m;
    while (m) {
        const int bit = __ffsll((long long)m) - 1;
        m &= m - 1;
        const int i = bit >> 2, c = bit & 3;
        const uint32_t off = (uint32_t)((i * 32 + lane) * 4 + c);
        const uint32_t bits = __ldcg(tile + off);
        const uint32_t before_lanes = (pick4(ms.excl[0], ms.excl[1], ms.excl[2], ms.excl[3], i >> 2) >> (8 * (i & 3))) & 0xffu;
        const uint32_t before_mine = __popc((uint32_t)(all >> (4 * i)) & ((1u << c) - 1u));
        put(wbase[i] + before_lanes + before_mine, bits, off);
    }
    __syncwarp();   // wbase is rewritten by the warp's next tile
}

// Reading pass over one tile.  kHist: count every element in the level-1 histogram h.
// Entries with key >= thr are staged behind the CTA's cursor (thr = 0xffffffff: none); h2 != NULL: with
// b1 = kCountStaged every staged entry is counted in h2 under its first-level bucket (first read with a
// speculative cut), else the staged entries of bucket b1 are counted in the level-2 histogram h2 (second
// read).  Returns (first entry, entries).
constexpr uint32_t kCountStaged = 0xffffffffu;
template <bool kHist, bool kMark = true>
__device__ __forceinline__ uint2 read_tile(const float* acc, const TileSpan& ts, uint32_t* h, uint32_t thr,
                                           const Stage& st, uint32_t ytag, uint32_t* cursor, uint32_t* wbase,
                                           int lane, uint32_t* h2 = nullptr, uint32_t b1 = 0) {
    TileRegs t;
    uint32_t vm[2];
    load_tile(acc, ts, lane, t, vm);
    if (kHist) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            atomicAdd(&h[key_of(t.v[i].x) >> kShift1], 1u);
            atomicAdd(&h[key_of(t.v[i].y) >> kShift1], 1u);
            atomicAdd(&h[key_of(t.v[i].z) >> kShift1], 1u);
            atomicAdd(&h[key_of(t.v[i].w) >> kShift1], 1u);
        }
        // the components outside the layer were loaded as zeros
        if (lane == 0 && ts.e - ts.s != kTile) atomicSub(&h[0], (uint32_t)(kTile - (ts.e - ts.s)));
    }
    if (!kMark) return make_uint2(0u, 0u);   // (a pass that only counts: thr is 0xffffffff)
    uint32_t keep[2];
    if (!mark_tile(t, vm, thr, keep)) return make_uint2(0u, 0u);
    auto put = [&](uint32_t pos, uint32_t bits, uint32_t off) {
        if (h2 != nullptr) {
            if (b1 == kCountStaged) atomicAdd(&h2[key_of(bits) >> kShift1], 1u);
            else if ((key_of(bits) >> kShift1) == b1)   // second read: b1 is known, feed level 2 on the way
                atomicAdd(&h2[(key_of(bits) >> kShift2) & (kBins2 - 1)], 1u);
        }
        stage_put(st, pos, make_uint2(bits, ytag | off));
    };
    uint32_t first = 0, n;
    if (marks_single(keep[0], keep[1])) {   // uniform over the warp
        n = count_single(keep[0], keep[1]);
        if (lane == 0) first = atomicAdd(cursor, n);
        first = __shfl_sync(0xffffffffu, first, 0);
        write_single(t, keep[0], keep[1], first, lane, put);
    } else {
        const MarkScan ms = scan_marks(keep[0], keep[1], lane);
        n = ms.n;
        if (lane == 0) first = atomicAdd(cursor, n);
        first = __shfl_sync(0xffffffffu, first, 0);
        write_scanned(reinterpret_cast<const uint32_t*>(acc + ts.lo), keep[0], keep[1], ms, first, wbase, lane, put);
    }
    return make_uint2(first, n);
}

// ---------------------------------------------------------------------------------
// work split
// ---------------------------------------------------------------------------------
// Two ways to split a rank's tiles over the CTAs.
//   contiguous:  CTA b owns tiles [q0, q1); local tile lq is tile q0 + lq.
//   interleaved: (one large layer only) the tiles are cut into super-tiles of kSuper tiles and
//                CTA b owns super-tiles b, b + G, b + 2G, ...; local tile lq is tile kSuper *
//                (b + (lq / kSuper) * G) + lq % kSuper.  Entries above the threshold cluster
//                wherever the vector is large; this split gives every CTA a sample of the whole
//                vector and hence an equal share of them.
struct CtaRange {
    int q0, q1, jA, jB;
    int nloc;      // local tiles (interleaved: the last super-tile may run past p.tiles)
    int il;        // interleaved
    int nsuper;    // interleaved: super-tiles of the rank
    const int* q0tab;   // cost-weighted split: first tile of every CTA (gridDim.x + 1 entries); else NULL
};

__device__ __forceinline__ int cta_q0(const SelParams& p, int b) { return (int)((int64_t)p.tiles * b / gridDim.x); }

// Tile id of local tile lq, or -1 where an interleaved CTA's last super-tile runs past the end.
__device__ __forceinline__ int local_tile(const SelParams& p, const CtaRange& r, int lq) {
    if (!r.il) return r.q0 + lq;
    const int q = kSuper * ((int)blockIdx.x + (lq / kSuper) * (int)gridDim.x) + lq % kSuper;
    return q < p.tiles ? q : -1;
}

// Largest j in [0, n-1] with tf[j] <= q (tf in shared memory).
__device__ __forceinline__ int layer_of_tile_sh(const int* tf, int n, int q) {
    int lo = 0, hi = n - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (tf[mid] <= q) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// The CTA's tiles and the layers they belong to.  The first kTfCache layers' tile_first are
// fetched with one coalesced request so that the search does not chase cold global loads.
__device__ __forceinline__ CtaRange cta_range(const SelParams& p, int* tf_cache) {
    CtaRange r;
    r.il = p.interleave;
    r.q0tab = nullptr;
    r.nsuper = (p.tiles + kSuper - 1) / kSuper;
    if (r.il) {   // one streamed layer
        const int b = blockIdx.x, G = gridDim.x;
        const int nm = b < r.nsuper ? (r.nsuper - b + G - 1) / G : 0;
        r.nloc = nm * kSuper;
        r.q0 = 0; r.q1 = nm ? p.tiles : 0;
        r.jA = 0; r.jB = nm ? 0 : -1;
        return r;
    }
    const int nc = p.n_my < kTfCache ? p.n_my : kTfCache;
    for (int i = threadIdx.x; i <= nc; i += kSelThreads) tf_cache[i] = p.desc[i].tile_first;
    __syncthreads();
    r.q0 = cta_q0(p, blockIdx.x);
    r.q1 = cta_q0(p, blockIdx.x + 1);
    r.nloc = r.q1 - r.q0;
    r.jA = 0; r.jB = -1;
    if (r.q0 < r.q1) {
        if (p.n_my <= kTfCache || r.q1 <= tf_cache[nc]) {
            r.jA = layer_of_tile_sh(tf_cache, nc, r.q0);
            r.jB = layer_of_tile_sh(tf_cache, nc, r.q1 - 1);
        } else {
            r.jA = layer_of_tile(p.desc, p.n_my, r.q0);
            r.jB = layer_of_tile(p.desc, p.n_my, r.q1 - 1);
        }
    }
    return r;
}

// First tile of CTA b under the split in force.
__device__ __forceinline__ int split_q0(const SelParams& p, const CtaRange& r, int b) {
    return r.q0tab ? r.q0tab[b] : cta_q0(p, b);
}

// The CTA whose run of tiles contains tile q.
__device__ __forceinline__ int split_cta_of_tile(const SelParams& p, const CtaRange& r, int q) {
    if (!r.q0tab) return (int)((((int64_t)q + 1) * gridDim.x + p.tiles - 1) / p.tiles) - 1;
    int lo = 0, hi = (int)gridDim.x - 1;          // largest b with q0tab[b] <= q
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (r.q0tab[mid] <= q) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// The cost-weighted split (see tile_weight): every CTA computes the same table of boundaries
// with integer arithmetic.  `work` = at least 3 * (n_my + 1) words of shared memory, free at
// the time of the call; q0tab = gridDim.x + 1 words that stay.
__device__ __forceinline__ CtaRange weighted_range(const SelParams& p, uint32_t* work, int* q0tab, uint32_t* scratch) {
    const int n = p.n_my;
    uint32_t* Wp = work;                 // n + 1
    uint32_t* w = work + (n + 1);        // n
    int* tf = reinterpret_cast<int*>(work + 2 * (n + 1));   // n + 1
    uint32_t carry = 0;
    for (int j0 = 0; j0 < n; j0 += kSelThreads) {
        const int j = j0 + (int)threadIdx.x;
        uint32_t cost = 0;
        if (j < n) {
            const uint32_t wj = tile_weight(p.desc[j].k, p.desc[j].end - p.desc[j].start);
            const int t0 = p.desc[j].tile_first;
            w[j] = wj;
            tf[j] = t0;
            cost = wj * (uint32_t)(p.desc[j + 1].tile_first - t0);
        }
        uint32_t tot;
        const uint32_t ex = block_excl_scan(cost, scratch, tot);
        if (j < n) Wp[j] = carry + ex;
        carry += tot;
    }
    if (threadIdx.x == 0) { Wp[n] = carry; tf[n] = p.tiles; }
    __syncthreads();
    for (int b = threadIdx.x; b <= (int)gridDim.x; b += kSelThreads)
        q0tab[b] = weighted_boundary(Wp, w, tf, n, p.tiles, b, (int)gridDim.x);
    __syncthreads();
    CtaRange r;
    r.il = 0;
    r.nsuper = 0;
    r.q0tab = q0tab;
    r.q0 = q0tab[blockIdx.x];
    r.q1 = q0tab[blockIdx.x + 1];
    r.nloc = r.q1 - r.q0;
    r.jA = 0; r.jB = -1;
    if (r.q0 < r.q1) {
        r.jA = layer_of_tile_sh(tf, n, r.q0);
        r.jB = layer_of_tile_sh(tf, n, r.q1 - 1);
    }
    __syncthreads();   // `work` is free again
    return r;
}

// Local tiles [a, b) of the CTA that can belong to local layers c0 .. c1 (inclusive).
__device__ __forceinline__ void local_span(const CtaRange& r, const LayerTable* lt, int c0, int c1, int& a, int& b) {
    if (r.il) { a = 0; b = r.nloc; return; }
    a = (r.q0 > lt->tf[c0] ? r.q0 : lt->tf[c0]) - r.q0;
    b = (r.q1 < lt->tfe[c1] ? r.q1 : lt->tfe[c1]) - r.q0;
}

// Tiles of local layer c that this CTA owns.
__device__ __forceinline__ uint32_t own_tiles(const SelParams& p, const CtaRange& r, const LayerTable* lt, int c) {
    if (r.il) {
        const int owns_last = (r.nsuper - 1) % (int)gridDim.x == (int)blockIdx.x;
        return (uint32_t)(r.nloc - (owns_last ? r.nsuper * kSuper - p.tiles : 0));
    }
    const int a = r.q0 > lt->tf[c] ? r.q0 : lt->tf[c], b = r.q1 < lt->tfe[c] ? r.q1 : lt->tfe[c];
    return b > a ? (uint32_t)(b - a) : 0u;
}

__device__ __forceinline__ bool is_direct(const SelParams& p, int j) {
    return !p.fixed_thr && p.desc[j].end - p.desc[j].start <= kDirectElems;
}

// The rank whose key the remembered bucket belongs to: some way below the k-th largest, so that the
// cut holds when the distribution moves a little (the k-th largest of a handful moves by several
// buckets from draw to draw, the k-th of a million hardly at all).
__device__ __forceinline__ uint32_t safe_rank(uint32_t k) { return k + (k / 8 > kSpecSlack ? k / 8 : kSpecSlack); }

// ---- the speculative cut of a layer, from what the previous call on the workspace left behind ----
// Remembered per layer: where the previous call found the key of rank safe_rank(k), as a position on the
// magnitude-key axis in units of 1/16 first-level bucket (= 1/256 octave: key >> 15), that call's norm
// and rank, and how well the predictions have been doing: a running mean of (position found - position
// predicted) and a running mean of that error's absolute deviation, in the same unit (the scheme TCP
// uses for its retransmission timer).
//
// Prediction for this call: the remembered position, moved by the change of the layer's norm (256 units
// per octave) and down by three buckets per doubling of the rank asked for (steeper than the tail of a
// Gaussian or Laplace distribution at these ranks).  The cut is the bucket boundary at or below the
// prediction plus the mean error minus twice the deviation: a stream whose thresholds drift against
// the norms, or jump around, gets lower cuts (more staged entries) instead of failed ones; a steady
// stream gets tight ones.
constexpr int kErrUnit = 16;          // positions and errors in 1/16 bucket
constexpr int kFinePosShift = kShift1 - 4;   // key >> kFinePosShift = position
constexpr int kDevInit = kErrUnit / 2, kDevMin = kErrUnit / 8, kDevMax = 2 * kErrUnit, kBiasMax = 24 * kErrUnit;
static_assert(kErrUnit == 16, "positions are key >> (kShift1 - 4)");

// The predicted position (not clamped), or INT_MIN if nothing usable is remembered.
__device__ __forceinline__ int predict_pos(const uint4& raw, uint32_t k, double norm) {
    const uint32_t pos_p1 = raw.x, rank = raw.z;
    if (pos_p1 == 0 || pos_p1 > (uint32_t)kBins1 * kErrUnit) return INT_MIN;
    int pf = (int)pos_p1 - 1;
    const float was = __uint_as_float(raw.y), now = (float)norm;
    if (was > 0.0f && now > 0.0f && was < 3.0e38f && now < 3.0e38f) pf += (int)floorf(16.0f * kErrUnit * log2f(now / was));
    const uint32_t want = safe_rank(k);
    if (rank > 0 && want > rank) pf -= (int)ceilf(3.0f * kErrUnit * log2f((float)want / (float)rank));
    return pf;
}
__device__ __forceinline__ int hint_bias(uint32_t w) { const int b = (int)(int16_t)(w & 0xffffu); return b < -kBiasMax ? -kBiasMax : (b > kBiasMax ? kBiasMax : b); }
__device__ __forceinline__ int hint_dev(uint32_t w) { const int d = (int)(w >> 16); return d < kDevMin ? kDevInit : (d > kDevMax ? kDevMax : d); }

// Staging threshold for a layer that is to select k of `size` entries and has norm `norm` now, a
// multiple of `align` positions (kErrUnit: a first-level bucket boundary, which the five-step kernel
// needs; the single-pass kernel takes a quarter of that); 0xffffffff = none (nothing remembered, or a
// layer too dense to speculate on).
__device__ __forceinline__ uint32_t predict_cut(const LayerHint* hp, int64_t k, int64_t size, double norm, int align) {
    if (k * kSpecDensity > size) return 0xffffffffu;
    const uint4 raw = __ldcg(reinterpret_cast<const uint4*>(hp));
    const int pf = predict_pos(raw, (uint32_t)k, norm);
    if (pf == INT_MIN) return 0xffffffffu;
    const int at = pf + hint_bias(raw.w) - 2 * hint_dev(raw.w);
    int pa = at >= 0 ? at / align : 0;   // rounded down to the boundary
    const int top = (kBins1 - 1) * kErrUnit / align;
    pa = pa > top ? top : pa;
    return (uint32_t)(pa * align) << kFinePosShift;
}

// Folds one prediction error into a packed (running mean, running mean deviation) word.
__device__ __forceinline__ uint32_t fold_error(uint32_t w, int err, int slack, int dev_max) {
    int bias = hint_bias(w), dev = (int)(w >> 16);
    dev = dev < kDevMin ? kDevInit : (dev > dev_max ? dev_max : dev);
    err = err < -kBiasMax ? -kBiasMax : (err > kBiasMax ? kBiasMax : err);
    const int d = err - bias;
    int ad = (d < 0 ? -d : d) - slack;
    ad = ad < 0 ? 0 : ad;
    bias += d / 4;
    dev += (ad - dev) / 4;
    if (d < -2 * dev - kErrUnit) dev += kErrUnit / 2;   // found well below what the cut allowed for: back off at once
    dev = dev < kDevMin ? kDevMin : (dev > dev_max ? dev_max : dev);
    return ((uint32_t)dev << 16) | ((uint32_t)bias & 0xffffu);
}
constexpr int kDevSameMax = 4 * kErrUnit;

// After a layer's selection: remembers `pos` (where the key of rank safe_rank(k) was found if `exact`, else an
// upper bound of it: just below the cut, when fewer than safe_rank(k) entries were at or above the cut)
// and folds the errors of two predictions into their running means: the one from this call's norm and
// rank (predict_pos), and "where it was last time" (what a pass that runs before the norms and the
// ranks are known has to go by).  `slack`: half the width of the interval the position is known to lie
// in (0 for the single-pass kernel's fine bins, half a bucket for a first-level bucket), which is not
// counted as deviation.  One thread.
__device__ __forceinline__ void hint_update(LayerHint* hp, uint32_t pos, bool exact, int slack, uint32_t k, double norm) {
    const uint4 raw = *reinterpret_cast<const uint4*>(hp);
    const int pf = predict_pos(raw, k, norm);
    const int low = exact ? 0 : kErrUnit / 2;   // the truth lies at or below a bound
    uint32_t w = ((uint32_t)kDevInit << 16), w_same = ((uint32_t)(2 * kDevInit) << 16);
    if (pf != INT_MIN) {
        w = fold_error(raw.w, (int)pos - pf - low, slack, kDevMax);
        w_same = fold_error(hp->err_same, (int)pos - ((int)raw.x - 1) - low, slack, kDevSameMax);
    }
    uint4 out;
    out.x = pos + 1u;
    out.y = __float_as_uint((float)norm);
    out.z = safe_rank(k);
    out.w = w;
    *reinterpret_cast<uint4*>(hp) = out;
    hp->err_same = w_same;
}

// The cut a pass stages by when it runs BEFORE the step's norms and ranks exist (the accumulate pass): the
// place the previous call found, lowered by the running mean and twice the deviation of how that simple
// prediction has been doing for the layer (changes of the norm and of k_l from step to step are in
// there), rounded down to a quarter bucket.  The rank of the previous call stands in for k_l in the density
// test.  0xffffffff = none.
__device__ __forceinline__ uint32_t prestage_cut(const LayerHint* hp, int64_t size) {
    const uint4 raw = __ldcg(reinterpret_cast<const uint4*>(hp));
    if (raw.x == 0u || raw.x > (uint32_t)kBins1 * kErrUnit) return 0xffffffffu;
    if ((int64_t)raw.z * kSpecDensity > size || !stream_can_finish((int64_t)raw.z * 8 / 9, true)) return 0xffffffffu;
    const uint32_t w = __ldcg(&hp->err_same);
    int dev = (int)(w >> 16);
    dev = dev < kDevMin ? 2 * kDevInit : (dev > kDevSameMax ? kDevSameMax : dev);
    const int at = (int)raw.x - 1 + hint_bias(w) - 2 * dev - kErrUnit / 8;
    constexpr int align = kErrUnit / 4;
    int pa = at >= 0 ? at / align : 0;
    const int top = (kBins1 - 1) * kErrUnit / align;
    pa = pa > top ? top : pa;
    return (uint32_t)(pa * align) << kFinePosShift;
}

// Fills the table of the CTA's streamed layers; returns how many there are (at most
// kMaxLocalLayers: checked on the host).
// spec_on: layers get a speculative cut (a multiple of cut_align positions) from what the previous call left behind.
__device__ __forceinline__ int build_layer_table(const SelParams& p, const CtaRange& r, LayerTable* lt,
                                                 uint32_t* scratch, bool spec_on, int cut_align, bool one_cta_finishes = false) {
    int nl = 0;
    // scratch[kMTried - kMScratch] is the CTA's "speculated" flag (same misc area)
    if (threadIdx.x == 0) scratch[kMTried - kMScratch] = 0u;
    __syncthreads();
    for (int j0 = r.jA; j0 <= r.jB; j0 += kSelThreads) {
        const int j = j0 + (int)threadIdx.x;
        const bool streamed = j <= r.jB && !is_direct(p, j);
        uint32_t tot;
        const int c = nl + (int)block_excl_scan(streamed ? 1u : 0u, scratch, tot);
        if (streamed && c < kMaxLocalLayers) {
            lt->j[c] = j;
            lt->lid[c] = p.desc[j].layer_id;
            lt->tf[c] = p.desc[j].tile_first;
            lt->tfe[c] = p.desc[j + 1].tile_first;
            lt->start[c] = p.desc[j].start;
            lt->end[c] = p.desc[j].end;
            lt->out_off[c] = p.desc[j].out_off;
            lt->elem_off[c] = p.desc[j].elem_off;
            lt->k[c] = (uint32_t)p.desc[j].k;
            // speculative cut from what the previous call left behind for this layer
            uint32_t sthr = 0xffffffffu;
            if (p.fixed_thr) {
                sthr = p.thr_key + 1u;                       // key >= thr_key + 1  <=>  key > thr_key
            } else if (spec_on && one_cta_finishes && !stream_can_finish(p.desc[j].k, p.prestaged != 0)) {
                sthr = 0xffffffffu;                          // too many entries for the caller's way of finishing a layer
            } else if (spec_on && p.prestaged) {
                sthr = p.stage_tab[p.desc[j].layer_id].cut;   // what the accumulate pass staged by
                if (sthr != 0xffffffffu) scratch[kMTried - kMScratch] = 1u;
            } else if (spec_on) {
                sthr = predict_cut(p.hint + p.desc[j].layer_id, p.desc[j].k, p.desc[j].end - p.desc[j].start,
                                   p.desc[j].norm, cut_align);
                if (sthr != 0xffffffffu) scratch[kMTried - kMScratch] = 1u;
            }
            lt->sthr[c] = sthr;
        }
        nl += (int)tot;
    }
    __syncthreads();
    return nl < kMaxLocalLayers ? nl : kMaxLocalLayers;
}

// Per-warp walk over tiles in ascending order: tile q belongs to local layer c (or to a direct
// layer lying between two streamed ones: result < 0).  `c` is a cursor that only moves forward.
__device__ __forceinline__ int tile_layer(const LayerTable* lt, int nl, int q, int& c) {
    while (c < nl - 1 && q >= lt->tfe[c]) ++c;
    return (q >= lt->tf[c] && q < lt->tfe[c]) ? c : -1;
}

// The warps of a CTA take its tiles one at a time from a counter in shared memory (in ascending
// order per warp): a fixed round-robin leaves the warps with the costlier tiles behind at the
// barrier that ends the loop.
__device__ __forceinline__ int grab_tile(uint32_t* counter, int lane) {
    int lq = 0;
    if (lane == 0) lq = (int)atomicAdd(counter, 1u);
    return __shfl_sync(0xffffffffu, lq, 0);
}


// ---- the ordered write, by staged entry ----
// A CTA's staged entries lie tile by tile (a tile's entries consecutive and in index order; the tiles in the
// order the warps got to them).  Every warp walks a contiguous range of them, 32 consecutive entries per
// step: an entry's place in the output is (entries of its layer above / equal to T in earlier tiles: pg / pe
// of its tile) + (such entries before it in its own tile), and the second term follows from ballots over the
// run of lanes that hold the same tile, plus what the warp carries over when a tile's entries began in an
// earlier step.  Cost follows the entries a CTA holds, not its tiles.
struct EmitOut { float* val; int64_t* idx; float* acc_rw; int64_t cap; };

// Ordered write of one batch of 32 consecutive entries of ONE layer (one per lane; the small-layer path).
// gt_before / eq_before: entries above / equal to the threshold that precede the batch in the layer.
__device__ __forceinline__ void emit_batch(const EmitOut& p, int64_t out_off, int64_t elem0, bool valid,
                                           uint32_t bits, int64_t off, uint32_t T, uint32_t need,
                                           uint32_t& gt_before, uint32_t& eq_before, int lane) {
    const uint32_t lt_mask = (1u << lane) - 1u;
    const uint32_t key = key_of(bits);
    const bool gt = valid && key > T, eq = valid && key == T;
    const unsigned gt_b = __ballot_sync(0xffffffffu, gt), eq_b = __ballot_sync(0xffffffffu, eq);
    const uint32_t my_gt = gt_before + __popc(gt_b & lt_mask), my_eq = eq_before + __popc(eq_b & lt_mask);
    if (gt || (eq && my_eq < need)) {
        // selected entries before me: every larger key, and the first `need` equal ones
        const int64_t pos = out_off + my_gt + (my_eq < need ? my_eq : need);
        if (pos < p.cap) {
            p.val[pos] = __uint_as_float(bits);
            p.idx[pos] = elem0 + off;
        }
        if (p.acc_rw) p.acc_rw[elem0 + off] = 0.0f;
    }
    gt_before += __popc(gt_b);
    eq_before += __popc(eq_b);
}

__device__ __forceinline__ void emit_entries(const SelParams& p, const CtaRange& r, const LayerTable* lt, const TileTable* tt,
                                             const Stage& st, const uint32_t* pg, const uint32_t* pe, uint32_t total) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t lt_mask = (1u << lane) - 1u;
    const uint32_t per = ((total + kSelWarps - 1) / kSelWarps + 31u) & ~31u;
    const uint32_t w_lo = (uint32_t)warp * per < total ? (uint32_t)warp * per : total;
    const uint32_t w_hi = w_lo + per < total ? w_lo + per : total;
    if (w_lo >= w_hi) return;
    // what the warp carries: the tile of the last entry seen and that tile's entries above / equal to T so far
    uint32_t carry_tile = 0xffffffffu, cg = 0, ce = 0;
    {
        const uint2 e0 = stage_get(st, w_lo);
        const uint32_t ti = y_tile(e0.y), c = y_layer(e0.y);
        const uint32_t first = tt->first[ti], T = lt->v0[c];
        carry_tile = ti;
        for (uint32_t pos = first + lane; pos < w_lo; pos += 32) {   // the part of the tile that lies in the range before
            const uint32_t key = key_of(stage_get(st, pos).x);
            cg += key > T ? 1u : 0u;
            ce += key == T ? 1u : 0u;
        }
        cg = __reduce_add_sync(0xffffffffu, cg);
        ce = __reduce_add_sync(0xffffffffu, ce);
    }
    for (uint32_t p4 = w_lo; p4 < w_hi; p4 += 32 * kEmitBatch) {   // kEmitBatch steps' entries are fetched together
        uint2 ent[kEmitBatch];
#pragma unroll
        for (int u = 0; u < kEmitBatch; ++u) {
            const uint32_t pos = p4 + u * 32 + lane;
            ent[u] = pos < w_hi ? stage_get(st, pos) : make_uint2(0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < kEmitBatch; ++u) {
            if (p4 + u * 32 >= w_hi) break;   // uniform over the warp
            const bool valid = p4 + u * 32 + lane < w_hi;
            const uint32_t y = ent[u].y, bits = ent[u].x;
            const uint32_t ti = valid ? y_tile(y) : 0xffffffffu, c = y_layer(y);
            const uint32_t T = valid ? lt->v0[c] : 0u, need = valid ? lt->v1[c] : 0u;
            const uint32_t key = key_of(bits);
            const bool gt = valid && key > T, eq = valid && key == T;
            const unsigned gtb = __ballot_sync(0xffffffffu, gt), eqb = __ballot_sync(0xffffffffu, eq);
            const uint32_t tprev = __shfl_up_sync(0xffffffffu, ti, 1);
            const unsigned sb = __ballot_sync(0xffffffffu, lane == 0 || ti != tprev);   // lanes at which a tile's run begins
            const int s0 = 31 - __clz((int)(sb & (lt_mask | (1u << lane))));              // where my tile's run begins
            const uint32_t run_before = lt_mask & ~((1u << s0) - 1u);
            const bool carried = s0 == 0 && ti == carry_tile;
            const uint32_t my_gt = (valid ? pg[ti] : 0u) + __popc(gtb & run_before) + (carried ? cg : 0u);
            const uint32_t my_eq = (valid ? pe[ti] : 0u) + __popc(eqb & run_before) + (carried ? ce : 0u);
            if (gt || (eq && my_eq < need)) {
                // selected entries of the layer before me: every larger key, and the first `need` equal ones
                const int q = local_tile(p, r, (int)ti);
                const int64_t elem = (lt->start[c] / kTile + (q - lt->tf[c])) * kTile + (int64_t)y_off(y);
                const int64_t pos = lt->out_off[c] + my_gt + (my_eq < need ? my_eq : need);
                if (pos < p.out_cap) {
                    p.val[pos] = __uint_as_float(bits);
                    p.idx[pos] = elem;
                }
                if (p.acc_rw) p.acc_rw[elem] = 0.0f;
            }
            // carry: the run that reaches the step's last lane
            const uint32_t t_last = __shfl_sync(0xffffffffu, ti, 31);
            const int s_last = 31 - __clz((int)sb);
            const uint32_t run_last = ~((1u << s_last) - 1u);
            const uint32_t g_last = __popc(gtb & run_last), e_last = __popc(eqb & run_last);
            if (s_last == 0 && t_last == carry_tile) { cg += g_last; ce += e_last; }
            else { carry_tile = t_last; cg = g_last; ce = e_last; }
        }
    }
}

// ---------------------------------------------------------------------------------
// direct layers: one CTA loads the layer whole and finishes it from shared memory
// (digits: bits 30..19, 18..9, 8..0)
// ---------------------------------------------------------------------------------
__device__ __forceinline__ void resolve_direct(const SelParams& p, int j, unsigned char* smem) {
    uint32_t* skey = reinterpret_cast<uint32_t*>(smem + kSmMain);
    uint32_t* h1 = reinterpret_cast<uint32_t*>(smem + kSmAux);
    uint32_t* h = h1 + kDBins1;
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kSmMisc);
    uint32_t* scratch = misc + kMScratch;
    uint32_t* out3 = misc + kMOut3;
    uint32_t* wcnt = misc + kMWarpCnt;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t start = p.desc[j].start;
    const uint32_t n = (uint32_t)(p.desc[j].end - start);
    const uint32_t k = (uint32_t)p.desc[j].k;
    const int64_t out_off = p.desc[j].out_off;
    const uint32_t* x = reinterpret_cast<const uint32_t*>(p.acc + start);
    for (int i = tid; i < kDBins1; i += kSelThreads) h1[i] = 0;
    for (int i = tid; i < kDBins2; i += kSelThreads) h[i] = 0;
    __syncthreads();
    // level 1 over the whole layer
    for (uint32_t fb = 0; fb < n; fb += 8 * kSelThreads) {
        uint32_t v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const uint32_t f = fb + u * kSelThreads + tid;
            v[u] = f < n ? __ldcg(x + f) : 0u;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const uint32_t f = fb + u * kSelThreads + tid;
            if (f < n) {
                skey[f] = v[u];
                atomicAdd(&h1[key_of(v[u]) >> kDShift1], 1u);
            }
        }
    }
    __syncthreads();
    block_scan_select(h1, kDBins1, false, k, k, scratch, out3);
    const uint32_t b1 = out3[0], above1 = out3[1];
    __syncthreads();
    // level 2 inside bucket b1
    for (uint32_t f = tid; f < n; f += kSelThreads) {
        const uint32_t key = key_of(skey[f]);
        if ((key >> kDShift1) == b1) atomicAdd(&h[(key >> kDShift2) & (kDBins2 - 1)], 1u);
    }
    __syncthreads();
    block_scan_select(h, kDBins2, false, k - above1, k - above1, scratch, out3);
    const uint32_t b2 = out3[0];
    const uint32_t krem2 = k - above1 - out3[1];
    __syncthreads();
    for (int i = tid; i < kDBins3; i += kSelThreads) h[i] = 0;
    __syncthreads();
    // level 3 inside (b1, b2)
    const uint32_t prefix = (b1 << (kDShift1 - kDShift2)) | b2;
    for (uint32_t f = tid; f < n; f += kSelThreads) {
        const uint32_t key = key_of(skey[f]);
        if ((key >> kDShift2) == prefix) atomicAdd(&h[key & (kDBins3 - 1)], 1u);
    }
    __syncthreads();
    block_scan_select(h, kDBins3, false, krem2, krem2, scratch, out3);
    const uint32_t T = (prefix << kDShift2) | out3[0];
    const uint32_t need = krem2 - out3[1];
    __syncthreads();
    // every warp counts its contiguous share, then the ordered, coalesced write
    const uint32_t wper = ((n + kSelWarps - 1) / kSelWarps + 31) & ~31u;   // multiple of 32
    const uint32_t f0 = (uint32_t)warp * wper < n ? (uint32_t)warp * wper : n;
    const uint32_t f1 = f0 + wper < n ? f0 + wper : n;
    uint32_t n_gt = 0, n_eq = 0;
    for (uint32_t f = f0 + lane; f < f1; f += 32) {
        const uint32_t key = key_of(skey[f]);
        n_gt += key > T;
        n_eq += key == T;
    }
    n_gt = __reduce_add_sync(0xffffffffu, n_gt);
    n_eq = __reduce_add_sync(0xffffffffu, n_eq);
    if (lane == 0) wcnt[warp] = n_gt | (n_eq << 16);   // both totals <= kDirectElems < 65536
    __syncthreads();
    const uint32_t mine = lane < kSelWarps ? wcnt[lane] : 0u;
    const uint32_t before = __shfl_sync(0xffffffffu, warp_incl_scan(mine, lane) - mine, warp);
    uint32_t gt_before = before & 0xffff, eq_before = before >> 16;
    for (uint32_t fb = f0; fb < f1; fb += 32) {
        const uint32_t f = fb + lane;
        const bool valid = f < f1;
        emit_batch(EmitOut{p.val, p.idx, p.acc_rw, p.out_cap}, out_off, start, valid, valid ? skey[f] : 0u, (int64_t)f, T, need,
                   gt_before, eq_before, lane);
    }
    __syncthreads();   // shared memory is reused by the next layer
}
static_assert(kDirectElems < 65536, "packed per-warp counts");

// The CTA's part of the staging area in HBM.
__device__ __forceinline__ uint2* spill_base(const SelParams& p, const CtaRange& r) {
    if (r.il) {
        // one slot per element of the super-tiles of the CTAs before it
        const int64_t before = (int64_t)blockIdx.x * (r.nsuper / (int)gridDim.x) +
                               min((int)blockIdx.x, r.nsuper % (int)gridDim.x);
        return p.staging + p.desc[0].elem_off + before * (kSuper * kTile);
    }
    if (r.q0 < r.q1) {
        // it starts where the CTA's first tile's elements would go
        const TileSpan ts = tile_span(p.desc[r.jA].start, p.desc[r.jA].end, p.desc[r.jA].tile_first, r.q0);
        return p.staging + p.desc[r.jA].elem_off + (ts.lo + ts.s - p.desc[r.jA].start);
    }
    return p.staging;
}

}  // namespace
}  // namespace deft
