// Layer-wise top-k selection for one worker (Algorithm 5) as ONE persistent cooperative
// kernel: a segmented radix select over magnitude bit patterns followed by an ordered
// compaction.  One CTA of 512 threads per SM; five steps separated by grid barriers.  Every
// CTA owns the same tiles of the call in every step and keeps what it stages for them (in
// shared memory; overflow spills to HBM), so after the reading steps all work is local to the
// CTA that staged the data.
//
//   A   read 1: per-layer histogram of key bits 30..19 in shared memory, flushed with integer
//       atomics; the CTA that flushes a layer's last tiles finds the bucket b1 holding the
//       k-th largest key.  In the same pass every entry at or above a SPECULATIVE cut — the
//       bucket in which the previous call found the layer's (k + max(k/2, 48))-th largest key,
//       moved by the change of the layer's norm — is moved, in index order, behind the CTA's
//       staging cursor.
//   B   a CTA whose cuts were all at or below the true b1 already holds everything it needs
//       and reads nothing; any other CTA drops what it staged and reads its tiles a second
//       time with the true cut.  Then the staged entries of bucket b1 feed the level-2
//       histogram (bits 18..9).
//   S2  every CTA finds bucket b2 of its layers from the level-2 histograms, then adds the
//       level-3 histogram (bits 8..0) of its staged entries of bucket (b1, b2)
//   S3  every CTA fixes the exact threshold key T and the number of entries equal to T to
//       take, counts its staged entries above / equal to T per tile, publishes its totals
//   S4  every CTA adds up the totals of the tiles before its own, scans its own tiles, and
//       writes (value, int64 index) in ascending index (equal keys: lowest indices first);
//       optionally zeroes the selected entries of the vector (residual update)
// Layers of at most kDirectElems elements take no part in this: at the end one CTA loads
// each of them whole and finishes it from shared memory.
//
// The speculative cut only decides whether step B has to read: the staged set is always a
// superset of what the true cut keeps, so the result does not depend on it.  In a training
// loop the cut of a layer moves little from step to step and the vector is read once.
//
// Determinism: histograms use integer atomics (order-free); the staging order inside a CTA
// depends on warp timing but every output position is a function of counts and of the tile
// an entry came from, so the result is bit-identical from run to run.
#include <cooperative_groups.h>

#include "deft_common.cuh"

namespace cg = cooperative_groups;

namespace deft {
namespace {

// Speculative staging (see the head of this file).  The cut a call leaves for the next one is the
// first-level bucket of the (k + max(k / 2, kSpecSlack))-th largest key: a margin in rank, so that it
// adapts to the tail of the layer's distribution and to k (the k-th largest of a handful moves
// by several buckets from draw to draw, the k-th of a million hardly at all).
constexpr uint32_t kSpecSlack = 48;
constexpr uint32_t kSpecBudgetFactor = 6;   // staging stops at this multiple of the entries the CTA has to select
constexpr int kSpecDensity = 8;             // no speculation for layers that select more than 1 / kSpecDensity of their entries
constexpr uint32_t kSpecCooldown = 1;       // calls without speculation after a call in which a speculative cut failed

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
constexpr int kSmLayerBytes = kMaxLocalLayers * 64;   // >= sizeof(LayerTable)
constexpr int kSmPref = kSmLayer + kSmLayerBytes;   // prefixes of one batch of tiles in S4
constexpr int kSmPrefBytes = kSelThreads * 8;
constexpr int kSmMisc = kSmPref + kSmPrefBytes;
constexpr int kSmMiscBytes = 1024;
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
    kMOut3 = 64,       // 4: result of block_scan_select
    kMLast = 72,       // kSlots: this CTA flushed the layer's last tiles
    kMCursor = 80,     // 1: staged entries of this CTA
    kMFlag = 96,       // 1: this CTA has to read its tiles again
    kMTried = 97,      // 1: at least one layer of this CTA had a speculative cut
    kMBudget = 98,     // entries the CTA may stage speculatively
    kMTileCtr = 99,    // next local tile to hand to a warp
    kMWarpCnt = 128,   // 32: per-warp packed counts (direct layers)
};
static_assert(kMWarpCnt + 32 <= kSmMiscBytes / 4 && kSlots <= 8, "misc area");

// Facts about the CTA's streamed layers (shared memory, struct of arrays).
struct LayerTable {
    int j[kMaxLocalLayers];          // position in the rank's layer list
    int lid[kMaxLocalLayers];        // layer id in the model (state / histogram index)
    int tf[kMaxLocalLayers];         // first tile (rank-local tile id)
    int tfe[kMaxLocalLayers];        // one past the last tile
    int64_t start[kMaxLocalLayers];  // first element
    int64_t end[kMaxLocalLayers];
    int64_t out_off[kMaxLocalLayers];
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
// the bucket of the k2-th largest key.  `global`: the histogram is in global memory and was
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
    if (threadIdx.x == 0) { out[0] = 0; out[1] = 0; out[2] = 0; }
    uint32_t total;
    const uint32_t excl = block_excl_scan(sum, scratch, total);   // keys in bins above mine
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
// Components outside the layer come back as +0.
__device__ __forceinline__ void load_tile(const float* __restrict__ acc, const TileSpan& ts, int lane,
                                          TileRegs& t, uint32_t (&vm)[2]) {
    const uint4* p4 = reinterpret_cast<const uint4*>(acc + ts.lo) + lane;
    if (ts.s == 0 && ts.e == kTile) {
#pragma unroll
        for (int i = 0; i < 16; ++i) t.v[i] = __ldg(p4 + i * 32);
        vm[0] = vm[1] = 0xffffffffu;
    } else {
        vm[0] = vm[1] = 0u;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const uint32_t m = valid4((i * 32 + lane) * 4, ts.s, ts.e);
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (m) v = __ldg(p4 + i * 32);
            t.v[i] = make_uint4(m & 1u ? v.x : 0u, m & 2u ? v.y : 0u, m & 4u ? v.z : 0u, m & 8u ? v.w : 0u);
            vm[i >> 3] |= m << (4 * (i & 7));
        }
    }
}

// Where a CTA's staged entry number `pos` lives.
struct Stage {
    uint2* res;      // shared memory, kResident entries
    uint2* spill;    // HBM, this CTA's part of the staging area
};
__device__ __forceinline__ void stage_put(const Stage& st, uint32_t pos, uint2 v) {
    if (pos < (uint32_t)kResident) st.res[pos] = v; else st.spill[pos - kResident] = v;
}
__device__ __forceinline__ uint2 stage_get(const Stage& st, uint32_t pos) {
    return pos < (uint32_t)kResident ? st.res[pos] : __ldcg(st.spill + (pos - kResident));
}

// CTA-wide pass over the CTA's staged entries, in no particular order.  The spilled part is
// read in batches of kSpillBatch loads per thread so that the pass is not bound by one
// HBM round trip per entry.
constexpr int kSpillBatch = 8;
constexpr int kEmitBatch = 4;
constexpr uint32_t kThreadEmit = 12;   // tiles with at most this many staged entries are written by one thread

template <typename F>
__device__ __forceinline__ void for_each_staged(const Stage& st, uint32_t total, F f) {
    const uint32_t nres = total < (uint32_t)kResident ? total : (uint32_t)kResident;
    for (uint32_t pos = threadIdx.x; pos < nres; pos += kSelThreads) f(st.res[pos]);
    if (total <= (uint32_t)kResident) return;
    const uint32_t nsp = total - kResident;
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

// The rare part of a reading pass, kept out of line and small (the hot loop around it must
// stay resident in the instruction cache): moves the tile's marked entries behind the CTA's
// cursor in index order (load, lane, component = ascending offset).  k0 / k1: bit (4 * (i % 8)
// + c) of word i / 8 marks component c of this lane's load i.  The values are read again from
// the vector (the tile has just been loaded: they come from L1 / L2).  wbase: 16 words of
// shared memory private to the warp.  Returns (first entry, entries).
__device__ __forceinline__ uint2 stage_marked_body(const uint32_t* __restrict__ tile, uint32_t k0, uint32_t k1,
                                                   uint2* res, uint2* spill, uint32_t ytag, uint32_t* cursor,
                                                   uint32_t* wbase, uint32_t* h2, uint32_t b1) {
    const int lane = threadIdx.x & 31;
    // per-load counts of this lane, 8 bits each, four loads per word; scanned over the lanes
    uint32_t excl[4], tot[4];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        const uint32_t kw = (g < 2 ? k0 : k1) >> (16 * (g & 1));
        const uint32_t packed = __popc(kw & 0xfu) | (__popc(kw & 0xf0u) << 8) | (__popc(kw & 0xf00u) << 16) |
                                (__popc(kw & 0xf000u) << 24);
        const uint32_t incl = warp_incl_scan(packed, lane);
        tot[g] = __shfl_sync(0xffffffffu, incl, 31);
        excl[g] = incl - packed;
    }
    // lane i < 16 owns load i: where the load's entries start
    const uint32_t mytot = lane < 16 ? (pick4(tot[0], tot[1], tot[2], tot[3], lane >> 2) >> (8 * (lane & 3))) & 0xffu : 0u;
    const uint32_t incl = warp_incl_scan(mytot, lane);
    const uint32_t n = __shfl_sync(0xffffffffu, incl, 31);
    uint32_t first = 0;
    if (lane == 0) first = atomicAdd(cursor, n);
    first = __shfl_sync(0xffffffffu, first, 0);
    if (lane < 16) wbase[lane] = first + incl - mytot;
    __syncwarp();
    const Stage st{res, spill};
    unsigned long long m = (unsigned long long)k0 | ((unsigned long long)k1 << 32);
    const unsigned long long all = m;
    while (m) {
        // up to four of this lane's entries per round: their reloads are in flight together
        int bit[4];
        uint32_t bits[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            bit[u] = -1;
            bits[u] = 0u;
            if (m) {
                bit[u] = __ffsll((long long)m) - 1;
                m &= m - 1;
                bits[u] = __ldg(tile + (((bit[u] >> 2) * 32 + lane) * 4 + (bit[u] & 3)));
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (bit[u] < 0) continue;
            const int i = bit[u] >> 2, c = bit[u] & 3;
            const uint32_t before_lanes = (pick4(excl[0], excl[1], excl[2], excl[3], i >> 2) >> (8 * (i & 3))) & 0xffu;
            const uint32_t before_mine = __popc((uint32_t)(all >> (4 * i)) & ((1u << c) - 1u));
            const uint32_t off = (uint32_t)((i * 32 + lane) * 4 + c);
            if (h2 != nullptr && (key_of(bits[u]) >> kShift1) == b1)   // second read: b1 is known, feed level 2 on the way
                atomicAdd(&h2[(key_of(bits[u]) >> kShift2) & (kBins2 - 1)], 1u);
            stage_put(st, wbase[i] + before_lanes + before_mine, make_uint2(bits[u], ytag | off));
        }
    }
    __syncwarp();   // wbase is rewritten by the warp's next tile
    return make_uint2(first, n);
}

// Out of line for the passes in which marked tiles are rare.
__device__ __noinline__ uint2 stage_marked(const uint32_t* __restrict__ tile, uint32_t k0, uint32_t k1, uint2* res,
                                           uint2* spill, uint32_t ytag, uint32_t* cursor, uint32_t* wbase,
                                           uint32_t* h2, uint32_t b1) {
    return stage_marked_body(tile, k0, k1, res, spill, ytag, cursor, wbase, h2, b1);
}

// keep[]: bit (4 * (i % 8) + c) of keep[i / 8] = component c of load i has key >= thr and lies in the layer.
__device__ __forceinline__ void mark_tile(const TileRegs& t, const uint32_t (&vm)[2], uint32_t thr, uint32_t (&keep)[2]) {
    keep[0] = keep[1] = 0u;
#pragma unroll
    for (int i = 0; i < 16; ++i) keep[i >> 3] |= keep4(t.v[i], thr) << (4 * (i & 7));
    keep[0] &= vm[0];
    keep[1] &= vm[1];
}

// Reading pass over one tile.  kHist: count every element in the level-1 histogram h.
// Entries with key >= thr are staged (thr = 0xffffffff: none).  Returns (first entry, entries).
template <bool kHist>
__device__ __forceinline__ uint2 read_tile(const float* __restrict__ acc, const TileSpan& ts, uint32_t* h,
                                           uint32_t thr, const Stage& st, uint32_t ytag, uint32_t* cursor,
                                           uint32_t* wbase, int lane, uint32_t* h2 = nullptr, uint32_t b1 = 0) {
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
    uint32_t keep[2];
    mark_tile(t, vm, thr, keep);
    if (!__any_sync(0xffffffffu, (keep[0] | keep[1]) != 0)) return make_uint2(0u, 0u);
    return stage_marked(reinterpret_cast<const uint32_t*>(acc + ts.lo), keep[0], keep[1], st.res, st.spill, ytag,
                        cursor, wbase, h2, b1);
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

// Fills the table of the CTA's streamed layers; returns how many there are (at most
// kMaxLocalLayers: checked on the host).
__device__ __forceinline__ int build_layer_table(const SelParams& p, const CtaRange& r, LayerTable* lt,
                                                 uint32_t* scratch) {
    int nl = 0;
    // scratch[kMTried - kMScratch] is the CTA's "speculated" flag (same misc area)
    const bool spec_on = !p.fixed_thr && __ldcg(p.spec_ctl) == 0u;
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
            lt->k[c] = (uint32_t)p.desc[j].k;
            // speculative cut: the bucket the previous call found for this layer, moved by as many
            // buckets (16 per octave) as the layer's norm has changed, lowered by a margin
            uint32_t sthr = 0xffffffffu;
            if (p.fixed_thr) {
                sthr = p.thr_key + 1u;                       // key >= thr_key + 1  <=>  key > thr_key
            } else if (spec_on && p.desc[j].k * kSpecDensity <= p.desc[j].end - p.desc[j].start) {
                const uint2 hint = __ldcg(p.hint + p.desc[j].layer_id);
                if (hint.x != 0 && hint.x <= (uint32_t)kBins1) {
                    int pb = (int)hint.x - 1;
                    const float was = __uint_as_float(hint.y), now = (float)p.desc[j].norm;
                    if (was > 0.0f && now > 0.0f && was < 3.0e38f && now < 3.0e38f)
                        pb += (int)floorf(16.0f * log2f(now / was));
                    pb = pb < 0 ? 0 : (pb > kBins1 - 1 ? kBins1 - 1 : pb);
                    sthr = (uint32_t)pb << kShift1;
                    scratch[kMTried - kMScratch] = 1u;
                }
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

// ---------------------------------------------------------------------------------
// step A: level-1 histograms (kSlots layers at a time) and speculative staging
// ---------------------------------------------------------------------------------
__device__ __forceinline__ void step_read1(const SelParams& p, const CtaRange& r, const LayerTable* lt, int nl,
                                           TileTable* tt, const Stage& st, unsigned char* smem) {
    uint32_t* hist = reinterpret_cast<uint32_t*>(smem + kSmMain);
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kSmMisc);
    uint32_t* wbase = reinterpret_cast<uint32_t*>(smem + kSmWBase);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) { misc[kMCursor] = 0; misc[kMFlag] = 0; misc[kMBudget] = 4096u; }
    __syncthreads();
    // staging budget: a few times what the CTA's tiles are expected to stage (k_l / size_l of its layers)
    for (int c = threadIdx.x; c < nl; c += kSelThreads) {
        const int64_t size = lt->end[c] - lt->start[c];
        const uint64_t per_tile = ((uint64_t)lt->k[c] * kTile + size - 1) / size;   // selected entries per tile, rounded up
        const uint64_t want = (uint64_t)own_tiles(p, r, lt, c) * per_tile * kSpecBudgetFactor;
        atomicAdd(&misc[kMBudget], (uint32_t)(want < 0x3fffffffull ? want : 0x3fffffffull));
    }
    __syncthreads();
    const uint32_t budget = misc[kMBudget] < 0x7fffffffu ? misc[kMBudget] : 0x7fffffffu;
    for (int c0 = 0; c0 < nl; c0 += kSlots) {
        const int ns = nl - c0 < kSlots ? nl - c0 : kSlots;
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
            const TileSpan ts = tile_span(lt->start[cl], lt->end[cl], lt->tf[cl], q);
            // a cut that turns out far too low must not flood the staging area: past the budget the
            // CTA stops staging and reads a second time in step B
            uint32_t thr = lt->sthr[cl];
            if (*reinterpret_cast<volatile uint32_t*>(misc + kMCursor) > budget) {
                thr = 0xffffffffu;
                if (lane == 0) {
                    misc[kMFlag] = 1u;
                    if (p.timing) p.timing[16 + 480 + blockIdx.x] = (1ull << 63) | ((unsigned long long)budget << 32) | (unsigned long long)cl;
                }
            }
            const uint2 fn = read_tile<true>(p.acc, ts, hist + (cl - c0) * kBins1, thr, st,
                                             pack_y(0u, (uint32_t)cl, (uint32_t)lq), misc + kMCursor,
                                             wbase + 16 * warp, lane);
            if (lane == 0) { tt->first[lq] = fn.x; tt->n[lq] = (uint16_t)fn.y; }
        }
        __syncthreads();
        stamp(p, 9);
        for (int i = threadIdx.x; i < ns * kBins1; i += kSelThreads) {
            const uint32_t cnt = hist[i];
            if (cnt) atomicAdd(p.hist1 + (size_t)lt->lid[c0 + i / kBins1] * kBins1 + (i % kBins1), cnt);
        }
        __syncthreads();
        stamp(p, 10);
        // ticket per layer: the CTA that flushes a layer's last tiles sees the complete histogram
        if ((int)threadIdx.x < ns) {
            const int cl = c0 + threadIdx.x;
            const uint32_t mine = own_tiles(p, r, lt, cl);
            __threadfence();
            const uint32_t old = atomicAdd(&p.state[lt->lid[cl]].ticket1, mine);
            misc[kMLast + threadIdx.x] = (old + mine == (uint32_t)(lt->tfe[cl] - lt->tf[cl])) ? 1u : 0u;
        }
        __syncthreads();
        stamp(p, 11);
        for (int s = 0; s < ns; ++s) {
            if (!misc[kMLast + s]) continue;   // uniform over the CTA
            const int cl = c0 + s;
            const int lid = lt->lid[cl];
            __threadfence();
            // besides b1: the bucket of a key some way further down, from which the next call takes its cut
            const uint32_t kk = lt->k[cl], k_safe = kk + (kk / 2 > kSpecSlack ? kk / 2 : kSpecSlack);
            block_scan_select(p.hist1 + (size_t)lid * kBins1, kBins1, true, kk, k_safe, misc + kMScratch,
                              misc + kMOut3);
            if (threadIdx.x == 0) {
                p.state[lid].b1 = misc[kMOut3];
                p.state[lid].above1 = misc[kMOut3 + 1];
                // the next call's speculative cut starts from here
                p.hint[lid] = make_uint2(misc[kMOut3 + 2] + 1u, __float_as_uint((float)p.desc[lt->j[cl]].norm));
            }
            __syncthreads();
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------
// step B: second read where the speculative cut was too high, then level-2 histograms
// ---------------------------------------------------------------------------------
__device__ __forceinline__ void step_read2(const SelParams& p, const CtaRange& r, LayerTable* lt, int nl,
                                           TileTable* tt, const Stage& st, unsigned char* smem) {
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
            if (lt->sthr[c] > need_thr) {                        // staged too little (or nothing) for this layer
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

// Ordered write of one batch of 32 consecutive staged entries (one per lane).  gt_before /
// eq_before: entries above / equal to the threshold that precede the batch in the layer.
struct EmitOut { float* val; int64_t* idx; float* acc_rw; int64_t cap; };

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

// ---------------------------------------------------------------------------------
// step S4: totals of the tiles before this CTA's, scan of the own tiles, ordered write
// ---------------------------------------------------------------------------------
// One batch of local tiles [t0, tend): pref[lq - t0] = entries above / equal to T that precede
// tile lq in its layer.  One warp per tile writes the tile's selected entries.
__device__ __noinline__ void emit_tiles(EmitOut out, int tiles, int il, int q0, const TileTable* tt, uint2* res,
                                        uint2* spill, const uint2* pref, int t0, int tend, int64_t start, int tf,
                                        int64_t out_off, uint32_t T, uint32_t need) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const Stage st{res, spill};
    // the warp's next tile that needs a warp: (lq, q) advance, false when there is none
    int lq = t0 + warp - kSelWarps, q = 0;
    auto next_tile = [&]() {
        for (lq += kSelWarps; lq < tend; lq += kSelWarps) {
            q = q0 + lq;
            if (il) {
                q = kSuper * ((int)blockIdx.x + (lq / kSuper) * (int)gridDim.x) + lq % kSuper;
                if (q >= tiles) continue;
            }
            if (tt->n[lq] > kThreadEmit) return true;   // the others: nothing staged, or written by their own thread
        }
        return false;
    };
    auto load_round = [&](uint32_t first, uint32_t n, uint32_t e0, uint2 (&ent)[kEmitBatch]) {
#pragma unroll
        for (int u = 0; u < kEmitBatch; ++u) {
            const uint32_t e = e0 + u * 32 + lane;
            ent[u] = e < n ? stage_get(st, first + e) : make_uint2(0u, 0u);
        }
    };
    bool have = next_tile();
    uint2 ent[kEmitBatch];
    if (have) load_round(tt->first[lq], tt->n[lq], 0u, ent);
    while (have) {
        const int lq_cur = lq;
        const uint32_t n = tt->n[lq_cur], first = tt->first[lq_cur];
        const int64_t lo = (start / kTile + (q - tf)) * kTile;
        uint32_t gt_before = pref[lq_cur - t0].x, eq_before = pref[lq_cur - t0].y;
        // the first round of the warp's next tile is in flight while this tile is written
        have = next_tile();
        uint2 ent_next[kEmitBatch];
        if (have) load_round(tt->first[lq], tt->n[lq], 0u, ent_next);
        for (uint32_t e0 = 0; e0 < n; e0 += 32 * kEmitBatch) {
            if (e0) load_round(first, n, e0, ent);
#pragma unroll
            for (int u = 0; u < kEmitBatch; ++u) {
                if (e0 + u * 32 < n)   // uniform over the warp
                    emit_batch(out, out_off, lo, e0 + u * 32 + lane < n, ent[u].x, (int64_t)y_off(ent[u].y), T, need,
                               gt_before, eq_before, lane);
            }
        }
#pragma unroll
        for (int u = 0; u < kEmitBatch; ++u) ent[u] = ent_next[u];
    }
}

// Tiles with at most kThreadEmit staged entries are written by ONE thread each (thread i of a
// batch owns tile t0 + i, whose prefix it has just computed): at a few entries per tile a warp
// per tile leaves most lanes idle and is bound by its own instruction latency.
__device__ __forceinline__ void emit_small_tile(const EmitOut& out, const Stage& st, uint32_t first, uint32_t n,
                                                int64_t out_off, int64_t lo, uint32_t T, uint32_t need,
                                                uint32_t gt_before, uint32_t eq_before) {
    for (uint32_t e = 0; e < n; ++e) {
        const uint2 ent = stage_get(st, first + e);
        const uint32_t key = key_of(ent.x);
        if (key > T || (key == T && eq_before < need)) {
            const int64_t pos = out_off + gt_before + (eq_before < need ? eq_before : need);
            const int64_t elem = lo + (int64_t)y_off(ent.y);
            if (pos < out.cap) {
                out.val[pos] = __uint_as_float(ent.x);
                out.idx[pos] = elem;
            }
            if (out.acc_rw) out.acc_rw[elem] = 0.0f;
        }
        gt_before += key > T;
        eq_before += key == T;
    }
}

__device__ __forceinline__ void step_emit(const SelParams& p, const CtaRange& r, LayerTable* lt, int nl,
                                          const TileTable* tt, const Stage& st, unsigned char* smem) {
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kSmMisc);
    uint2* pref = reinterpret_cast<uint2*>(smem + kSmPref);
    uint32_t* scratch = misc + kMScratch;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (r.il) {
        if (nl == 0) return;
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
        const uint32_t T = lt->v0[0], need = lt->v1[0];
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
            const uint2 sb = i < r.nloc ? sbase[i / kSuper] : make_uint2(0u, 0u);
            pref[threadIdx.x] = make_uint2(sb.x + (ex & 0xffffu), sb.y + (ex >> 16));
            bool big = false;
            {
                const int q = i < r.nloc ? local_tile(p, r, i) : -1;
                const uint32_t n = q >= 0 ? tt->n[i] : 0u;
                if (n != 0 && n <= kThreadEmit)
                    emit_small_tile(EmitOut{p.val, p.idx, p.acc_rw, p.out_cap}, st, tt->first[i], n, lt->out_off[0],
                                    (lt->start[0] / kTile + (q - lt->tf[0])) * kTile, T, need,
                                    sb.x + (ex & 0xffffu), sb.y + (ex >> 16));
                big = n > kThreadEmit;
            }
            const int tend = t0 + kSelThreads < r.nloc ? t0 + kSelThreads : r.nloc;
            if (__syncthreads_or(big ? 1 : 0))   // some tile of the batch needs a warp
                emit_tiles(EmitOut{p.val, p.idx, p.acc_rw, p.out_cap}, p.tiles, 1, 0, tt, st.res, st.spill, pref, t0, tend, lt->start[0],
                       lt->tf[0], lt->out_off[0], T, need);
            __syncthreads();   // pref is rewritten by the next batch
        }
        return;
    }
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
        const uint32_t T = lt->v0[c], need = lt->v1[c];
        uint32_t base_gt = lt->base_gt[c], base_eq = lt->base_eq[c];
        for (int t0 = ta; t0 < tb; t0 += kSelThreads) {   // batches of kSelThreads tiles
            const int i = t0 + (int)threadIdx.x;
            const uint32_t v = i < tb ? tt->ge[i] : 0u;
            uint32_t tot_gt, tot_eq;
            const uint32_t e_gt = block_excl_scan(v & 0xffffu, scratch, tot_gt);
            const uint32_t e_eq = block_excl_scan(v >> 16, scratch, tot_eq);
            pref[threadIdx.x] = make_uint2(base_gt + e_gt, base_eq + e_eq);
            bool big = false;
            {
                const uint32_t n = i < tb ? tt->n[i] : 0u;
                if (n != 0 && n <= kThreadEmit)
                    emit_small_tile(EmitOut{p.val, p.idx, p.acc_rw, p.out_cap}, st, tt->first[i], n, lt->out_off[c],
                                    (lt->start[c] / kTile + (r.q0 + i - lt->tf[c])) * kTile, T, need,
                                    base_gt + e_gt, base_eq + e_eq);
                big = n > kThreadEmit;
            }
            const int tend = t0 + kSelThreads < tb ? t0 + kSelThreads : tb;
            if (__syncthreads_or(big ? 1 : 0))   // some tile of the batch needs a warp
                emit_tiles(EmitOut{p.val, p.idx, p.acc_rw, p.out_cap}, p.tiles, 0, r.q0, tt, st.res, st.spill, pref, t0, tend, lt->start[c],
                       lt->tf[c], lt->out_off[c], T, need);
            base_gt += tot_gt;
            base_eq += tot_eq;
            __syncthreads();   // pref is rewritten by the next batch
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
            v[u] = f < n ? __ldg(x + f) : 0u;
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

// ---------------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------------
__global__ void __launch_bounds__(kSelThreads, 1) k_select_fused(const SelParams p) {
    extern __shared__ __align__(16) unsigned char smem[];
    cg::grid_group grid = cg::this_grid();

    if (p.timing && threadIdx.x == 0 && blockIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        p.timing[0] = t;
    }
    LayerTable* lt = reinterpret_cast<LayerTable*>(smem + kSmLayer);
    TileTable* tt = reinterpret_cast<TileTable*>(smem + kSmTile);
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kSmMisc);
    CtaRange r = cta_range(p, reinterpret_cast<int*>(smem + kSmTf));
    if (p.weighted)   // contiguous runs of equal estimated cost instead of equal length
        r = weighted_range(p, reinterpret_cast<uint32_t*>(smem + kSmMain), reinterpret_cast<int*>(smem + kSmTf),
                           misc + kMScratch);
    const int nl = build_layer_table(p, r, lt, misc + kMScratch);
    Stage st;
    st.res = reinterpret_cast<uint2*>(smem + kSmRes);
    st.spill = spill_base(p, r);

    if (!p.fixed_thr) {   // uniform over the grid
        unsigned long long ta0 = 0;
        if (p.timing && threadIdx.x == 0) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ta0));
        step_read1(p, r, lt, nl, tt, st, smem);
        if (p.timing && threadIdx.x == 0) {
            unsigned long long ta1;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ta1));
            p.timing[16 + 800 + blockIdx.x] = ta1 - ta0;
        }
        stamp(p, 1);
        grid.sync();
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
        // the last CTA to finish settles whether the next calls speculate: after a call with a failed
        // cut, the next kSpecCooldown calls read twice as a matter of course
        __threadfence();
        if (atomicAdd(p.spec_ctl + 2, 1u) == gridDim.x - 1) {
            const uint32_t cool = __ldcg(p.spec_ctl), failed = __ldcg(p.spec_ctl + 1);
            p.spec_ctl[0] = cool > 0 ? cool - 1 : (failed > 0 ? kSpecCooldown : 0u);
            p.spec_ctl[1] = 0u;
            p.spec_ctl[2] = 0u;
        }
    }
}

__global__ void k_zero_at(float* __restrict__ acc, const int64_t* __restrict__ idx, int64_t count) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count;
         i += (int64_t)gridDim.x * blockDim.x)
        acc[idx[i]] = 0.0f;
}

// CLT-k follower: own values at the leader's indices, then cleared.
__global__ void k_gather_zero(float* __restrict__ acc, const int64_t* __restrict__ idx, int64_t count,
                              float* __restrict__ val) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t j = idx[i];
        val[i] = acc[j];
        acc[j] = 0.0f;
    }
}

}  // namespace

deft_status launch_select(const SelParams& p, cudaStream_t stream) {
    static thread_local int attr_dev = -1;
    int dev = 0;
    DEFT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != attr_dev) {
        DEFT_CUDA_TRY(cudaFuncSetAttribute(k_select_fused, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           kSmemBytes));
        attr_dev = dev;
    }
    SelParams args = p;
    void* kargs[] = {&args};
    DEFT_CUDA_TRY(cudaLaunchCooperativeKernel(reinterpret_cast<void*>(k_select_fused), dim3(p.grid),
                                              dim3(kSelThreads), kargs, kSmemBytes, stream));
    return DEFT_OK;
}

deft_status launch_residual_update(float* acc_d, const int64_t* idx_d, int64_t count,
                                   cudaStream_t stream) {
    if (count == 0) return DEFT_OK;
    const int64_t want = (count + 255) / 256;
    const int64_t cap = (int64_t)sm_count() * 16;
    k_zero_at<<<(int)(want < cap ? want : cap), 256, 0, stream>>>(acc_d, idx_d, count);
    DEFT_CUDA_TRY(cudaGetLastError());
    return DEFT_OK;
}

deft_status launch_gather_update(float* acc_d, const int64_t* idx_d, int64_t count, float* val_d,
                                 cudaStream_t stream) {
    if (count == 0) return DEFT_OK;
    const int64_t want = (count + 255) / 256;
    const int64_t cap = (int64_t)sm_count() * 16;
    k_gather_zero<<<(int)(want < cap ? want : cap), 256, 0, stream>>>(acc_d, idx_d, count, val_d);
    DEFT_CUDA_TRY(cudaGetLastError());
    return DEFT_OK;
}

}  // namespace deft
