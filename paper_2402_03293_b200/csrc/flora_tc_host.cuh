// Host side of the tensor-core path: per-set tables and TMA descriptors, the work decomposition of the two kernels
// (plan_compress, plan_decompress) and their launches.  The kernels themselves are in flora_tc.cuh.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <atomic>
#include <vector>

#include <mutex>
#include <new>

#include "flora_pair.cuh"
#include "flora_pair_k2.cuh"
#include "flora_pool.cuh"
#include "flora_tc.cuh"

namespace flora {

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
struct TcSet {
    bool compress_ready = false;
    bool decompress_ready = false;
    bool transient = false;             // device buffers come from the stream-ordered allocator
    int count = 0, r = 0;
    int T = 1, gstages = 2, astages = 2, S = 1, GW = 8, P = 1;
    std::vector<int> k1_launch_first_mat;
    size_t k1_smem = 0;
    TcMatrix* d_mats = nullptr;
    K1Item* d_k1 = nullptr;
    int* d_split = nullptr;
    std::vector<TcMatrix> h_mats;
    std::vector<K1Item> h_k1;
    std::vector<int> k1_launch_begin;   // item ranges per launch (at most SEEDS_PER_LAUNCH matrices each)
    std::vector<int> split_mats;        // matrices whose sketch is updated by several items
    // ranks above 64: the persistent CTA-pair kernel; a launch's clusters ("slots") each walk their own list of units
    bool k1_pair = false;
    int k1_n = 0;                       // accumulator columns: r rounded up to a multiple of 64
    std::vector<int> h_slots;           // per launch: slots + 1 first-unit indices (relative to the launch's first unit)
    std::vector<int> k1_slots_begin;    // where each launch's table starts in h_slots
    int* d_slots = nullptr;
    // decompression
    int bn = 128, slots = 2, cstages = 2, k2_gw = 8, k2_nslabs = 2, k2_grid_max = 148;
    bool k2_bf16 = false;               // ranks above 64: the kernel reads a bf16 copy of the sketches
    bool k2_pair = false;               // ... and runs on CTA pairs (decompress_pair_kernel); k2_grid_max then counts pairs
    __nv_bfloat16* d_sb = nullptr;      // that copy (scratch owned by the set)
    std::vector<int> k2_launch_first_mat;
    size_t k2_smem = 0;
    K2Item* d_k2 = nullptr;
    std::vector<K2Item> h_k2;
    std::vector<int> k2_launch_begin;
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Looked up once per process (thread-safe: initialisation of a function-local static).
inline EncodeTiledFn encode_tiled_fn()
{
    static const EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            return reinterpret_cast<EncodeTiledFn>(p);
        cudaGetLastError();
        return static_cast<EncodeTiledFn>(nullptr);
    }();
    return fn;
}

// bf16 matrix, box = 64 columns x 128 rows, 128-byte swizzle, zero fill outside the matrix
inline bool make_map(CUtensorMap* out, const flora_mat& a)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)a.cols, (cuuint64_t)a.rows};
    cuuint64_t strides[1] = {(cuuint64_t)a.ld * 2};
    cuuint32_t box[2] = {64, 128};
    cuuint32_t estr[2] = {1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, a.data, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// fp32 sketch, box = 32 columns x 128 rows, 128-byte swizzle, zero fill outside the matrix
inline bool make_map_f32(CUtensorMap* out, const flora_mat& a)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)a.cols, (cuuint64_t)a.rows};
    cuuint64_t strides[1] = {(cuuint64_t)a.ld * 4};
    cuuint32_t box[2] = {32, 128};
    cuuint32_t estr[2] = {1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, a.data, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline bool tc_sketch_ok(const flora_mat& s)
{
    return (reinterpret_cast<uintptr_t>(s.data) & 15) == 0 && (s.ld & 3) == 0 && s.cols >= 1 && s.cols <= 256;
}

inline bool tc_mat_ok(const flora_mat& a)
{
    return a.dtype == FLORA_BF16 && a.rows >= 128 && a.cols >= 64 && (reinterpret_cast<uintptr_t>(a.data) & 15) == 0 &&
           (a.ld & 7) == 0 && a.rows < (1ll << 31) - 256 && a.cols < (1ll << 31) - 256;
}

inline bool tc_compress_supported(const flora_mat* big, const flora_mat* sketch)
{
    return tc_mat_ok(*big) && tc_sketch_ok(*sketch) && encode_tiled_fn() != nullptr;
}

// SMs of the current device (queried on every call: a process may drive several devices).
inline int sm_count()
{
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
        cudaGetLastError();
        n = 148;
    }
    return n;
}

constexpr size_t SMEM_BUDGET = 226 * 1024;   // per SM, below the 227 KB limit of sm_100

// Process-wide switch (flora_set_deterministic): when on, no sum is split over CTAs that add their parts in arrival
// order, so that repeated runs give the same bits.  Read when a set is planned and at every transfer.
inline std::atomic<int>& deterministic_flag()
{
    static std::atomic<int> flag{0};
    return flag;
}

// Tile shapes and the work split are chosen by the planners below.  A build with -DFLORA_TUNE lets environment
// variables override single choices for parameter sweeps (they never change what is computed); the library as
// shipped reads no environment variable.
#ifdef FLORA_TUNE
inline int tune_knob(const char* name, int dflt, int lo, int hi)
{
    const char* v = getenv(name);
    if (!v || !*v) return dflt;
    return std::max(lo, std::min(hi, atoi(v)));
}
#else
inline int tune_knob(const char*, int dflt, int, int) { return dflt; }
#endif

// Lifts a kernel's limit on dynamic shared memory to what the device allows, once per kernel and device.  The
// attribute belongs to the function, not to a launch: it is raised to the maximum once and never lowered, so sets
// with different footprints can be alive, and launched in any order, at the same time.
template <auto Kernel>
inline bool raise_smem_limit()
{
    static std::mutex mutex;
    static bool done[POOL_MAX_DEVICES] = {};
    int dev = -1, optin = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= POOL_MAX_DEVICES) {
        cudaGetLastError();
        return false;
    }
    std::lock_guard<std::mutex> lock(mutex);
    if (done[dev]) return true;
    if (cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess ||
        cudaFuncSetAttribute(Kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, optin) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    done[dev] = true;
    return true;
}

// Clusters of `S` CTAs of `Kernel` that can be resident at once (fewer than SMs / S: a cluster sits inside one GPC);
// SMs / S when there is no device to ask.
template <auto Kernel>
inline int resident_clusters(int S, int threads, size_t smem)
{
    int slots = std::max(1, sm_count() / S);
    if (!raise_smem_limit<Kernel>()) return slots;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(S * 64));
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)S;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int active = 0;
    if (cudaOccupancyMaxActiveClusters(&active, Kernel, &cfg) == cudaSuccess && active > 0) slots = active;
    else cudaGetLastError();
    return slots;
}

// Cost model of the compression planners, in units of one 64-column step of a full CTA: what a work unit costs
// before its first and after its last step (barriers, first loads, writing the accumulators out).
constexpr double K1_UNIT_OVERHEAD_STEPS = 6.0;
// Cost model of the r <= 64 compression planner: generating one value of A costs this many times the share of HBM
// time that one element of a 128-row G tile costs its CTA (measured: an r x 64 tile takes about r * 64 * 0.18 ns of
// one SM's ALUs, the 16 KB of a G tile 0.37 us of its share of HBM, and the ratio of the two per rank is about 0.045 / T).
constexpr double K1_GENERATION_PER_RANK = 0.045;
// Cost model of the decompression planner (microseconds on one SM): bytes an SM takes in per microsecond whatever their
// source (about 60 GB/s with the tiles it can keep in flight), values of A per microsecond that the generator warps
// make next to the streaming warps (8 or fewer warps), the share of a slab's generation that stays exposed with one
// slab buffer (the combine warps help) or overlaps badly with two, and the fixed cost of an item.
constexpr double K2_SM_BYTES_PER_US = 60e3;
constexpr double K2_VALUES_PER_US_8_WARPS = 2000.0, K2_VALUES_PER_US_FEWER = 1300.0;
constexpr double K2_EXPOSED_ONE_SLAB = 0.55, K2_OVERLAP_PENALTY = 0.35, K2_ITEM_OVERHEAD_US = 0.2;

// Work decomposition of compress_pair_kernel (ranks above 64).
//
// A unit is (matrix, group of up to S * PAIR_T 128-row tiles, range of 64-column steps); a cluster of S CTAs
// (S/2 pairs) handles one unit at a time, the CTAs taking consecutive rows.  Units are balanced over the clusters
// that can be resident ("slots"), largest first; every slot gets its own list, which its cluster walks.
inline void plan_compress_pair(TcSet& set, const std::vector<flora_mat>& G, int r)
{
    const int N = (r + 63) & ~63;
    const int T = PAIR_T;
    int64_t max_tiles = 1, total_work = 0;
    for (const auto& g : G) {
        const int64_t tiles = (g.rows + 127) / 128, ks = (g.cols + 63) / 64;
        max_tiles = std::max(max_tiles, tiles);
        total_work += tiles * ks;
    }
    // Clusters of eight wherever the matrices have the rows for them: a slice of A then serves 2048 rows, and a 1600-row
    // matrix is one unit (at N = 128 clusters of four keep a CTA's share of a slice within what its generators make
    // during a step, and fit 132 SMs instead of 120, but generate every slice of such a matrix twice: 824 against 714 us
    // on config 5's set at r = 128, 32.8 against 28.9 us on one 4096 x 11008 matrix).
    int S = 8;
    while (S > 2 && (int64_t)S * T > 2 * max_tiles) S >>= 1;          // not more CTAs than there are rows to share
    S = tune_knob("FLORA_K1_CLUSTER", S, 2, 8);
    if (S & (S - 1)) S = 2;
    const size_t g_stage = (size_t)T * G_TILE_BYTES, a_stage = (size_t)(N / 2) * 128, staging = 2 * (size_t)S_CHUNK_BYTES_K1;
    const size_t ring_budget = SMEM_BUDGET - sizeof(PairSmem) - 1024 - staging;
    // A tiles are made on chip by warps that each need about two microseconds for their share of a slice, and travel
    // between the CTAs of a cluster, whose slowest member paces all: six stages keep enough slices in the making
    // (five when that leaves fewer than three stages for G).  The G tiles come from HBM and get the rest.
    int astages = 6;
    if ((ring_budget - astages * a_stage) / g_stage < 3) astages = 5;
    {
        // ... and enough of them that sixteen generator warps and the epilogue warps can all hold a claim (see below):
        // narrow slices (N = 128 in a cluster of eight: four work items per step) need up to eight stages of 8 KB
        const int parts = (N / S * 8 + 31) / 32;
        const int wanted = (PAIR_MAX_GEN_WARPS + PAIR_EPI_WARPS + parts - 1) / parts + 2;
        while (astages < std::min(8, wanted) && (ring_budget - (astages + 1) * a_stage) / g_stage >= 3) ++astages;
    }
    astages = tune_knob("FLORA_K1_ASTAGES", astages, 2, 8);
    int gstages = (int)std::min<size_t>(PAIR_RELAY_DEPTH - 1, (ring_budget - astages * a_stage) / g_stage);
    gstages = tune_knob("FLORA_K1_GSTAGES", std::max(1, gstages), 1, std::max(1, gstages));
    // Worker warps claim generation work items (32 tasks of one slice) in order.  A warp waits for its stage by the
    // parity of the stage's use count, which is only sound while no claim is a whole ring ahead of the oldest
    // unfinished one: the warps together must hold fewer than (astages - 1) steps' worth of items.
    int GW = tune_knob("FLORA_K1_GEN_WARPS", PAIR_MAX_GEN_WARPS, 12, PAIR_MAX_GEN_WARPS) & ~3;
    {
        const int parts = (N / S * 8 + 31) / 32;
        while (GW > 12 && (GW + PAIR_EPI_WARPS + parts - 1) / parts + 1 >= astages) GW -= 4;    // (the kernel's warp layout wants at least 12)
        set.P = 1;
    }
    set.k1_pair = true;
    set.k1_n = N;
    set.T = T;
    set.S = S;
    set.GW = GW;
    set.gstages = gstages;
    set.astages = astages;
    set.k1_smem = (size_t)gstages * g_stage + (size_t)astages * a_stage + staging + sizeof(PairSmem) + 1024;
    const int64_t slots = resident_clusters<compress_pair_kernel>(S, pair_threads(GW), set.k1_smem);
    const int64_t group_tiles = (int64_t)S * T;
    struct Unit { int mat; int64_t tile0, tiles, kstep0, ksteps; bool direct; };
    auto build_units = [&](int64_t target, std::vector<Unit>& units, std::vector<int>& split) {
        units.clear();
        split.clear();
        for (size_t i = 0; i < G.size(); ++i) {
            const auto& g = G[i];
            if (g.rows == 0 || g.cols == 0) continue;
            const int64_t tiles = (g.rows + 127) / 128, ks = (g.cols + 63) / 64;
            const int64_t groups = (tiles + group_tiles - 1) / group_tiles;
            const int64_t per_group = (tiles + groups - 1) / groups;     // rows spread evenly over the groups
            int64_t chunk = std::max<int64_t>(8, target / per_group);
            int64_t nchunks = (ks + chunk - 1) / chunk;
            if (nchunks > 1 && ks - (nchunks - 1) * chunk < chunk / 2) --nchunks;    // no short tail unit
            chunk = (ks + nchunks - 1) / nchunks;
            nchunks = (ks + chunk - 1) / chunk;
            if (nchunks > 1) split.push_back((int)i);
            for (int64_t t0 = 0; t0 < tiles; t0 += per_group)
                for (int64_t c = 0; c < nchunks; ++c)
                    units.push_back({(int)i, t0, std::min(per_group, tiles - t0), c * chunk, std::min(chunk, ks - c * chunk), nchunks == 1});
        }
    };
    // a cluster moves in lockstep and every step costs a full CTA's worth of MMAs: a unit's time is its steps plus
    // the fixed cost of starting and finishing it
    auto unit_time = [&](const Unit& u) { return K1_UNIT_OVERHEAD_STEPS + (double)u.ksteps; };
    // longest-processing-time assignment of units[first, last) to the slots; returns the makespan
    auto assign = [&](const std::vector<Unit>& units, size_t first, size_t last, std::vector<std::vector<int>>* lists) {
        std::vector<int> order;
        for (size_t u = first; u < last; ++u) order.push_back((int)u);
        std::stable_sort(order.begin(), order.end(), [&](int x, int y) { return unit_time(units[x]) > unit_time(units[y]); });
        std::vector<std::pair<double, int>> heap;                // (time assigned, slot), smallest time on top
        for (int s = 0; s < (int)slots; ++s) heap.push_back({0.0, s});
        auto cmp = [](const std::pair<double, int>& x, const std::pair<double, int>& y) { return x.first > y.first || (x.first == y.first && x.second > y.second); };
        std::make_heap(heap.begin(), heap.end(), cmp);
        if (lists) lists->assign((size_t)slots, std::vector<int>());
        double span = 0.0;
        for (int u : order) {
            std::pop_heap(heap.begin(), heap.end(), cmp);
            heap.back().first += unit_time(units[u]);
            span = std::max(span, heap.back().first);
            if (lists) (*lists)[(size_t)heap.back().second].push_back(u);
            std::push_heap(heap.begin(), heap.end(), cmp);
        }
        return span;
    };
    // column chunks: try several granularities (about 1..4 units per slot) and keep the shortest schedule
    std::vector<Unit> units, cand_units;
    std::vector<int> cand_split;
    double best_span = 1e300;
    for (int w = 1; w <= 4; ++w) {
        for (double f : {1.0, 1.1, 1.2, 1.35, 1.5}) {
            const int64_t target = (int64_t)((double)total_work / (double)(w * slots * group_tiles) * f * (double)group_tiles) + 1;
            build_units(target, cand_units, cand_split);
            const double span = assign(cand_units, 0, cand_units.size(), nullptr);
            if (span < best_span * 0.98) {
                best_span = span;
                units = cand_units;
                set.split_mats = cand_split;
            }
        }
    }
    // a schedule without any split over columns is preferred when it is nearly as short: every row of a sketch then
    // has one owner, so a momentum update needs neither the pre-scaling pass nor atomic adds
    build_units((int64_t)1 << 60, cand_units, cand_split);
    if (deterministic_flag().load() || assign(cand_units, 0, cand_units.size(), nullptr) <= 1.12 * best_span) {
        units = cand_units;
        set.split_mats = cand_split;
    }
    // launches cover at most SEEDS_PER_LAUNCH consecutive matrices (units are in matrix order)
    set.h_k1.clear();
    set.h_slots.clear();
    set.k1_launch_begin.clear();
    set.k1_launch_first_mat.clear();
    set.k1_slots_begin.clear();
    size_t u0 = 0;
    while (u0 < units.size()) {
        size_t u1 = u0;
        while (u1 < units.size() && units[u1].mat < units[u0].mat + SEEDS_PER_LAUNCH) ++u1;
        std::vector<std::vector<int>> lists;
        assign(units, u0, u1, &lists);
        set.k1_launch_begin.push_back((int)set.h_k1.size());
        set.k1_launch_first_mat.push_back(units[u0].mat);
        set.k1_slots_begin.push_back((int)set.h_slots.size());
        int emitted = 0;                                        // units of this launch so far
        for (const auto& list : lists) {
            if (list.empty()) continue;                         // slots without work are not launched
            set.h_slots.push_back(emitted);
            for (int u : list) {
                // the unit's tiles spread evenly over the S CTAs of the cluster (some may get none)
                const Unit& un = units[(size_t)u];
                int64_t t0 = un.tile0;
                for (int c = 0; c < S; ++c) {
                    const int64_t left = un.tile0 + un.tiles - t0;
                    const int64_t mine = std::min<int64_t>(T, (left + (S - c) - 1) / (S - c));
                    K1Item it;
                    it.mat = un.mat;
                    it.row0 = (int)(t0 * 128);
                    it.tiles = (int)std::max<int64_t>(0, mine);
                    it.kstep0 = (int)un.kstep0;
                    it.ksteps = (int)un.ksteps;
                    it.direct = un.direct;
                    set.h_k1.push_back(it);
                    t0 += it.tiles;
                }
                ++emitted;
            }
        }
        set.h_slots.push_back(emitted);
        u0 = u1;
    }
    set.k1_launch_begin.push_back((int)set.h_k1.size());
    set.k1_slots_begin.push_back((int)set.h_slots.size());
}

// Work decomposition of the compression kernel over a set of matrices.
//
// A CTA handles up to T 128-row tiles; S CTAs (a thread-block cluster) handle neighbouring row groups of the
// same matrix over the same columns and share the generation of A.  The generation of one r x 64 tile costs
// about r*64*0.18 ns of one SM's ALUs, the loads of a CTA's T tiles T*0.37 us of its share of HBM: S is chosen
// so that the former stays under half of the latter.
inline void plan_compress(TcSet& set, const std::vector<flora_mat>& G, int r)
{
    if (r > 64) {
        plan_compress_pair(set, G, r);
        return;
    }
    set.k1_pair = false;
    const int r_pad = (r + 15) & ~15;
    int64_t max_tiles = 1, total_work = 0;       // work unit: one 128-row tile over one 64-column step
    for (const auto& g : G) {
        const int64_t tiles = (g.rows + 127) / 128, ks = (g.cols + 63) / 64;
        max_tiles = std::max(max_tiles, tiles);
        total_work += tiles * ks;
    }
    // T: bounded by tensor memory (T * r_pad <= 512 columns).  The largest value, unless a smaller one removes
    // more than a fifth of the tile slots that row counts which are no multiple of T * 128 leave empty
    // (empty slots cost MMA issue and shared memory, not HBM traffic).
    // (for r <= 32 at most 3 tiles, so that two CTAs with two stages each fit one SM)
    const int t_cap = (int)std::min<int64_t>(std::min<int64_t>(max_tiles, 512 / r_pad), r_pad <= 32 ? 3 : 4);
    auto padded_work = [&](int cand) {
        double padded = 0;
        for (const auto& g : G) {
            const int64_t tiles = (g.rows + 127) / 128, ks = (g.cols + 63) / 64;
            padded += (double)((tiles + cand - 1) / cand * cand) * ks;
        }
        return padded;
    };
    int T = t_cap;
    for (int cand = t_cap - 1; cand >= 1; --cand)
        if (padded_work(cand) < 0.8 * padded_work(T)) T = cand;
    T = tune_knob("FLORA_K1_T", T, 1, 512 / r_pad);
    const size_t stage = (size_t)T * G_TILE_BYTES + (size_t)r_pad * 128;
    uint32_t cols = 32;
    while ((int)cols < T * r_pad) cols <<= 1;
    // cluster size from the generation / load ratio
    const double ratio = r * K1_GENERATION_PER_RANK / T;
    int S = 1;
    while (S < 8 && ratio / S > 0.5) S <<= 1;
    while (S > 1 && (int64_t)S * T > 2 * max_tiles) S >>= 1;         // not more CTAs than there are rows to share
    S = tune_knob("FLORA_K1_CLUSTER", S, 1, 8);
    if (S & (S - 1)) S = 1;
    while (S > 1 && r_pad % (8 * S)) S >>= 1;                     // every CTA's slice of A is whole 8-row groups
    // two CTAs per SM when tensor memory allows it and each still gets two stages: the epilogue of one
    // overlaps the loads of the other (single-CTA clusters only)
    int per_sm = (S == 1 && cols <= 256 && 2 * stage <= SMEM_BUDGET / 2) ? 2 : 1;
    per_sm = tune_knob("FLORA_K1_PER_SM", per_sm, 1, (S == 1 && cols <= 256) ? 2 : 1);
    // Two rings.  The G tiles come from HBM: with a latency near 2 us under load, the bytes in flight per SM, not the
    // link, bound the intake, so the G ring gets all the shared memory the A ring does not need.  A tiles are made on
    // chip: two stages; three (four for the large tiles of ranks above 128) where slices travel between the CTAs of a
    // cluster and the slowest CTA paces all of them.
    const size_t g_stage = (size_t)T * G_TILE_BYTES, a_stage = (size_t)r_pad * 128;
    const size_t ring_budget = SMEM_BUDGET / per_sm - sizeof(K1Smem) - 1024;
    int astages = S > 1 ? (r_pad > 128 ? 4 : 3) : 2;
    if ((ring_budget - astages * a_stage) / g_stage < 2) astages = 2;
    astages = tune_knob("FLORA_K1_ASTAGES", astages, 1, 8);
    int gstages = (int)std::min<size_t>(8, (ring_budget - std::min(ring_budget, astages * a_stage)) / g_stage);
    gstages = tune_knob("FLORA_K1_GSTAGES", std::max(1, gstages), 1, std::max(1, gstages));
    // generator warps: 16 where one CTA owns the SM and generation is a sizeable share of the work
    int GW = (per_sm == 1 && ratio / S > 0.15) ? 16 : 8;
    GW = tune_knob("FLORA_K1_GEN_WARPS", GW, 4, per_sm == 1 ? K1_MAX_GEN_WARPS : 8);
    set.GW = GW;
    // generator teams: as many as keep every thread of a team busy with at least one task per tile
    {
        const int tile_tasks = (S > 1 ? r_pad / S : r) * 8;
        int P = 1;
        while (2 * P <= astages && GW % (2 * P) == 0 && 32 * GW / (2 * P) >= tile_tasks) P *= 2;
        P = tune_knob("FLORA_K1_TEAMS", P, 1, 8);
        while (P > 1 && (GW % P || P > astages || (P & (P - 1)))) --P;
        set.P = P;
    }
    set.T = T;
    set.S = S;
    set.gstages = gstages;
    set.astages = astages;
    set.k1_smem = (size_t)gstages * g_stage + (size_t)astages * a_stage + sizeof(K1Smem) + 1024;
    // column chunks: aim at about `waves` items per slot (a slot is a CTA, or a cluster), at least 8 steps each
    int64_t slots = std::max<int64_t>(1, (int64_t)sm_count() * per_sm / S);
    if (S > 1) slots = resident_clusters<compress_tc_kernel>(S, k1_threads(set.GW), set.k1_smem);
    const int64_t group_tiles = (int64_t)S * T;                      // rows of one slot, in tiles
    struct Unit { int mat; int64_t tile0, tiles, kstep0, ksteps; bool direct; };
    auto build_units = [&](int64_t target, std::vector<Unit>& units, std::vector<int>& split) {
        units.clear();
        split.clear();
        for (size_t i = 0; i < G.size(); ++i) {
            const auto& g = G[i];
            if (g.rows == 0 || g.cols == 0) continue;
            const int64_t tiles = (g.rows + 127) / 128, ks = (g.cols + 63) / 64;
            const int64_t groups = (tiles + group_tiles - 1) / group_tiles;
            const int64_t per_group = (tiles + groups - 1) / groups;     // rows spread evenly over the groups
            int64_t chunk = std::max<int64_t>(8, target / per_group);
            int64_t nchunks = (ks + chunk - 1) / chunk;
            if (nchunks > 1 && ks - (nchunks - 1) * chunk < chunk / 2) --nchunks;    // no short tail item
            chunk = (ks + nchunks - 1) / nchunks;
            nchunks = (ks + chunk - 1) / chunk;
            if (nchunks > 1) split.push_back((int)i);
            for (int64_t t0 = 0; t0 < tiles; t0 += per_group)
                for (int64_t c = 0; c < nchunks; ++c)
                    units.push_back({(int)i, t0, std::min(per_group, tiles - t0), c * chunk, std::min(chunk, ks - c * chunk), nchunks == 1});
        }
    };
    // time of a unit on its slot, in 64-column steps of a full slot: a fixed start-up / epilogue cost plus its steps,
    // scaled by the rows a CTA streams (a cluster moves in lockstep, so its most loaded CTA counts)
    auto unit_time = [&](const Unit& u) {
        const double per_cta = (double)((u.tiles + S - 1) / S);
        return (K1_UNIT_OVERHEAD_STEPS + (double)u.ksteps) * std::max(per_cta, 0.5 * T);
    };
    auto makespan = [&](const std::vector<Unit>& units) {
        std::vector<double> tms;
        for (const auto& u : units) tms.push_back(unit_time(u));
        std::sort(tms.begin(), tms.end(), std::greater<double>());
        std::vector<double> free_at((size_t)slots, 0.0);     // min-heap of slot availability
        auto cmp = std::greater<double>();
        for (double t : tms) {
            std::pop_heap(free_at.begin(), free_at.end(), cmp);
            free_at.back() += t;
            std::push_heap(free_at.begin(), free_at.end(), cmp);
        }
        return *std::max_element(free_at.begin(), free_at.end());
    };
    // column chunks: try several granularities (about 1..4 units per slot) and keep the shortest schedule
    std::vector<Unit> units, cand_units;
    std::vector<int> cand_split;
    double best_span = 1e300;
    const int fixed_waves = tune_knob("FLORA_K1_WAVES", 0, 0, 64);
    for (int w = 1; w <= 4; ++w) {
        for (double f : {1.0, 1.1, 1.2, 1.35, 1.5}) {
            if (fixed_waves && (w != fixed_waves || f != 1.0)) continue;
            const int64_t target = (int64_t)((double)total_work / (double)((fixed_waves ? fixed_waves : w) * slots) * f) + 1;
            build_units(target, cand_units, cand_split);
            const double span = makespan(cand_units);
            if (span < best_span * 0.98) {
                best_span = span;
                units = cand_units;
                set.split_mats = cand_split;
            }
        }
    }
    // a schedule without any split over columns is preferred when it is nearly as short: every row of a sketch then
    // has one owner, so a momentum update needs neither the pre-scaling pass nor atomic adds
    if (!fixed_waves) {
        build_units((int64_t)1 << 60, cand_units, cand_split);
        if (deterministic_flag().load() || makespan(cand_units) <= 1.12 * best_span) {
            units = cand_units;
            set.split_mats = cand_split;
        }
    }
    // launches cover at most SEEDS_PER_LAUNCH consecutive matrices; inside a launch the largest units go first
    set.h_k1.clear();
    set.k1_launch_begin.clear();
    set.k1_launch_first_mat.clear();
    size_t u0 = 0;
    while (u0 < units.size()) {
        size_t u1 = u0;
        while (u1 < units.size() && units[u1].mat < units[u0].mat + SEEDS_PER_LAUNCH) ++u1;
        const int first_mat = units[u0].mat;          // before sorting: units are still in matrix order here
        if (tune_knob("FLORA_K1_SORT", 1, 0, 1))
            std::stable_sort(units.begin() + u0, units.begin() + u1,
                             [](const Unit& x, const Unit& y) { return x.tiles * x.ksteps > y.tiles * y.ksteps; });
        set.k1_launch_begin.push_back((int)set.h_k1.size());
        set.k1_launch_first_mat.push_back(first_mat);
        for (size_t u = u0; u < u1; ++u) {
            // the unit's tiles spread evenly over the S CTAs of the slot (some may get none)
            const Unit& un = units[u];
            int64_t t0 = un.tile0;
            for (int c = 0; c < S; ++c) {
                const int64_t left = un.tile0 + un.tiles - t0;
                const int64_t mine = std::min<int64_t>(T, (left + (S - c) - 1) / (S - c));
                K1Item it;
                it.mat = un.mat;
                it.row0 = (int)(t0 * 128);
                it.tiles = (int)std::max<int64_t>(0, mine);
                it.kstep0 = (int)un.kstep0;
                it.ksteps = (int)un.ksteps;
                it.direct = un.direct;
                set.h_k1.push_back(it);
                t0 += it.tiles;
            }
        }
        u0 = u1;
    }
    set.k1_launch_begin.push_back((int)set.h_k1.size());
}

// Work decomposition of the decompression kernel: column slabs of bn columns, cut into runs of row tiles; the
// persistent CTAs take the items round-robin, largest first.
inline void plan_decompress(TcSet& set, const std::vector<flora_mat>& W, int r)
{
    // ranks up to 64 read the fp32 sketch directly (tf32 MMA); above that the bytes of S that a CTA pulls per W
    // tile exceed what shared memory can keep in flight, so a bf16 copy of S is made first (half the bytes,
    // twice the K depth per 128-byte row) and the MMA runs in bf16
    const bool bf16s = tune_knob("FLORA_K2_BF16S", r > 64 ? 1 : 0, 0, 1) != 0;
    set.k2_bf16 = bf16s;
    const int kchunks = bf16s ? (r + 63) / 64 : (r + 31) / 32;
    // slabs of 128 columns (every chunk of S then serves twice the columns of W) whenever two slabs, two W slots and
    // two S chunks of that width fit; 64 columns otherwise
    const size_t ctl = sizeof(K2Smem) + 1024;
    int bn = (2 * (size_t)kchunks * 128 * 128 + 2 * S_CHUNK_BYTES + 2 * 2 * (size_t)W_BOX_BYTES + ctl <= SMEM_BUDGET) ? 128 : 64;
    bn = tune_knob("FLORA_K2_BN", bn, 64, 128) >= 128 ? 128 : 64;
    const size_t slab_bytes = (size_t)kchunks * bn * 128, slot = (size_t)(bn / 64) * W_BOX_BYTES;
    // two CTAs per SM when two of them fit (each with two slabs, two W slots and one S chunk)
    const size_t per_cta_max = 113 * 1024;                       // half of an SM's shared memory minus the reserve
    int per_sm = (2 * slab_bytes + S_CHUNK_BYTES + 2 * slot + ctl <= per_cta_max) ? 2 : 1;
    per_sm = 1;   // twelve fixed warps plus generators: one CTA per SM
    // Two slab buffers (the next item's slab is generated while the current item streams) unless that leaves fewer
    // than four S chunks in flight: the chunks of one W tile are kchunks x 16 KB, and with too few of them under way
    // the loads' latency, not bandwidth, sets the pace.  With one buffer every warp that is idle between two items
    // (the combine warps) shares the generation.
    int nslabs = (2 * slab_bytes + 4 * S_CHUNK_BYTES + 2 * slot + ctl <= SMEM_BUDGET) ? 2 : 1;
    nslabs = tune_knob("FLORA_K2_SLABS", nslabs, 1, 2);
    const size_t budget = (per_sm == 2 ? per_cta_max : SMEM_BUDGET) - ctl - nslabs * slab_bytes;
    int cstages = std::max(2, std::min(nslabs == 1 ? 2 * kchunks : kchunks + 1, nslabs == 1 ? K2_MAX_CSTAGES : 4));
    cstages = tune_knob("FLORA_K2_CSTAGES", cstages, 1, K2_MAX_CSTAGES);
    while (cstages > 1 && (size_t)cstages * S_CHUNK_BYTES + 2 * slot > budget) --cstages;
    int slots = (int)std::min<size_t>(K2_MAX_SLOTS, (budget - (size_t)cstages * S_CHUNK_BYTES) / slot);
    slots = tune_knob("FLORA_K2_SLOTS", slots, 1, std::max(1, slots));
    int GW = 8;
    GW = tune_knob("FLORA_K2_GEN_WARPS", GW, 1, K2_MAX_GEN_WARPS);
    set.bn = bn;
    set.slots = slots;
    set.cstages = cstages;
    set.k2_gw = GW;
    set.k2_nslabs = nslabs;
    set.k2_smem = nslabs * slab_bytes + (size_t)cstages * S_CHUNK_BYTES + (size_t)slots * slot + sizeof(K2Smem) + 1024;
    int grid_max = sm_count() * per_sm;
    // Ranks above 128 run on CTA pairs: each CTA holds half of a 128-column slab (two buffers of kchunks x 8 KB), the
    // sketch chunks of its own tiles (as many stages as fit beside two W tiles, at most two tiles' worth) and its W tiles.
    // Above r = 192 one CTA has room for a single slab buffer only; from r = 129 to 192 it has room for two, and the pair
    // is still the faster (config 5's set at r = 192: 1335 against 1447 us; one 4096 x 11008 matrix: 54 against 58 us).
    // Up to r = 128 one CTA per SM wins on sets (1087 against 1453 us).
    const bool pair = bf16s && tune_knob("FLORA_K2_PAIR", kchunks >= 3 ? 1 : 0, 0, 1) != 0;
    set.k2_pair = pair;
    if (pair) {
        const size_t half_slab = (size_t)kchunks * 64 * 128, pslot = 2 * (size_t)W_BOX_BYTES;
        const size_t pbudget = SMEM_BUDGET - sizeof(K2PairSmem) - 1024 - 2 * half_slab;
        int pc = std::min(K2_MAX_CSTAGES, 2 * kchunks);
        pc = tune_knob("FLORA_K2_CSTAGES", pc, 2, K2_MAX_CSTAGES);
        while (pc > 2 && (size_t)pc * S_CHUNK_BYTES + 2 * pslot > pbudget) --pc;
        pc &= ~1;                                        // two rings of equal depth, one per MMA-issuing thread
        int ps = (int)std::min<size_t>(K2_MAX_SLOTS, (pbudget - (size_t)pc * S_CHUNK_BYTES) / pslot);
        ps = tune_knob("FLORA_K2_SLOTS", ps, 2, std::max(2, ps));
        bn = set.bn = K2P_BN;
        nslabs = set.k2_nslabs = 2;
        cstages = set.cstages = pc;
        slots = set.slots = ps;
        GW = set.k2_gw = K2P_GEN_WARPS;
        set.k2_smem = decompress_pair_smem_bytes(r, ps, pc);
        grid_max = std::max(1, sm_count() / 2);
    }
    const double pair_f = pair ? 0.5 : 1.0;          // a pair streams an item's tiles two at a time, and each CTA generates half a slab
    // cost model (microseconds of one SM): a tile streams bn*128*4 bytes at the SM's share of HBM; a slab costs
    // r*bn normals at the generator warps' rate and overlaps the previous item's streaming
    // (an SM takes in about 60 GB/s whatever the source: the chunks of S count like the W tile itself)
    const double t_tile = std::max((double)bn * 128 * 4 / (6.5e6 / sm_count()),
                                   ((double)bn * 128 * 2 + (double)kchunks * S_CHUNK_BYTES) / K2_SM_BYTES_PER_US);
    const double t_slab = (double)r * bn / (GW >= 8 ? K2_VALUES_PER_US_8_WARPS : K2_VALUES_PER_US_FEWER);   // generator warps share the SM with the streaming warps
    auto build = [&](int run, std::vector<K2Item>& out) {
        out.clear();
        for (size_t i = 0; i < W.size(); ++i) {
            const auto& w = W[i];
            if (w.rows == 0 || w.cols == 0) continue;
            const int64_t rtiles = (w.rows + 127) / 128, slabs = (w.cols + bn - 1) / bn;
            const int64_t groups = (rtiles + run - 1) / run;
            const int64_t per = (rtiles + groups - 1) / groups;
            for (int64_t sl = 0; sl < slabs; ++sl)
                for (int64_t t0 = 0; t0 < rtiles; t0 += per) {
                    K2Item it;
                    it.mat = (int)i;
                    it.col0 = (int)(sl * bn);
                    it.row0 = (int)(t0 * 128);
                    it.tiles = (int)std::min<int64_t>(per, rtiles - t0);
                    out.push_back(it);
                }
        }
    };
    auto sort_items = [&](std::vector<K2Item>& v, size_t b0, size_t b1) {
        std::stable_sort(v.begin() + b0, v.begin() + b1, [](const K2Item& x, const K2Item& y) { return x.tiles > y.tiles; });
    };
    auto makespan = [&](const std::vector<K2Item>& v) {
        const int grid = (int)std::min<size_t>(grid_max, v.size());
        std::vector<K2Item> sorted = v;
        sort_items(sorted, 0, sorted.size());
        std::vector<double> t((size_t)std::max(grid, 1), 0.0);
        for (size_t k = 0; k < sorted.size(); ++k) {
            // generation overlaps the streaming of the previous item, but the two compete for issue slots
            const double stream = (pair ? (sorted[k].tiles + 1) / 2 : sorted[k].tiles) * t_tile, gen = pair_f * t_slab;
            t[k % t.size()] += nslabs == 1 ? K2_EXPOSED_ONE_SLAB * gen + stream + K2_ITEM_OVERHEAD_US
                                           : std::max(gen, stream) + K2_OVERLAP_PENALTY * std::min(gen, stream) + K2_ITEM_OVERHEAD_US;
        }
        return *std::max_element(t.begin(), t.end());
    };
    const int fixed_run = tune_knob("FLORA_K2_TILES", 0, 0, 1 << 20);
    std::vector<K2Item> cand;
    double best = 1e300;
    for (int run : {1 << 20, 48, 32, 24, 16, 12, 11, 8, 6, 4, 3, 2}) {
        if (fixed_run && run != (1 << 20)) continue;
        build(fixed_run ? fixed_run : run, cand);
        const double span = makespan(cand);
        if (span < best * 0.97) {
            best = span;
            set.h_k2 = cand;
        }
    }
    // A set with few slabs per CTA (one matrix, say: 86 slabs for 74 pairs) leaves the CTAs unevenly loaded however the
    // slabs are cut into runs.  Candidate: every CTA (pair) gets an equal, contiguous share of the row-tile steps of all
    // slabs in order, cut wherever the share ends.  A share is one to three pieces of neighbouring slabs, taken largest
    // first so that the generation of the next piece's slab hides behind the streaming of the current one.  The kernels
    // hand out items round-robin, so piece j of CTA c sits at index j * G + c; a CTA with fewer pieces than the others
    // gets an empty item (no tiles: nothing is generated or streamed for it) at the end.
    bool balanced = false;
    int balanced_grid = 0;
    if (!fixed_run && W.size() <= (size_t)SEEDS_PER_LAUNCH) {
        const int per_step = pair ? 2 : 1;
        int64_t total = 0;
        for (const auto& w : W)
            if (w.rows > 0 && w.cols > 0) total += (((w.rows + 127) / 128 + per_step - 1) / per_step) * ((w.cols + bn - 1) / bn);
        const int G = (int)std::min<int64_t>(grid_max, total);
        if (G > 0) {
            std::vector<std::vector<K2Item>> share((size_t)G);
            int64_t pos = 0;
            int c = 0;
            for (size_t i = 0; i < W.size(); ++i) {
                const auto& w = W[i];
                if (w.rows == 0 || w.cols == 0) continue;
                const int64_t rtiles = (w.rows + 127) / 128, steps = (rtiles + per_step - 1) / per_step, nsl = (w.cols + bn - 1) / bn;
                for (int64_t sl = 0; sl < nsl; ++sl) {
                    int64_t s0 = 0;
                    while (s0 < steps) {
                        while (c + 1 < G && pos >= ((int64_t)(c + 1) * total + G - 1) / G) ++c;
                        const int64_t end_c = c + 1 < G ? ((int64_t)(c + 1) * total + G - 1) / G : total;
                        const int64_t take = std::min<int64_t>(steps - s0, end_c - pos);
                        K2Item it;
                        it.mat = (int)i;
                        it.col0 = (int)(sl * bn);
                        it.row0 = (int)(s0 * per_step * 128);
                        it.tiles = (int)std::min<int64_t>(take * per_step, rtiles - s0 * per_step);
                        share[(size_t)c].push_back(it);
                        pos += take;
                        s0 += take;
                    }
                }
            }
            size_t most = 0;
            double span = 0.0;
            for (auto& sh : share) {
                std::stable_sort(sh.begin(), sh.end(), [](const K2Item& x, const K2Item& y) { return x.tiles > y.tiles; });
                most = std::max(most, sh.size());
                // the slab of piece k + 1 is generated while piece k streams (the first one is charged like any item of
                // the run-based candidates, which the comparison is with)
                double t = 0.0;
                const double gen = pair_f * t_slab;
                for (size_t k = 0; k < sh.size(); ++k) {
                    const double stream = (pair ? (sh[k].tiles + 1) / 2 : sh[k].tiles) * t_tile;
                    if (nslabs == 1) {
                        t += K2_EXPOSED_ONE_SLAB * gen + stream + K2_ITEM_OVERHEAD_US;
                    } else {
                        const double next_gen = k + 1 < sh.size() ? gen : 0.0;
                        t += stream + K2_OVERLAP_PENALTY * std::min(next_gen, stream) + std::max(0.0, next_gen - stream) + K2_ITEM_OVERHEAD_US;
                    }
                }
                span = std::max(span, t);
            }
            if (span < best * 0.97) {
                best = span;
                balanced = true;
                balanced_grid = G;
                set.h_k2.assign(most * (size_t)G, K2Item());
                for (int q = 0; q < G; ++q)
                    for (size_t j = 0; j < most; ++j) {
                        K2Item& slot = set.h_k2[j * (size_t)G + (size_t)q];
                        if (j < share[(size_t)q].size()) {
                            slot = share[(size_t)q][j];
                        } else {
                            slot.mat = share[(size_t)q][0].mat;
                            slot.col0 = 0;
                            slot.row0 = 0;
                            slot.tiles = 0;
                        }
                    }
            }
        }
    }
    // launches cover at most SEEDS_PER_LAUNCH consecutive matrices; inside a launch the largest items go first
    set.k2_launch_begin.clear();
    set.k2_launch_first_mat.clear();
    size_t u0 = 0;
    if (balanced) {                     // one launch over all matrices (there are at most SEEDS_PER_LAUNCH), order as laid out
        set.k2_launch_begin.push_back(0);
        set.k2_launch_first_mat.push_back(0);
        u0 = set.h_k2.size();
    }
    while (u0 < set.h_k2.size()) {
        size_t u1 = u0;
        while (u1 < set.h_k2.size() && set.h_k2[u1].mat < set.h_k2[u0].mat + SEEDS_PER_LAUNCH) ++u1;
        set.k2_launch_begin.push_back((int)u0);
        set.k2_launch_first_mat.push_back(set.h_k2[u0].mat);
        sort_items(set.h_k2, u0, u1);
        u0 = u1;
    }
    set.k2_launch_begin.push_back((int)set.h_k2.size());
    set.k2_grid_max = balanced ? balanced_grid : grid_max;
}

inline void tc_set_free_stream(TcSet& s, cudaStream_t st)
{
    if (s.transient) {
        if (s.d_mats) cudaFreeAsync(s.d_mats, st);
        if (s.d_k1) cudaFreeAsync(s.d_k1, st);
        if (s.d_k2) cudaFreeAsync(s.d_k2, st);
        if (s.d_split) cudaFreeAsync(s.d_split, st);
        if (s.d_slots) cudaFreeAsync(s.d_slots, st);
        if (s.d_sb) cudaFreeAsync(s.d_sb, st);
    } else {
        if (s.d_mats) cudaFree(s.d_mats);
        if (s.d_k1) cudaFree(s.d_k1);
        if (s.d_k2) cudaFree(s.d_k2);
        if (s.d_split) cudaFree(s.d_split);
        if (s.d_slots) cudaFree(s.d_slots);
        if (s.d_sb) cudaFree(s.d_sb);
    }
    s.d_mats = nullptr;
    s.d_k1 = nullptr;
    s.d_k2 = nullptr;
    s.d_split = nullptr;
    s.d_slots = nullptr;
    s.d_sb = nullptr;
    s.compress_ready = s.decompress_ready = false;
}
inline void tc_set_free(TcSet& s) { tc_set_free_stream(s, nullptr); }

template <typename T>
inline flora_status upload(T** dst, const std::vector<T>& src, bool transient, cudaStream_t st)
{
    if (src.empty()) return FLORA_OK;
    const size_t bytes = src.size() * sizeof(T);
    if (!*dst) {
        cudaError_t e = transient ? scratch_alloc((void**)dst, bytes, st) : cudaMalloc((void**)dst, bytes);
        if (e != cudaSuccess) {
            cudaGetLastError();
            return FLORA_ERR_ALLOC;
        }
    }
    // pageable source: the runtime stages it before returning, so the vector may change afterwards
    if (cudaMemcpyAsync(*dst, src.data(), bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return FLORA_ERR_CUDA;
    return FLORA_OK;
}

inline flora_status tc_fill_matrices(TcSet& set, const std::vector<flora_mat>& G, const std::vector<flora_mat>& W,
                                     const std::vector<flora_mat>& S)
{
    set.h_mats.assign(S.size(), TcMatrix());
    for (size_t i = 0; i < S.size(); ++i) {
        TcMatrix& tm = set.h_mats[i];
        memset(&tm, 0, sizeof(tm));
        tm.S = (float*)S[i].data;
        tm.lds = S[i].ld;
        const flora_mat& big = !G.empty() ? G[i] : W[i];
        tm.n = (int32_t)big.rows;
        tm.m = (int32_t)big.cols;
        if (!G.empty() && G[i].rows && G[i].cols && !make_map(&tm.map_g, G[i])) return FLORA_ERR_CUDA;
        if (!W.empty() && W[i].rows && W[i].cols && !make_map(&tm.map_w, W[i])) return FLORA_ERR_CUDA;
        if (S[i].rows && S[i].cols && !make_map_f32(&tm.map_s, S[i])) return FLORA_ERR_CUDA;
    }
    return FLORA_OK;
}

// Builds the tensor-core side of a set; leaves it "not ready" (SIMT kernels are used) if any matrix is not eligible.
inline flora_status tc_set_build_on(TcSet& set, const std::vector<flora_mat>& G, const std::vector<flora_mat>& W,
                                    const std::vector<flora_mat>& S, bool transient, cudaStream_t st)
{
    set.transient = transient;
    set.count = (int)S.size();
    if (S.empty() || !encode_tiled_fn()) return FLORA_OK;
    set.r = (int)S[0].cols;
    bool g_ok = !G.empty(), w_ok = !W.empty();
    for (size_t i = 0; i < S.size(); ++i) {
        if (!G.empty() && (!tc_mat_ok(G[i]) || !tc_sketch_ok(S[i]))) g_ok = false;       // the epilogue writes S through its tensor map
        if (!W.empty() && (!tc_mat_ok(W[i]) || !tc_sketch_ok(S[i]))) w_ok = false;
    }
    if (!g_ok && !w_ok) return FLORA_OK;
    std::vector<flora_mat> none;
    flora_status rc = tc_fill_matrices(set, g_ok ? G : none, w_ok ? W : none, S);
    if (rc) return rc;
    if (w_ok) {
        plan_decompress(set, W, set.r);
        if (set.k2_bf16) {
            // scratch for the bf16 copies of the sketches: n x k_pad each, 1 KB aligned
            const int k_pad = (set.r + 63) & ~63;
            size_t total = 0;
            std::vector<size_t> offset(S.size());
            for (size_t i = 0; i < S.size(); ++i) {
                offset[i] = total;
                total += (((size_t)S[i].rows * k_pad * 2) + 1023) & ~(size_t)1023;
            }
            if (total) {
                cudaError_t e = transient ? scratch_alloc((void**)&set.d_sb, total, st) : cudaMalloc((void**)&set.d_sb, total);
                if (e != cudaSuccess) {
                    cudaGetLastError();
                    return FLORA_ERR_ALLOC;
                }
            }
            for (size_t i = 0; i < S.size(); ++i) {
                if (S[i].rows == 0) continue;
                TcMatrix& tm = set.h_mats[i];
                tm.Sb = reinterpret_cast<__nv_bfloat16*>(reinterpret_cast<uint8_t*>(set.d_sb) + offset[i]);
                flora_mat sb;
                sb.data = tm.Sb;
                sb.rows = S[i].rows;
                sb.cols = k_pad;
                sb.ld = k_pad;
                sb.dtype = FLORA_BF16;
                if (!make_map(&tm.map_sb, sb)) return FLORA_ERR_CUDA;
            }
        }
    }
    rc = upload(&set.d_mats, set.h_mats, transient, st);
    if (rc) return rc;
    if (g_ok) {
        plan_compress(set, G, set.r);
        rc = upload(&set.d_k1, set.h_k1, transient, st);
        if (rc) return rc;
        rc = upload(&set.d_split, set.split_mats, transient, st);
        if (rc) return rc;
        rc = upload(&set.d_slots, set.h_slots, transient, st);
        if (rc) return rc;
        set.compress_ready = true;
    }
    if (w_ok) {
        rc = upload(&set.d_k2, set.h_k2, transient, st);
        if (rc) return rc;
        set.decompress_ready = true;
    }
    return FLORA_OK;
}

inline flora_status tc_set_build(TcSet& set, const std::vector<flora_mat>& G, const std::vector<flora_mat>& W,
                                 const std::vector<flora_mat>& S)
{
    return tc_set_build_on(set, G, W, S, false, nullptr);
}

// New gradient pointers, same shapes: only the tensor maps change.
inline flora_status tc_set_rebind(TcSet& set, const std::vector<flora_mat>& G, cudaStream_t st)
{
    if (!set.compress_ready) return FLORA_OK;
    for (size_t i = 0; i < G.size(); ++i) {
        if (!tc_mat_ok(G[i])) return FLORA_ERR_ALIGN;
        if (G[i].rows && G[i].cols && !make_map(&set.h_mats[i].map_g, G[i])) return FLORA_ERR_CUDA;
    }
    return upload(&set.d_mats, set.h_mats, false, st);
}

// Blocks per matrix for the element-wise helper kernels (zero, scale): about four elements per thread of the
// largest sketch.
constexpr int64_t K1_SCALE_PASS_MAX_STATE_BYTES = 32ll << 20;   // sketches of a set up to this size are blended by a scaling pass (below)

inline unsigned helper_blocks(const TcSet& set)
{
    int64_t most = 1;
    for (const auto& tm : set.h_mats) most = std::max<int64_t>(most, (int64_t)tm.n * set.r);
    return (unsigned)std::min<int64_t>(1024, (most + 1023) / 1024);
}

// behind_own_kernel: the kernel before this call on the stream is one of the library's own that does not touch G and lets
// its dependents start early (the transfer's apply kernel): only the write-out of the compression waits for it.
inline flora_status tc_set_compress(TcSet& set, const uint64_t* seeds, float a, float b, cudaStream_t st,
                                    std::atomic<uint64_t>& launches, bool behind_own_kernel = false)
{
    const int r = set.r;
    const float scale = 1.0f / sqrtf((float)r);
    int late_wait = behind_own_kernel ? tune_knob("FLORA_PDL", 1, 0, 1) : 0;
    const bool pair = set.k1_pair;
    // The pair kernel blends an old sketch in (S <- b S + a G A^T) faster as a scaling pass followed by its reducing
    // write-out than by reading the old values back in its epilogue, as long as the sketches are few enough to stay in
    // L2 between the two (one 4096 x 11008 matrix at r = 256: 45.7 against 49.8 us; on 550 MB of sketches the pass
    // costs what it saves).  Every element still has one writer per launch, so the result does not depend on the schedule.
    int64_t state_bytes = 0;
    for (const auto& tm : set.h_mats) state_bytes += (int64_t)tm.n * r * 4;
    const bool scale_all = pair && b != 0.0f && b != 1.0f && state_bytes <= K1_SCALE_PASS_MAX_STATE_BYTES;
    if (scale_all || (b != 1.0f && !set.split_mats.empty())) {
        late_wait = tune_knob("FLORA_PDL", 1, 0, 1);
        // rows that receive adds (from several CTAs, or from the pair kernel's reducing write-out): scale them by b first
        const size_t total = scale_all ? (size_t)set.count : set.split_mats.size();
        for (size_t begin = 0; begin < total; begin += 65535) {
            const size_t jobs_here = std::min<size_t>(65535, total - begin);
            // few enough blocks to be resident at once: the compression kernel may only start once all have started
            dim3 grid((unsigned)std::max<size_t>(1, std::min<size_t>(helper_blocks(set), (size_t)sm_count() * 6 / jobs_here)), (unsigned)jobs_here);
            scale_sketches_kernel<<<grid, 256, 0, st>>>(set.d_mats, scale_all ? nullptr : set.d_split + begin, (int)begin, r, b);
            launches.fetch_add(1, std::memory_order_relaxed);
        }
        if (scale_all) b = 1.0f;
    }
    if (!(pair ? raise_smem_limit<compress_pair_kernel>() : raise_smem_limit<compress_tc_kernel>())) return FLORA_ERR_CUDA;
    for (size_t l = 0; l + 1 < set.k1_launch_begin.size(); ++l) {
        const int begin = set.k1_launch_begin[l], end = set.k1_launch_begin[l + 1];
        if (end == begin) continue;
        const int seed_base = set.k1_launch_first_mat[l];
        SeedTable table;
        for (int i = 0; i < SEEDS_PER_LAUNCH; ++i) table.s[i] = seed_base + i < set.count ? seeds[seed_base + i] : 0;
        // the pair kernel is persistent: one cluster per slot that has work; the other kernel runs one CTA per item
        const int n_slots = pair ? set.k1_slots_begin[l + 1] - set.k1_slots_begin[l] - 1 : 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(pair ? n_slots * set.S : end - begin));
        cfg.blockDim = dim3((unsigned)(pair ? pair_threads(set.GW) : k1_threads(set.GW)));
        cfg.dynamicSmemBytes = set.k1_smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // the kernel waits for its predecessor itself
        attr[0].val.programmaticStreamSerializationAllowed = tune_knob("FLORA_PDL", 1, 0, 1);
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = (unsigned)set.S;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = set.S > 1 ? 2 : 1;
        const TcMatrix* mats = set.d_mats;
        const K1Item* items = set.d_k1 + begin;
        const int lw = l == 0 ? late_wait : 0;
        cudaError_t e;
        if (pair) {
            const int* slot_table = set.d_slots + set.k1_slots_begin[l];
            e = cudaLaunchKernelEx(&cfg, compress_pair_kernel, mats, items, slot_table, table, seed_base, r, set.k1_n, scale, a, b, set.gstages,
                                   set.astages, set.S, set.GW, lw);
        } else {
            e = cudaLaunchKernelEx(&cfg, compress_tc_kernel, mats, items, table, seed_base, r, scale, a, b, set.T, set.gstages, set.astages, set.S,
                                   set.GW, set.P, lw);
        }
        if (e != cudaSuccess) return FLORA_ERR_CUDA;
        launches.fetch_add(1, std::memory_order_relaxed);
    }
    return cudaPeekAtLastError() == cudaSuccess ? FLORA_OK : FLORA_ERR_CUDA;
}

// Single-matrix calls go through a set of one matrix.  Planning it (work split, tensor maps, device tables) costs far
// more than the launch, and an optimizer calls with the same matrices step after step: the most recent plans are kept,
// keyed by device, operation, addresses, shapes and rank.  A plan only names addresses and shapes, so it stays valid
// when the caller's buffers are rewritten (or freed and handed out again with the same shape).  Calls that use the
// cache are serialised by its mutex; a plan is built with a synchronous upload, so any stream may use it afterwards.
struct SinglePlanKey {
    int dev, kind, r, det;
    const void *big, *sketch;
    int64_t rows, cols, ld, lds;
    bool operator==(const SinglePlanKey& o) const
    {
        return dev == o.dev && kind == o.kind && r == o.r && det == o.det && big == o.big && sketch == o.sketch && rows == o.rows &&
               cols == o.cols && ld == o.ld && lds == o.lds;
    }
};
struct SinglePlan {
    SinglePlanKey key;
    TcSet set;
};
constexpr size_t SINGLE_PLAN_CACHE = 32;
inline std::mutex& single_plan_mutex()
{
    static std::mutex m;
    return m;
}
// Call with single_plan_mutex() held.  kind 0: compression (big = G), 1: decompression (big = W).
inline TcSet* single_plan(int kind, const flora_mat& big, const flora_mat& sketch, cudaStream_t st, flora_status* rc)
{
    static std::vector<SinglePlan*> cache;                     // most recently used first
    *rc = FLORA_OK;
    SinglePlanKey key;
    memset(&key, 0, sizeof(key));
    if (cudaGetDevice(&key.dev) != cudaSuccess) {
        cudaGetLastError();
        *rc = FLORA_ERR_CUDA;
        return nullptr;
    }
    key.kind = kind;
    key.r = (int)sketch.cols;
    key.det = deterministic_flag().load();
    key.big = big.data;
    key.sketch = sketch.data;
    key.rows = big.rows;
    key.cols = big.cols;
    key.ld = big.ld;
    key.lds = sketch.ld;
    for (size_t i = 0; i < cache.size(); ++i)
        if (cache[i]->key == key) {
            SinglePlan* hit = cache[i];
            cache.erase(cache.begin() + i);
            cache.insert(cache.begin(), hit);
            return &hit->set;
        }
    SinglePlan* plan = new (std::nothrow) SinglePlan();
    if (!plan) {
        *rc = FLORA_ERR_ALLOC;
        return nullptr;
    }
    plan->key = key;
    std::vector<flora_mat> b(1, big), s(1, sketch), none;
    *rc = kind == 0 ? tc_set_build_on(plan->set, b, none, s, false, st) : tc_set_build_on(plan->set, none, b, s, false, st);
    if (*rc == FLORA_OK && cudaStreamSynchronize(st) != cudaSuccess) *rc = FLORA_ERR_CUDA;      // the tables are in place for every stream
    if (*rc != FLORA_OK) {
        tc_set_free(plan->set);
        delete plan;
        return nullptr;
    }
    cache.insert(cache.begin(), plan);
    if (cache.size() > SINGLE_PLAN_CACHE) {
        SinglePlan* old = cache.back();
        cache.pop_back();
        tc_set_free(old->set);                                 // cudaFree waits for kernels that still read the tables
        delete old;
    }
    return &plan->set;
}

inline flora_status tc_compress_single(const flora_mat* G, flora_mat* S, uint64_t seed, float a, float b, cudaStream_t st,
                                       std::atomic<uint64_t>& launches)
{
    std::lock_guard<std::mutex> lock(single_plan_mutex());
    flora_status rc;
    TcSet* set = single_plan(0, *G, *S, st, &rc);
    if (!set) return rc;
    return set->compress_ready ? tc_set_compress(*set, &seed, a, b, st, launches) : FLORA_ERR_UNSUPPORTED;
}

inline flora_status tc_set_decompress(TcSet& set, const uint64_t* seeds, float step, cudaStream_t st,
                                      std::atomic<uint64_t>& launches)
{
    const int r = set.r;
    const float scale = 1.0f / sqrtf((float)r);
    if (set.k2_bf16) {
        const int k_pad = (r + 63) & ~63;
        int max_rows = 1;
        for (const auto& tm : set.h_mats) max_rows = std::max(max_rows, tm.n);
        const int rows_per_block = 256 / (k_pad / 8);
        const unsigned bx = (unsigned)std::max<int64_t>(1, std::min<int64_t>(256, ((int64_t)max_rows + 4 * rows_per_block - 1) / (4 * rows_per_block)));   // about four rows per thread
        for (int begin = 0; begin < set.count; begin += 65535) {
            dim3 grid(bx, (unsigned)std::min(65535, set.count - begin));
            sketch_to_bf16_kernel<<<grid, 256, 0, st>>>(set.d_mats + begin, r, k_pad);
            launches.fetch_add(1, std::memory_order_relaxed);
        }
    }
    if (!(set.k2_pair ? raise_smem_limit<decompress_pair_kernel>()
                      : set.k2_bf16 ? raise_smem_limit<decompress_tc_kernel<true>>() : raise_smem_limit<decompress_tc_kernel<false>>()))
        return FLORA_ERR_CUDA;
    for (size_t l = 0; l + 1 < set.k2_launch_begin.size(); ++l) {
        const int begin = set.k2_launch_begin[l], end = set.k2_launch_begin[l + 1];
        if (end == begin) continue;
        const int seed_base = set.k2_launch_first_mat[l];
        SeedTable table;
        for (int i = 0; i < SEEDS_PER_LAUNCH; ++i) table.s[i] = seed_base + i < set.count ? seeds[seed_base + i] : 0;
        const int grid = std::min(set.k2_grid_max, end - begin);
        if (set.k2_pair) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3((unsigned)(2 * grid));                // `grid` pairs
            cfg.blockDim = dim3((unsigned)K2P_THREADS);
            cfg.dynamicSmemBytes = set.k2_smem;
            cfg.stream = st;
            cudaLaunchAttribute attr[2];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = 2;
            attr[0].val.clusterDim.y = 1;
            attr[0].val.clusterDim.z = 1;
            attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // the kernel's sketch loader waits for its predecessor itself
            attr[1].val.programmaticStreamSerializationAllowed = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 2;
            const TcMatrix* mats = set.d_mats;
            const K2Item* items = set.d_k2 + begin;
            if (cudaLaunchKernelEx(&cfg, decompress_pair_kernel, mats, items, end - begin, table, seed_base, r, scale, step, set.slots, set.cstages) !=
                cudaSuccess)
                return FLORA_ERR_CUDA;
        } else if (set.k2_bf16)
            decompress_tc_kernel<true><<<grid, 32 * (K2_FIXED_WARPS + set.k2_gw), set.k2_smem, st>>>(
                set.d_mats, set.d_k2 + begin, end - begin, table, seed_base, r, scale, step, set.bn, set.slots, set.cstages, set.k2_gw, set.k2_nslabs);
        else
            decompress_tc_kernel<false><<<grid, 32 * (K2_FIXED_WARPS + set.k2_gw), set.k2_smem, st>>>(
                set.d_mats, set.d_k2 + begin, end - begin, table, seed_base, r, scale, step, set.bn, set.slots, set.cstages, set.k2_gw, set.k2_nslabs);
        launches.fetch_add(1, std::memory_order_relaxed);
    }
    return cudaPeekAtLastError() == cudaSuccess ? FLORA_OK : FLORA_ERR_CUDA;
}

inline flora_status tc_decompress_single(flora_mat* W, const flora_mat* S, uint64_t seed, float step, cudaStream_t st,
                                         std::atomic<uint64_t>& launches)
{
    std::lock_guard<std::mutex> lock(single_plan_mutex());
    flora_status rc;
    TcSet* set = single_plan(1, *W, *S, st, &rc);
    if (!set) return rc;
    return set->decompress_ready ? tc_set_decompress(*set, &seed, step, st, launches) : FLORA_ERR_UNSUPPORTED;
}

inline bool tc_decompress_supported(const flora_mat* big, const flora_mat* sketch)
{
    return tc_mat_ok(*big) && tc_sketch_ok(*sketch) && encode_tiled_fn() != nullptr;
}

inline flora_status tc_set_zero(TcSet& set, cudaStream_t st, std::atomic<uint64_t>& launches)
{
    for (int begin = 0; begin < set.count; begin += 65535) {
        dim3 grid(helper_blocks(set), (unsigned)std::min(65535, set.count - begin));
        zero_sketches_kernel<<<grid, 256, 0, st>>>(set.d_mats + begin, set.r);
        launches.fetch_add(1, std::memory_order_relaxed);
    }
    return cudaPeekAtLastError() == cudaSuccess ? FLORA_OK : FLORA_ERR_CUDA;
}

inline bool tc_read_and_clear_error(int* word)
{
    int zero = 0;
    if (cudaMemcpyFromSymbol(word, g_flora_error_word, sizeof(int)) != cudaSuccess) return false;
    return cudaMemcpyToSymbol(g_flora_error_word, &zero, sizeof(int)) == cudaSuccess;
}

}  // namespace flora
