// Host side of the C ABI declared in include/nvfp4.h: argument checks, TMA
// descriptor set-up (cached), tile-shape choice and launches.  No allocation,
// no synchronisation (except nvfp4_device_status), nothing thrown.
#include <array>
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <unordered_map>

#include <cuda.h>
#include <cuda_runtime.h>

#include "../../include/nvfp4.h"
#include "decode.cuh"
#include "gemm.cuh"
#include "quantize.cuh"
#include "recurrence.cuh"

namespace nvfp4 {
namespace {

std::atomic<uint64_t> g_launches{0};
std::atomic<int> g_variant{0};
std::atomic<uint64_t> g_wait_limit_ns{0};          // 0 = default
constexpr uint64_t kWaitLimitNs = 2000000000ull;   // every in-kernel wait gives up after 2 s

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct DeviceInfo {
    int sm_count = 0;
    int cc_major = 0;
    bool ok = false;
};

DeviceInfo device_info() {
    static std::mutex mu;
    static std::unordered_map<int, DeviceInfo> cache;
    int dev = 0;
    DeviceInfo info;
    if (cudaGetDevice(&dev) != cudaSuccess) return info;
    std::lock_guard<std::mutex> lock(mu);
    auto it = cache.find(dev);
    if (it != cache.end()) return it->second;
    if (cudaDeviceGetAttribute(&info.sm_count, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&info.cc_major, cudaDevAttrComputeCapabilityMajor, dev) == cudaSuccess)
        info.ok = true;
    cache[dev] = info;
    return info;
}

nvfp4_status check_arch(DeviceInfo& info) {
    info = device_info();
    if (!info.ok) return NVFP4_ERR_CUDA;
    if (info.cc_major != 10) return NVFP4_ERR_ARCH;
    return NVFP4_OK;
}

nvfp4_status check_segments(const nvfp4_segment* segs, int nseg, int64_t N) {
    if (segs == nullptr) return NVFP4_ERR_NULL;
    if (nseg < 1 || nseg > NVFP4_MAX_SEGMENTS) return NVFP4_ERR_SEGMENTS;
    int64_t pos = 0;
    for (int i = 0; i < nseg; ++i) {
        if (segs[i].col_begin != pos || segs[i].col_count <= 0) return NVFP4_ERR_SEGMENTS;
        pos += segs[i].col_count;
    }
    return pos == N ? NVFP4_OK : NVFP4_ERR_SEGMENTS;
}

// ---------------------------------------------------------------- tensor maps
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

struct MapKey {
    const void* ptr;
    int64_t rows, kbytes;
    int box_rows, dev;
    bool operator==(const MapKey& o) const {
        return ptr == o.ptr && rows == o.rows && kbytes == o.kbytes && box_rows == o.box_rows && dev == o.dev;
    }
};
struct MapKeyHash {
    size_t operator()(const MapKey& k) const {
        size_t h = std::hash<const void*>()(k.ptr);
        h ^= std::hash<int64_t>()(k.rows * 1315423911ll + k.kbytes) + 0x9e3779b97f4a7c15ull + (h << 6) + (h >> 2);
        return h ^ static_cast<size_t>(k.box_rows * 31 + k.dev);
    }
};

// Encoded tensor maps by (pointer, shape).  A map costs about a microsecond of host time to encode; a
// loop over the same buffers (a model's weights, a server's ring of activation buffers) never encodes
// twice.  A caller that hands in fresh pointers for ever fills the table: when it is full the older
// half of the entries goes (by insertion stamp), not the entries that are in use.
class MapCache {
public:
    bool find(const MapKey& key, CUtensorMap* out) {
        std::lock_guard<std::mutex> lock(mu_);
        auto it = map_.find(key);
        if (it == map_.end()) return false;
        *out = it->second.map;
        return true;
    }
    void insert(const MapKey& key, const CUtensorMap& m) {
        std::lock_guard<std::mutex> lock(mu_);
        if (map_.size() >= kCapacity) {
            const uint64_t cut = stamp_ - kCapacity / 2;
            for (auto it = map_.begin(); it != map_.end();) {
                if (it->second.stamp < cut) it = map_.erase(it); else ++it;
            }
        }
        map_[key] = Entry{m, stamp_++};
    }

private:
    static constexpr size_t kCapacity = 4096;
    struct Entry {
        CUtensorMap map;
        uint64_t stamp;
    };
    std::mutex mu_;
    std::unordered_map<MapKey, Entry, MapKeyHash> map_;
    uint64_t stamp_ = kCapacity;
};

// codes [rows, K/2] bytes, tiles of box_rows x 128 bytes, 128-byte swizzle, zero fill outside
nvfp4_status codes_tensor_map(const uint8_t* d_codes, int64_t rows, int64_t K, int box_rows, CUtensorMap* out) {
    static MapCache cache;
    int dev = 0;
    cudaGetDevice(&dev);
    MapKey key{d_codes, rows, K / 2, box_rows, dev};
    if (cache.find(key, out)) return NVFP4_OK;
    EncodeTiledFn enc = encode_fn();
    if (enc == nullptr) return NVFP4_ERR_CUDA;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(K / 2), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(K / 2)};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(kBKBytes), static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(d_codes), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return NVFP4_ERR_CUDA;
    cache.insert(key, *out);
    return NVFP4_OK;
}

// scale bytes in the tensor-core layout seen as [band][k-atom][128 x u32]; a box takes four
// k-atoms of `box_bands` bands; bands and k-atoms past the tensor read as zero
nvfp4_status scales_tensor_map(const uint8_t* d_sf, int64_t rows, int64_t K, int box_bands, CUtensorMap* out) {
    static MapCache cache;
    int dev = 0;
    cudaGetDevice(&dev);
    const int64_t bands = (rows + 127) / 128, katoms = K / 64;
    MapKey key{d_sf, bands, katoms, box_bands, dev};
    if (cache.find(key, out)) return NVFP4_OK;
    EncodeTiledFn enc = encode_fn();
    if (enc == nullptr) return NVFP4_ERR_CUDA;
    const cuuint64_t dims[3] = {128, static_cast<cuuint64_t>(katoms), static_cast<cuuint64_t>(bands)};
    const cuuint64_t strides[2] = {512, static_cast<cuuint64_t>(katoms) * 512u};
    const cuuint32_t box[3] = {128, static_cast<cuuint32_t>(kStepsPerStage), static_cast<cuuint32_t>(box_bands)};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<uint8_t*>(d_sf), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return NVFP4_ERR_CUDA;
    cache.insert(key, *out);
    return NVFP4_OK;
}

// bf16 output [M, N] with row stride ldy, 32 x 64 boxes, 128-byte swizzle (TMA stores clip at M and N)
nvfp4_status output_tensor_map(void* d_y, int64_t M, int64_t N, int64_t ldy, CUtensorMap* out) {
    static MapCache cache;
    int dev = 0;
    cudaGetDevice(&dev);
    MapKey key{d_y, M, N * 4096 + (ldy % 4096), static_cast<int>(ldy / 4096), dev};
    if (cache.find(key, out)) return NVFP4_OK;
    EncodeTiledFn enc = encode_fn();
    if (enc == nullptr) return NVFP4_ERR_CUDA;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(N), static_cast<cuuint64_t>(M)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(ldy) * 2u};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(kOutPieceCols), 32u};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, d_y, dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return NVFP4_ERR_CUDA;
    cache.insert(key, *out);
    return NVFP4_OK;
}

// ---------------------------------------------------------------- GEMM launch
struct GemmMaps {
    CUtensorMap a, b, sfa, sfb, y;
};

template <int BN, int STAGES, bool PAIR, bool FULLK, int EPI = kEpiPlain>
nvfp4_status launch_gemm(const GemmMaps& tm, GemmParams& p, int sm_count, cudaStream_t stream) {
    using C = GemmCfg<BN, STAGES, PAIR>;
    static std::mutex mu;
    static std::unordered_map<int, int> max_units;      // per device: CTAs (single) or clusters (pair); 0 = unset
    int dev = 0;
    cudaGetDevice(&dev);
    p.n_tiles = (p.N + BN - 1) / BN;
    const int64_t m_units = PAIR ? (p.m_tiles + 1) / 2 : p.m_tiles;
    const int64_t tiles = m_units * p.n_tiles * (p.split_k > 0 ? p.split_k : 1);
    {
        // rows of A kept live per raster group: about 32 MB of codes and scales (a quarter of L2)
        const int64_t unit_bytes = static_cast<int64_t>(PAIR ? 256 : 128) * (p.K / 2 + p.K / 16);
        const int64_t budget = 32ll << 20;
        int64_t g = budget / (unit_bytes > 0 ? unit_bytes : 1);
        if (g < 1) g = 1;
        if (g > m_units) g = m_units;
        p.group_m = static_cast<int32_t>(g);
    }
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof(cfg));
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = PAIR ? 2 : 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // may start while the quantize kernel in front of it still runs (that kernel says when);
    // only the loads of its output wait for it
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.blockDim = dim3(kGemmThreads, 1, 1);
    cfg.dynamicSmemBytes = C::SMEM_BYTES;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    int units = 0;
    {
        std::lock_guard<std::mutex> lock(mu);
        units = max_units[dev];
        if (units == 0) {
            if (cudaFuncSetAttribute(gemm_kernel<BN, STAGES, PAIR, FULLK, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     C::SMEM_BYTES) != cudaSuccess)
                return NVFP4_ERR_CUDA;
            units = PAIR ? sm_count / 2 : sm_count;
            if (PAIR) {
                cfg.gridDim = dim3(static_cast<unsigned>(sm_count & ~1), 1, 1);
                int n = 0;
                if (cudaOccupancyMaxActiveClusters(&n, gemm_kernel<BN, STAGES, PAIR, FULLK, EPI>, &cfg) == cudaSuccess && n >= 1) {
                    if (n < units) units = n;
                } else {
                    cudaGetLastError();
                }
            }
            max_units[dev] = units;
        }
    }
    const int64_t use = tiles < units ? tiles : units;
    cfg.gridDim = dim3(static_cast<unsigned>((PAIR ? 2 : 1) * use), 1, 1);
    cudaError_t e = cudaLaunchKernelEx(&cfg, gemm_kernel<BN, STAGES, PAIR, FULLK, EPI>, tm.a, tm.b, tm.sfa, tm.sfb, tm.y, p);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return e == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

// Decode-sized M with fewer 128 x 128 tiles than SMs: clusters of `S` CTAs share a tile along K and
// meet in the shared memory of the cluster's first CTA (gemm.cuh, kEpiClusterSplit*).  Two builds of
// the kernel divide shared memory differently: five stages and two landing slots (a slot holds one
// CTA's partial sums of one 32-row quarter), or four stages and five slots.
template <int EPI>
struct ClusterSplit {
    static constexpr int BN = 128;
    static constexpr int STAGES = EPI == kEpiClusterSplitFew ? 5 : 4;
    static constexpr int SLOTS = cluster_split_slots(EPI);
    static constexpr int kMaxS = 1 + SLOTS;
    using C = GemmCfg<BN, STAGES, false, SLOTS * kClusterSplitSlotBytes>;

    static cudaLaunchConfig_t config(cudaLaunchAttribute (&attr)[2], cudaStream_t stream) {
        cudaLaunchConfig_t cfg;
        std::memset(&cfg, 0, sizeof(cfg));
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 1;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.blockDim = dim3(kGemmThreads, 1, 1);
        cfg.dynamicSmemBytes = C::SMEM_BYTES;
        cfg.stream = stream;
        cfg.attrs = attr;
        cfg.numAttrs = 2;
        return cfg;
    }

    // The largest S (2..kMaxS) for which every tile's cluster is resident at once, every CTA gets at
    // least two K tiles and the partial sums fit the slots; 1 if there is none but `allow_single`
    // (the caller wants this kernel for its in-kernel activation quantization); 0 otherwise, or -1
    // after a CUDA error.  Sets p.k_per_split for the S it returns.
    static int plan(GemmParams& p, int sm_count, bool allow_single) {
        auto kernel = gemm_kernel<BN, STAGES, false, true, EPI>;
        static std::mutex mu;
        static std::unordered_map<int, std::array<int, kMaxS + 1>> resident;    // per device and S (0 = unset)
        int dev = 0;
        cudaGetDevice(&dev);
        const int64_t tiles = static_cast<int64_t>(p.m_tiles) * ((p.N + BN - 1) / BN);
        if (tiles <= 0 || p.m_tiles != 1) return 0;
        if (tiles * 2 > sm_count && !allow_single) return 0;
        int S = static_cast<int>(sm_count / tiles);
        const int live_q = ((p.M < kBM ? p.M : kBM) + 31) / 32;      // 32-row quarters of the tile that hold rows of Y
        if (S > 1 + SLOTS / live_q) S = 1 + SLOTS / live_q;
        if (S > p.k_tiles / 2) S = p.k_tiles / 2;
        {
            std::lock_guard<std::mutex> lock(mu);
            auto& r = resident[dev];
            if (r[0] == 0) {
                if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES) != cudaSuccess)
                    return -1;
                r[0] = 1;
            }
            for (; S >= 2; --S) {
                if (r[S] == 0) {
                    cudaLaunchAttribute attr[2];
                    cudaLaunchConfig_t cfg = config(attr, nullptr);
                    attr[0].val.clusterDim.x = static_cast<unsigned>(S);
                    cfg.gridDim = dim3(static_cast<unsigned>(sm_count / S * S), 1, 1);
                    int n = 0;
                    if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
                    r[S] = n > 0 ? n : -1;
                }
                if (r[S] >= tiles) break;
            }
        }
        if (S < 1) S = 1;
        p.k_per_split = (p.k_tiles + S - 1) / S;
        while (S > 1 && static_cast<int64_t>(S - 1) * p.k_per_split >= p.k_tiles) {          // every CTA has work
            --S;
            p.k_per_split = (p.k_tiles + S - 1) / S;
        }
        if (S < 2 && !allow_single) return 0;
        return S;
    }

    static nvfp4_status launch(const GemmMaps& tm, GemmParams& p, int S, cudaStream_t stream) {
        auto kernel = gemm_kernel<BN, STAGES, false, true, EPI>;
        p.n_tiles = (p.N + BN - 1) / BN;
        p.group_m = p.m_tiles;
        p.k_per_split = (p.k_tiles + S - 1) / S;
        p.split_k = S;
        p.partial = nullptr;
        p.counters = nullptr;
        cudaLaunchAttribute attr[2];
        cudaLaunchConfig_t cfg = config(attr, stream);
        attr[0].val.clusterDim.x = static_cast<unsigned>(S);
        cfg.gridDim = dim3(static_cast<unsigned>(static_cast<int64_t>(p.n_tiles) * S), 1, 1);
        cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, tm.a, tm.b, tm.sfa, tm.sfb, tm.y, p);
        g_launches.fetch_add(1, std::memory_order_relaxed);
        return e == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
    }
};

// Launches the cluster-split kernel if the shape takes one: the build with more stages when it
// splits K as many ways as the other would.  NVFP4_ERR_SHAPE, with nothing launched, if neither applies.
nvfp4_status launch_gemm_cluster_split(const GemmMaps& tm, GemmParams& p, int sm_count, cudaStream_t stream,
                                       bool allow_single) {
    GemmParams few = p, many = p;
    const int s_few = ClusterSplit<kEpiClusterSplitFew>::plan(few, sm_count, allow_single);
    const int s_many = ClusterSplit<kEpiClusterSplit>::plan(many, sm_count, allow_single);
    if (s_few < 0 || s_many < 0) return NVFP4_ERR_CUDA;
    if (s_few >= 1 && s_few >= s_many) return ClusterSplit<kEpiClusterSplitFew>::launch(tm, p, s_few, stream);
    if (s_many >= 1) return ClusterSplit<kEpiClusterSplit>::launch(tm, p, s_many, stream);
    return NVFP4_ERR_SHAPE;
}

// 128 / 256: one CTA per 128 x BN tile; 2: CTA pair per 256 x 256 tile
int choose_variant(int64_t M, int64_t N) {
    const int forced = g_variant.load(std::memory_order_relaxed);
    if (forced != 0) return forced;
    if (M > 128 && N >= 256) return 2;
    if (M <= 128) return 128;                 // decode-sized: more, smaller tiles (and split-K)
    return N >= 256 ? 256 : 128;
}

template <bool MMA, int MODE>
nvfp4_status launch_quantize(const uint16_t* x, int64_t M, int64_t K, int64_t ld, const float* d_g,
                             const SegTable& segs, uint8_t* d_codes, uint8_t* d_sf, int64_t chunks, int64_t per_unit,
                             int64_t units_per_row, int64_t units, int sm_count, cudaStream_t stream,
                             const uint16_t* aux, float eps, uint16_t* h_out) {
    constexpr int kUnroll = 2;
    // persistent grid: exactly what is resident at once, so that no partial second wave forms
    static std::atomic<int> per_sm_cache{0};
    int per_sm = per_sm_cache.load(std::memory_order_relaxed);
    if (per_sm == 0) {
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, quantize_kernel<MMA, kUnroll, MODE>, 256, 0) !=
                cudaSuccess || per_sm < 1) {
            cudaGetLastError();
            per_sm = 4;
        }
        per_sm_cache.store(per_sm, std::memory_order_relaxed);
    }
    int64_t blocks = (units + 7) / 8;
    const int64_t max_blocks = static_cast<int64_t>(sm_count) * per_sm;
    if (blocks > max_blocks) blocks = max_blocks;
    if (blocks < 1) blocks = 1;
    // launched so that it may start while the kernel in front of it drains (if that kernel says so, as
    // this one does for its own dependents); its first global read waits for that kernel's completion
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof(cfg));
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3(static_cast<unsigned>(blocks), 1, 1);
    cfg.blockDim = dim3(256, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t le = cudaLaunchKernelEx(&cfg, quantize_kernel<MMA, kUnroll, MODE>, x, static_cast<int32_t>(M),
                                              static_cast<int32_t>(K), ld, d_g, segs, aux, eps, d_codes, d_sf, h_out,
                                              static_cast<int32_t>(chunks), static_cast<int32_t>(per_unit),
                                              static_cast<int32_t>(units_per_row), static_cast<int32_t>(units));
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return le == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

// RMSNorm -> quantize with the row held in registers by W warps of NCH chunks each
template <bool MMA, int W, int NCH>
nvfp4_status launch_rmsnorm(const uint16_t* x, int64_t M, int64_t rows_total, int64_t K, int64_t ld, const float* d_g,
                            const uint16_t* gain, float eps, uint8_t* d_codes, uint8_t* d_sf, uint16_t* y_out,
                            int64_t chunks, int sm_count, cudaStream_t stream) {
    static std::atomic<int> per_sm_cache{0};
    int per_sm = per_sm_cache.load(std::memory_order_relaxed);
    if (per_sm == 0) {
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, rmsnorm_quantize_kernel<MMA, W, NCH>, 256, 0) != cudaSuccess ||
            per_sm < 1) {
            cudaGetLastError();
            per_sm = 2;
        }
        per_sm_cache.store(per_sm, std::memory_order_relaxed);
    }
    constexpr int kGroups = 8 / W;
    int64_t blocks = (rows_total + kGroups - 1) / kGroups;
    const int64_t max_blocks = static_cast<int64_t>(sm_count) * per_sm;
    if (blocks > max_blocks) blocks = max_blocks;
    if (blocks < 1) blocks = 1;
    rmsnorm_quantize_kernel<MMA, W, NCH><<<static_cast<int>(blocks), 256, 0, stream>>>(
        x, static_cast<int32_t>(M), static_cast<int32_t>(rows_total), static_cast<int32_t>(K), ld, d_g, gain, eps,
        d_codes, d_sf, y_out, static_cast<int32_t>(chunks), static_cast<int32_t>((chunks + W - 1) / W));
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

nvfp4_status quantize_impl(const void* d_x, int64_t M, int64_t K, int64_t ld, const float* d_g,
                           const SegTable& segs, uint8_t* d_codes, uint8_t* d_sf, nvfp4_sf_layout layout,
                           const DeviceInfo& info, cudaStream_t stream, int mode = kQuantPlain,
                           const uint16_t* aux = nullptr, float eps = 0.0f, uint16_t* h_out = nullptr) {
    const int64_t chunks = (K + 511) / 512;              // 512 elements = one block per lane
    if (M >= (1ll << 31) || K >= (1ll << 31)) return NVFP4_ERR_SHAPE;
    if (mode == kQuantRmsnorm && chunks <= 8 * kRmsChunksMax) {
        const uint16_t* xr = reinterpret_cast<const uint16_t*>(d_x);
        const int64_t rows_all = (layout == NVFP4_SF_MMA) ? (M + 127) / 128 * 128 : M;
        const bool mma_l = layout == NVFP4_SF_MMA;
        // fewest warps per row that keep a warp's share at kRmsChunksMax chunks
        int w = 1;
        while (w < 8 && (chunks + w - 1) / w > kRmsChunksMax) w *= 2;
#define NVFP4_LAUNCH_R(MMA_, W_, NCH_) \
    launch_rmsnorm<MMA_, W_, NCH_>(xr, M, rows_all, K, ld, d_g, aux, eps, d_codes, d_sf, h_out, chunks, info.sm_count, stream)
        switch (w) {
            case 1: return mma_l ? NVFP4_LAUNCH_R(true, 1, 5) : NVFP4_LAUNCH_R(false, 1, 5);
            case 2: return mma_l ? NVFP4_LAUNCH_R(true, 2, 5) : NVFP4_LAUNCH_R(false, 2, 5);
            case 4: return mma_l ? NVFP4_LAUNCH_R(true, 4, 5) : NVFP4_LAUNCH_R(false, 4, 5);
            default: return mma_l ? NVFP4_LAUNCH_R(true, 8, 5) : NVFP4_LAUNCH_R(false, 8, 5);
        }
#undef NVFP4_LAUNCH_R
    }
    // a unit = up to `per_unit` consecutive chunks of one row, handled by one warp
    constexpr int kUnroll = 2;      // matches launch_quantize
    const int64_t resident_warps = static_cast<int64_t>(info.sm_count) * 40;   // 5 blocks of 8 warps per SM
    int64_t per_unit = (M * chunks > 2 * resident_warps) ? kUnroll : 1;
    if (mode == kQuantRmsnorm) per_unit = chunks;           // the row reduction needs the whole row in one warp
    const int64_t units_per_row = (chunks + per_unit - 1) / per_unit;
    // in the tensor-core layout the kernel also zero-fills the scales of the rows that pad the last band
    const int64_t rows_total = (layout == NVFP4_SF_MMA) ? (M + 127) / 128 * 128 : M;
    const int64_t units = rows_total * units_per_row;
    if (units >= (1ll << 31)) return NVFP4_ERR_SHAPE;
    const uint16_t* x = reinterpret_cast<const uint16_t*>(d_x);
    const bool mma = layout == NVFP4_SF_MMA;
#define NVFP4_LAUNCH_Q(MMA_, MODE_)                                                                          \
    launch_quantize<MMA_, MODE_>(x, M, K, ld, d_g, segs, d_codes, d_sf, chunks, per_unit, units_per_row, units, \
                                 info.sm_count, stream, aux, eps, h_out)
    if (mode == kQuantSwiglu) return mma ? NVFP4_LAUNCH_Q(true, kQuantSwiglu) : NVFP4_LAUNCH_Q(false, kQuantSwiglu);
    if (mode == kQuantRmsnorm) return mma ? NVFP4_LAUNCH_Q(true, kQuantRmsnorm) : NVFP4_LAUNCH_Q(false, kQuantRmsnorm);
    return mma ? NVFP4_LAUNCH_Q(true, kQuantPlain) : NVFP4_LAUNCH_Q(false, kQuantPlain);
#undef NVFP4_LAUNCH_Q
}

nvfp4_status check_quantize_args(const void* d_x, int64_t rows, int64_t K, int64_t ld, const float* d_g,
                                 const uint8_t* d_codes, const uint8_t* d_sf, nvfp4_sf_layout layout) {
    if (d_x == nullptr || d_g == nullptr || d_codes == nullptr || d_sf == nullptr) return NVFP4_ERR_NULL;
    if (rows < 0 || K <= 0 || (K % 16) != 0 || ld < K) return NVFP4_ERR_SHAPE;
    if (layout != NVFP4_SF_LINEAR && layout != NVFP4_SF_MMA) return NVFP4_ERR_LAYOUT;
    if ((reinterpret_cast<uintptr_t>(d_x) & 31u) != 0 || (ld % 16) != 0 || !aligned16(d_codes)) return NVFP4_ERR_ALIGN;
    if (layout == NVFP4_SF_MMA && (reinterpret_cast<uintptr_t>(d_sf) & 3u) != 0) return NVFP4_ERR_ALIGN;
    return NVFP4_OK;
}

constexpr size_t kStatusBytes = 256;
constexpr size_t kSplitReserve = NVFP4_SPLIT_RESERVE_BYTES;

// Split-K area of a workspace: counters, then fp32 partial sums.  It always starts directly behind
// the status block, whatever the problem size, and never reaches past the reserve, so that nothing
// else the library keeps in a workspace (the quantized activations of nvfp4_linear_bf16 live behind
// the reserve) can ever land on it: it stays zero between calls by construction.
struct SplitArea {
    size_t counters_bytes = 0, partial_bytes = 0;
    int64_t ldp = 0;
    size_t total() const { return counters_bytes + partial_bytes; }
};
SplitArea split_area(int64_t M, int64_t N) {
    SplitArea a;
    if (M <= 0 || N <= 0 || M > 256) return a;                 // split-K serves decode-sized batches only
    const int64_t m_tiles = (M + 127) / 128, n_tiles = (N + 127) / 128;
    a.counters_bytes = (static_cast<size_t>(m_tiles * n_tiles * 4) * sizeof(uint32_t) + 255) & ~static_cast<size_t>(255);
    a.ldp = n_tiles * 128;
    a.partial_bytes = static_cast<size_t>(m_tiles * 128) * static_cast<size_t>(a.ldp) * sizeof(float);
    if (a.total() > kSplitReserve) return SplitArea();         // too large for the reserve: no split-K
    return a;
}

}  // namespace
}  // namespace nvfp4

using namespace nvfp4;

extern "C" {

size_t nvfp4_sf_bytes(int64_t rows, int64_t K, nvfp4_sf_layout layout) {
    if (rows < 0 || K < 0 || (K % 16) != 0) return 0;
    const int64_t kb = K / 16;
    if (layout == NVFP4_SF_LINEAR) return static_cast<size_t>(rows * kb);
    return static_cast<size_t>(((rows + 127) / 128) * ((kb + 3) / 4) * 512);
}

nvfp4_status nvfp4_calibrate(const void* d_x, int64_t rows, int64_t cols, int64_t ld, float* d_g, float* d_amax,
                             void* stream) {
    if (d_g == nullptr || (d_x == nullptr && rows * cols != 0)) return NVFP4_ERR_NULL;
    if (rows < 0 || cols < 0 || ld < cols) return NVFP4_ERR_SHAPE;
    DeviceInfo info;
    nvfp4_status st = check_arch(info);
    if (st != NVFP4_OK) return st;
    cudaStream_t s = as_stream(stream);
    if (cudaMemsetAsync(d_g, 0, sizeof(float), s) != cudaSuccess) return NVFP4_ERR_CUDA;
    if (rows * cols > 0) {
        const uint16_t* x = reinterpret_cast<const uint16_t*>(d_x);
        const int64_t chunks = (cols + 255) / 256;
        if (aligned16(d_x) && (ld % 8) == 0 && rows * chunks < (1ll << 31) && cols < (1ll << 31)) {
            const int32_t total = static_cast<int32_t>(rows * chunks);
            int64_t blocks = (total + 31) / 32;        // about four items per warp
            const int64_t max_blocks = static_cast<int64_t>(info.sm_count) * 8;
            if (blocks > max_blocks) blocks = max_blocks;
            if (blocks < 1) blocks = 1;
            amax_kernel<<<static_cast<int>(blocks), 256, 0, s>>>(x, static_cast<int32_t>(rows),
                                                                 static_cast<int32_t>(cols), ld,
                                                                 static_cast<int32_t>(chunks), total,
                                                                 reinterpret_cast<uint32_t*>(d_g));
        } else {
            amax_scalar_kernel<<<info.sm_count * 4, 256, 0, s>>>(x, rows, cols, ld, reinterpret_cast<uint32_t*>(d_g));
        }
        g_launches.fetch_add(1, std::memory_order_relaxed);
        if (cudaGetLastError() != cudaSuccess) return NVFP4_ERR_CUDA;
    }
    finalize_scale_kernel<<<1, 1, 0, s>>>(d_g, d_amax);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

nvfp4_status nvfp4_quantize_act(const void* d_x, int64_t M, int64_t K, int64_t ld, const float* d_g,
                                uint8_t* d_codes, uint8_t* d_sf, nvfp4_sf_layout layout, void* stream) {
    nvfp4_status st = check_quantize_args(d_x, M, K, ld, d_g, d_codes, d_sf, layout);
    if (st != NVFP4_OK) return st;
    if (M == 0) return NVFP4_OK;
    DeviceInfo info;
    st = check_arch(info);
    if (st != NVFP4_OK) return st;
    SegTable segs;
    std::memset(&segs, 0, sizeof(segs));
    return quantize_impl(d_x, M, K, ld, d_g, segs, d_codes, d_sf, layout, info, as_stream(stream));
}

nvfp4_status nvfp4_quantize_weight(const void* d_w, int64_t N, int64_t K, int64_t ld, const nvfp4_segment* segs,
                                   int nseg, float* d_g_seg, int calibrate_segments, uint8_t* d_codes,
                                   uint8_t* d_sf, nvfp4_sf_layout layout, void* stream) {
    nvfp4_status st = check_quantize_args(d_w, N, K, ld, d_g_seg, d_codes, d_sf, layout);
    if (st != NVFP4_OK) return st;
    st = check_segments(segs, nseg, N);
    if (st != NVFP4_OK) return st;
    if (N >= (1ll << 31)) return NVFP4_ERR_SHAPE;
    DeviceInfo info;
    st = check_arch(info);
    if (st != NVFP4_OK) return st;
    SegTable table;
    std::memset(&table, 0, sizeof(table));
    table.nseg = nseg;
    for (int i = 0; i < nseg; ++i) table.row_end[i] = static_cast<int32_t>(segs[i].col_begin + segs[i].col_count);
    if (calibrate_segments != 0) {
        const uint16_t* w = reinterpret_cast<const uint16_t*>(d_w);
        for (int i = 0; i < nseg; ++i) {
            st = nvfp4_calibrate(w + segs[i].col_begin * ld, segs[i].col_count, K, ld, d_g_seg + i, nullptr, stream);
            if (st != NVFP4_OK) return st;
        }
    }
    return quantize_impl(d_w, N, K, ld, d_g_seg, table, d_codes, d_sf, layout, info, as_stream(stream));
}

nvfp4_status nvfp4_quantize_weight_gate_up(const void* d_w, int64_t inner, int64_t K, int64_t ld, float* d_g_gate_up,
                                           int calibrate_segments, uint8_t* d_codes, uint8_t* d_sf, void* stream) {
    const int64_t N = 2 * inner;
    nvfp4_status st = check_quantize_args(d_w, N, K, ld, d_g_gate_up, d_codes, d_sf, NVFP4_SF_MMA);
    if (st != NVFP4_OK) return st;
    if (inner <= 0 || (inner % 16) != 0 || N >= (1ll << 31)) return NVFP4_ERR_SHAPE;
    DeviceInfo info;
    st = check_arch(info);
    if (st != NVFP4_OK) return st;
    SegTable table;
    std::memset(&table, 0, sizeof(table));
    table.nseg = 2;
    table.row_end[0] = static_cast<int32_t>(inner);
    table.row_end[1] = static_cast<int32_t>(N);
    table.il_inner = static_cast<int32_t>(inner);
    if (calibrate_segments != 0) {
        const uint16_t* w = reinterpret_cast<const uint16_t*>(d_w);
        for (int i = 0; i < 2; ++i) {
            st = nvfp4_calibrate(w + i * inner * ld, inner, K, ld, d_g_gate_up + i, nullptr, stream);
            if (st != NVFP4_OK) return st;
        }
    }
    return quantize_impl(d_w, N, K, ld, d_g_gate_up, table, d_codes, d_sf, NVFP4_SF_MMA, info, as_stream(stream));
}

nvfp4_status nvfp4_swiglu_quantize(const void* d_gate_up, int64_t M, int64_t inner, int64_t ld, const float* d_g,
                                   uint8_t* d_codes, uint8_t* d_sf, nvfp4_sf_layout layout, void* d_h, void* stream) {
    nvfp4_status st = check_quantize_args(d_gate_up, M, inner, ld, d_g, d_codes, d_sf, layout);
    if (st != NVFP4_OK) return st;
    if (ld < 2 * inner) return NVFP4_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(d_h) & 31u) != 0) return NVFP4_ERR_ALIGN;
    if (M == 0) return NVFP4_OK;
    DeviceInfo info;
    st = check_arch(info);
    if (st != NVFP4_OK) return st;
    SegTable segs;
    std::memset(&segs, 0, sizeof(segs));
    return quantize_impl(d_gate_up, M, inner, ld, d_g, segs, d_codes, d_sf, layout, info, as_stream(stream), kQuantSwiglu,
                         nullptr, 0.0f, reinterpret_cast<uint16_t*>(d_h));
}

nvfp4_status nvfp4_harmonize_scales(const uint8_t* d_sf_in, int64_t N, int64_t K, nvfp4_sf_layout layout,
                                    const nvfp4_segment* segs, const float* d_g_seg, int nseg, uint8_t* d_sf_out,
                                    float* d_g_shared, void* stream) {
    if (d_sf_in == nullptr || d_sf_out == nullptr || d_g_seg == nullptr || d_g_shared == nullptr) return NVFP4_ERR_NULL;
    if (N < 0 || K <= 0 || (K % 16) != 0 || N >= (1ll << 31) || K >= (1ll << 31)) return NVFP4_ERR_SHAPE;
    if (layout != NVFP4_SF_LINEAR && layout != NVFP4_SF_MMA) return NVFP4_ERR_LAYOUT;
    nvfp4_status st = check_segments(segs, nseg, N);
    if (st != NVFP4_OK) return st;
    if (layout == NVFP4_SF_MMA && (((reinterpret_cast<uintptr_t>(d_sf_in) | reinterpret_cast<uintptr_t>(d_sf_out)) & 3u) != 0))
        return NVFP4_ERR_ALIGN;
    DeviceInfo info;
    st = check_arch(info);
    if (st != NVFP4_OK) return st;
    cudaStream_t s = as_stream(stream);
    if (layout == NVFP4_SF_MMA && d_sf_out != d_sf_in) {
        // padding rows and blocks of the output read as zero scales
        if (cudaMemsetAsync(d_sf_out, 0, nvfp4_sf_bytes(N, K, layout), s) != cudaSuccess) return NVFP4_ERR_CUDA;
    }
    SegTable table;
    std::memset(&table, 0, sizeof(table));
    table.nseg = nseg;
    for (int i = 0; i < nseg; ++i) table.row_end[i] = static_cast<int32_t>(segs[i].col_begin + segs[i].col_count);
    const int64_t words = N * ((K / 16 + 3) / 4);
    int64_t blocks = (words + 255) / 256;
    if (blocks > info.sm_count * 8) blocks = info.sm_count * 8;
    if (blocks < 1) blocks = 1;
    harmonize_kernel<<<static_cast<int>(blocks), 256, 0, s>>>(d_sf_in, d_sf_out, static_cast<int32_t>(N),
                                                             static_cast<int32_t>(K / 16), layout == NVFP4_SF_MMA ? 1 : 0,
                                                             d_g_seg, table, d_g_shared);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

nvfp4_status nvfp4_rmsnorm_quantize(const void* d_x, int64_t M, int64_t K, int64_t ld, const void* d_weight, float eps,
                                    const float* d_g, uint8_t* d_codes, uint8_t* d_sf, nvfp4_sf_layout layout,
                                    void* d_y, void* stream) {
    nvfp4_status st = check_quantize_args(d_x, M, K, ld, d_g, d_codes, d_sf, layout);
    if (st != NVFP4_OK) return st;
    if (d_weight == nullptr) return NVFP4_ERR_NULL;
    if (((reinterpret_cast<uintptr_t>(d_weight) | reinterpret_cast<uintptr_t>(d_y)) & 31u) != 0) return NVFP4_ERR_ALIGN;
    if (!(eps >= 0.0f)) return NVFP4_ERR_SHAPE;
    if (M == 0) return NVFP4_OK;
    DeviceInfo info;
    st = check_arch(info);
    if (st != NVFP4_OK) return st;
    SegTable segs;
    std::memset(&segs, 0, sizeof(segs));
    return quantize_impl(d_x, M, K, ld, d_g, segs, d_codes, d_sf, layout, info, as_stream(stream), kQuantRmsnorm,
                         reinterpret_cast<const uint16_t*>(d_weight), eps, reinterpret_cast<uint16_t*>(d_y));
}

nvfp4_status nvfp4_tensor_stats(const void* d_x, int64_t rows, int64_t cols, int64_t ld, const float* d_g,
                                double* d_out, void* stream) {
    if (d_x == nullptr || d_g == nullptr || d_out == nullptr) return NVFP4_ERR_NULL;
    if (rows < 0 || cols <= 0 || (cols % 16) != 0 || ld < cols || cols >= (1ll << 31) || rows >= (1ll << 31))
        return NVFP4_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(d_x) & 31u) != 0 || (ld % 16) != 0 || (reinterpret_cast<uintptr_t>(d_out) & 7u) != 0)
        return NVFP4_ERR_ALIGN;
    DeviceInfo info;
    nvfp4_status st = check_arch(info);
    if (st != NVFP4_OK) return st;
    cudaStream_t s = as_stream(stream);
    // out[0..5] accumulators, out[6] (first 4 bytes) the running maximum as float bits
    if (cudaMemsetAsync(d_out, 0, 7 * sizeof(double), s) != cudaSuccess) return NVFP4_ERR_CUDA;
    const int64_t blocks16 = rows * (cols / 16);
    if (blocks16 > 0) {
        int64_t grid = (blocks16 + 255) / 256;
        if (grid > info.sm_count * 8) grid = info.sm_count * 8;
        stats_kernel<<<static_cast<int>(grid), 256, 0, s>>>(reinterpret_cast<const uint16_t*>(d_x),
                                                            static_cast<int32_t>(rows), static_cast<int32_t>(cols), ld,
                                                            d_g, d_out, reinterpret_cast<uint32_t*>(d_out + 6));
        g_launches.fetch_add(1, std::memory_order_relaxed);
        if (cudaGetLastError() != cudaSuccess) return NVFP4_ERR_CUDA;
    }
    stats_finalize_kernel<<<1, 1, 0, s>>>(d_out, reinterpret_cast<const uint32_t*>(d_out + 6),
                                          static_cast<double>(blocks16));
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

size_t nvfp4_linear_workspace_bytes(int64_t M, int64_t N, int64_t K, int nseg) {
    (void)K; (void)nseg;
    return kStatusBytes + split_area(M, N).total();
}

nvfp4_status nvfp4_workspace_reset(void* d_workspace, size_t workspace_bytes, void* stream) {
    if (d_workspace == nullptr) return NVFP4_ERR_NULL;
    if (workspace_bytes < kStatusBytes) return NVFP4_ERR_WORKSPACE;
    return cudaMemsetAsync(d_workspace, 0, kStatusBytes, as_stream(stream)) == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

}  // extern "C"

namespace {
// `d_split` / `split_bytes`: zero-filled split-K area (may be null: then no split-K)
nvfp4_status linear_impl(const uint8_t* d_a_codes, const uint8_t* d_a_sf, const float* d_g_a, int64_t M,
                         int64_t K, const uint8_t* d_w_codes, const uint8_t* d_w_sf, int64_t N,
                         const nvfp4_segment* segs, const float* d_g_seg, int nseg, void* d_y, int64_t ldy,
                         uint32_t flags, void* d_workspace, size_t workspace_bytes, void* d_split, size_t split_bytes,
                         void* stream, int64_t a_rows_alloc = 0, const GemmParams* fused = nullptr,
                         const uint16_t* aq_x = nullptr, int64_t aq_ldx = 0) {
    // aq_x: bf16 activations that the kernel quantizes itself (the caller has checked that the shape
    // takes the cluster-split variant); then there are no A codes or scales
    if (((d_a_codes == nullptr || d_a_sf == nullptr) && aq_x == nullptr) || d_g_a == nullptr || d_w_codes == nullptr ||
        d_w_sf == nullptr || d_g_seg == nullptr || (d_y == nullptr && fused == nullptr))
        return NVFP4_ERR_NULL;
    if (M < 0 || N < 0 || K <= 0 || (K % 64) != 0 || ldy < N) return NVFP4_ERR_SHAPE;
    if (M >= (1ll << 31) - 256 || N >= (1ll << 31) - 256 || K >= (1ll << 31)) return NVFP4_ERR_SHAPE;
    nvfp4_status st = check_segments(segs, nseg, N);
    if (N == 0 && segs != nullptr) st = NVFP4_OK;
    if (st != NVFP4_OK) return st;
    if ((aq_x == nullptr && (!aligned16(d_a_codes) || !aligned16(d_a_sf))) || !aligned16(d_w_codes) || !aligned16(d_w_sf))
        return NVFP4_ERR_ALIGN;
    if (d_workspace == nullptr || workspace_bytes < kStatusBytes) return NVFP4_ERR_WORKSPACE;
    if (!aligned16(d_workspace)) return NVFP4_ERR_ALIGN;
    if ((flags & ~(NVFP4_OUT_F32 | NVFP4_WS_ZEROED | NVFP4_W_RESIDENT)) != 0u) return NVFP4_ERR_SHAPE;
    if (M == 0 || N == 0) return NVFP4_OK;
    DeviceInfo info;
    st = check_arch(info);
    if (st != NVFP4_OK) return st;

    int bn = choose_variant(M, N);
    if (fused != nullptr && bn == 128) bn = 256;          // the fused epilogue pairs 32 columns: 256-wide tiles only
    const int tile_n = bn == 128 ? 128 : 256;
    GemmMaps tm;
    std::memset(&tm, 0, sizeof(tm));
    // rows the code buffer really has (>= M): with whole 128-row boxes in bounds TMA takes no
    // out-of-bounds path, which is measurably slower; rows past M hold zero scales and are never stored
    // Decode-sized M: the A box holds only the rows that exist (rounded up to the 8-row swizzle period).
    // Every CTA reads the same A from L2 at the same moment; a full 128-row box there costs as much
    // load-path time per stage as the W tile it is multiplied with.
    const int a_box_rows = M < kBM ? static_cast<int>((M + 7) / 8 * 8) : kBM;
    if (aq_x == nullptr) st = codes_tensor_map(d_a_codes, a_rows_alloc > M ? a_rows_alloc : M, K, a_box_rows, &tm.a);
    if (st != NVFP4_OK) return st;
    st = codes_tensor_map(d_w_codes, N, K, bn == 2 ? 128 : tile_n, &tm.b);
    if (st != NVFP4_OK) return st;
    if (aq_x == nullptr) st = scales_tensor_map(d_a_sf, M, K, 1, &tm.sfa);
    if (st != NVFP4_OK) return st;
    st = scales_tensor_map(d_w_sf, N, K, tile_n / 128, &tm.sfb);
    if (st != NVFP4_OK) return st;

    GemmParams p;
    std::memset(&p, 0, sizeof(p));
    if (fused == nullptr && (flags & NVFP4_OUT_F32) == 0u && aligned16(d_y) && (ldy % 8) == 0) {
        st = output_tensor_map(d_y, M, N, ldy, &tm.y);
        if (st != NVFP4_OK) return st;
        p.tma_store = 1u;
    }
    p.g_a = d_g_a;
    p.g_seg = d_g_seg;
    p.y = d_y;
    p.ldy = ldy;
    p.status = reinterpret_cast<uint32_t*>(d_workspace);
    p.M = static_cast<int32_t>(M);
    p.N = static_cast<int32_t>(N);
    p.K = static_cast<int32_t>(K);
    p.m_tiles = static_cast<int32_t>((M + kBM - 1) / kBM);
    p.k_tiles = static_cast<int32_t>((K + 255) / 256);
    p.katoms = static_cast<int32_t>(K / 64);
    p.a_box_bytes = a_box_rows * kBKBytes;
    p.split_k = 1;
    p.k_per_split = p.k_tiles;
    if (bn == 128 && (flags & NVFP4_WS_ZEROED) != 0u && d_split != nullptr && (K % 256) == 0) {
        // small M: too few tiles for the machine -> several CTAs share a tile along K
        const SplitArea area = split_area(M, N);
        const int64_t tiles = static_cast<int64_t>(p.m_tiles) * ((N + 127) / 128);
        int64_t want = tiles > 0 ? info.sm_count / tiles : 1;
        if (want > p.k_tiles) want = p.k_tiles;
        // pays only when the K loop is long: the meeting in the workspace costs about 4 us of latency
        if (area.total() > 0 && split_bytes >= area.total() && want >= 2 && p.k_tiles >= 32) {
            p.k_per_split = static_cast<int32_t>((p.k_tiles + want - 1) / want);
            p.split_k = static_cast<int32_t>((p.k_tiles + p.k_per_split - 1) / p.k_per_split);
            p.counters = reinterpret_cast<uint32_t*>(d_split);
            p.partial = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(d_split) + area.counters_bytes);
            p.ldp = static_cast<int32_t>(area.ldp);
        }
    }
    p.flags = flags;
    p.nseg = nseg;
    for (int i = 0; i < nseg; ++i) p.seg_end[i] = static_cast<int32_t>(segs[i].col_begin + segs[i].col_count);
    {
        const uint64_t lim = g_wait_limit_ns.load(std::memory_order_relaxed);
        p.wait_limit_ns = lim != 0 ? lim : kWaitLimitNs;
    }
    cudaStream_t s = as_stream(stream);
    const bool fullk = (K % 256) == 0;
    if (fused != nullptr) {
        p.g_h = fused->g_h;
        p.h_codes = fused->h_codes;
        p.h_sf = fused->h_sf;
        p.h_katoms = fused->h_katoms;
        p.inner = fused->inner;
        p.dbg_y = fused->dbg_y;
        p.dbg_h = fused->dbg_h;
        p.split_k = 1;
        p.k_per_split = p.k_tiles;
        if (bn == 2) return fullk ? launch_gemm<256, 5, true, true, kEpiSwiglu>(tm, p, info.sm_count, s)
                                  : launch_gemm<256, 5, true, false, kEpiSwiglu>(tm, p, info.sm_count, s);
        return fullk ? launch_gemm<256, 3, false, true, kEpiSwiglu>(tm, p, info.sm_count, s)
                     : launch_gemm<256, 3, false, false, kEpiSwiglu>(tm, p, info.sm_count, s);
    }
    if (bn == 128 && fullk && M <= 128 && g_variant.load(std::memory_order_relaxed) == 0) {
        // decode-sized and fewer tiles than half the machine: share each tile along K inside a cluster
        GemmParams pc = p;
        pc.x = aq_x;
        pc.ldx = aq_ldx;
        const nvfp4_status cst = launch_gemm_cluster_split(tm, pc, info.sm_count, s, aq_x != nullptr);
        if (cst != NVFP4_ERR_SHAPE || aq_x != nullptr) return cst;
    }
    if (aq_x != nullptr) return NVFP4_ERR_SHAPE;
    switch (bn) {
        case 128: return fullk ? launch_gemm<128, 5, false, true>(tm, p, info.sm_count, s) : launch_gemm<128, 5, false, false>(tm, p, info.sm_count, s);
        case 256: return fullk ? launch_gemm<256, 3, false, true>(tm, p, info.sm_count, s) : launch_gemm<256, 3, false, false>(tm, p, info.sm_count, s);
        case 2: return fullk ? launch_gemm<256, 5, true, true>(tm, p, info.sm_count, s) : launch_gemm<256, 5, true, false>(tm, p, info.sm_count, s);
        default: return NVFP4_ERR_SHAPE;
    }
}

// 1 or 2 tokens: weight-streaming kernel on the CUDA cores, quantization included (decode.cuh)
template <int MT>
nvfp4_status launch_decode(const DecodeParams& p, int sm_count, cudaStream_t stream) {
    static std::mutex mu;
    static std::unordered_map<int, size_t> configured;     // per device: largest smem size set so far
    const size_t smem = decode_smem_bytes(MT, p.K);
    int dev = 0;
    cudaGetDevice(&dev);
    {
        std::lock_guard<std::mutex> lock(mu);
        if (configured[dev] < smem) {
            if (cudaFuncSetAttribute(decode_gemv_kernel<MT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     static_cast<int>(smem)) != cudaSuccess)
                return NVFP4_ERR_CUDA;
            configured[dev] = smem;
        }
    }
    const int64_t rows_per_cta = kDecodeThreads / 32;
    int64_t grid = (p.N + rows_per_cta - 1) / rows_per_cta;
    if (grid > sm_count) grid = sm_count;
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof(cfg));
    cudaLaunchAttribute attr[1];
    // may start while the kernel in front of it still runs (the kernel itself waits where it has to)
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3(static_cast<unsigned>(grid), 1, 1);
    cfg.blockDim = dim3(kDecodeThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, decode_gemv_kernel<MT>, p);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return e == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

// workspace of the fused call: [status][split-K reserve][codes][scales]; every part at an offset
// that does not depend on the problem size
size_t fused_codes_bytes(int64_t M, int64_t K) {        // rows padded to whole 128-row tiles
    const int64_t m_pad = (M + 127) / 128 * 128;
    return (static_cast<size_t>(m_pad) * static_cast<size_t>(K / 2) + 255) & ~static_cast<size_t>(255);
}
constexpr size_t kFusedCodesOffset = kStatusBytes + kSplitReserve;
size_t fused_min_bytes(int64_t M, int64_t K) {
    const size_t sf = (nvfp4_sf_bytes(M, K, NVFP4_SF_MMA) + 255) & ~static_cast<size_t>(255);
    return kFusedCodesOffset + fused_codes_bytes(M, K) + sf;
}

// rows up to which nvfp4_linear_bf16 quantizes the activations inside the GEMM kernel: every CTA
// quantizes the K range it multiplies, 48 times over for a 6144-wide layer.  The four warps that do
// it are otherwise idle during the main loop, but each of them sits alone on its scheduler: one
// 16-element block per thread and K tile (8 rows) hides under the weight stream (measured, 5120 ->
// 6144, CUDA-graph replay: 9.5-10.0 us against 11.5 us with the quantize kernel in front), two
// blocks per thread (9 to 16 rows) do not (11.0-11.9 us).
constexpr int64_t kInKernelQuantRows = 8;

// nvfp4_linear_bf16 on a workspace of the layout above; every argument is checked before
// anything is enqueued
nvfp4_status linear_bf16_impl(const void* d_x, int64_t ldx, const float* d_g_a, int64_t M, int64_t K,
                              const uint8_t* d_w_codes, const uint8_t* d_w_sf, int64_t N,
                              const nvfp4_segment* segs, const float* d_g_seg, int nseg, void* d_y, int64_t ldy,
                              uint32_t flags, void* d_workspace, size_t workspace_bytes, void* stream) {
    if (d_workspace == nullptr) return NVFP4_ERR_WORKSPACE;
    if (M < 0 || N < 0 || K <= 0 || (K % 64) != 0) return NVFP4_ERR_SHAPE;
    if (d_x == nullptr || d_g_a == nullptr || d_w_codes == nullptr || d_w_sf == nullptr || d_g_seg == nullptr ||
        d_y == nullptr)
        return NVFP4_ERR_NULL;
    if (ldx < K || ldy < N || M >= (1ll << 31) - 256 || N >= (1ll << 31) - 256 || K >= (1ll << 31)) return NVFP4_ERR_SHAPE;
    if ((flags & ~(NVFP4_OUT_F32 | NVFP4_WS_ZEROED | NVFP4_W_RESIDENT)) != 0u) return NVFP4_ERR_SHAPE;
    nvfp4_status st = check_segments(segs, nseg, N);
    if (N == 0 && segs != nullptr) st = NVFP4_OK;
    if (st != NVFP4_OK) return st;
    if ((reinterpret_cast<uintptr_t>(d_x) & 31u) != 0 || (ldx % 16) != 0 || !aligned16(d_w_codes) || !aligned16(d_w_sf) ||
        !aligned16(d_workspace))
        return NVFP4_ERR_ALIGN;
    const size_t min_bytes = fused_min_bytes(M, K);
    if (workspace_bytes < min_bytes) return NVFP4_ERR_WORKSPACE;
    if (M == 0 || N == 0) return NVFP4_OK;
    // measured on B200 (5120 -> 6144, CUDA-graph replay): one token is as fast through the
    // weight-streaming kernel as through the tensor cores (9.7 us); two tokens take 12.7 us there and
    // 9.7 us on the tensor cores, which need K to be a multiple of 256 to quantize A themselves
    if (M <= (((K % 256) == 0) ? 1 : 2) && g_variant.load(std::memory_order_relaxed) == 0 && decode_smem_bytes(M, K) <= 200 * 1024) {
        // decode-sized batch: one weight-streaming kernel; of the workspace only the status word is used
        DeviceInfo info;
        st = check_arch(info);
        if (st != NVFP4_OK) return st;
        DecodeParams dp;
        std::memset(&dp, 0, sizeof(dp));
        dp.x = reinterpret_cast<const uint16_t*>(d_x);
        dp.ldx = ldx;
        dp.g_a = d_g_a;
        dp.w_codes = d_w_codes;
        dp.w_sf = d_w_sf;
        dp.g_seg = d_g_seg;
        dp.y = d_y;
        dp.ldy = ldy;
        dp.status = reinterpret_cast<uint32_t*>(d_workspace);
        dp.M = static_cast<int32_t>(M);
        dp.N = static_cast<int32_t>(N);
        dp.K = static_cast<int32_t>(K);
        dp.flags = flags;
        dp.nseg = nseg;
        for (int i = 0; i < nseg; ++i) dp.seg_end[i] = static_cast<int32_t>(segs[i].col_begin + segs[i].col_count);
        cudaStream_t s = as_stream(stream);
        if (M == 1) return launch_decode<1>(dp, info.sm_count, s);
        return launch_decode<2>(dp, info.sm_count, s);
    }
    uint8_t* ws = reinterpret_cast<uint8_t*>(d_workspace);
    if (M <= kInKernelQuantRows && (K % 256) == 0 && g_variant.load(std::memory_order_relaxed) == 0) {
        // a handful of tokens: one kernel, which quantizes the K tiles of A it multiplies (gemm.cuh)
        return linear_impl(nullptr, nullptr, d_g_a, M, K, d_w_codes, d_w_sf, N, segs, d_g_seg, nseg, d_y, ldy, flags,
                           d_workspace, kStatusBytes, nullptr, 0, stream, 0, nullptr,
                           reinterpret_cast<const uint16_t*>(d_x), ldx);
    }
    uint8_t* codes = ws + kFusedCodesOffset;
    uint8_t* sf = codes + fused_codes_bytes(M, K);
    st = nvfp4_quantize_act(d_x, M, K, ldx, d_g_a, codes, sf, NVFP4_SF_MMA, stream);
    if (st != NVFP4_OK) return st;
    return linear_impl(codes, sf, d_g_a, M, K, d_w_codes, d_w_sf, N, segs, d_g_seg, nseg, d_y, ldy, flags, d_workspace,
                       kStatusBytes, ws + kStatusBytes, kSplitReserve, stream, (M + 127) / 128 * 128);
}
}  // namespace

extern "C" {

nvfp4_status nvfp4_linear(const uint8_t* d_a_codes, const uint8_t* d_a_sf, const float* d_g_a, int64_t M,
                          int64_t K, const uint8_t* d_w_codes, const uint8_t* d_w_sf, int64_t N,
                          const nvfp4_segment* segs, const float* d_g_seg, int nseg, void* d_y, int64_t ldy,
                          uint32_t flags, void* d_workspace, size_t workspace_bytes, void* stream) {
    void* split = nullptr;
    size_t split_bytes = 0;
    if (d_workspace != nullptr && workspace_bytes > kStatusBytes) {
        split = reinterpret_cast<uint8_t*>(d_workspace) + kStatusBytes;
        split_bytes = workspace_bytes - kStatusBytes;
        if (split_bytes > kSplitReserve) split_bytes = kSplitReserve;
    }
    return linear_impl(d_a_codes, d_a_sf, d_g_a, M, K, d_w_codes, d_w_sf, N, segs, d_g_seg, nseg, d_y, ldy, flags,
                       d_workspace, workspace_bytes, split, split_bytes, stream);
}

nvfp4_status nvfp4_linear_swiglu(const uint8_t* d_a_codes, const uint8_t* d_a_sf, const float* d_g_a, int64_t M, int64_t K,
                                 const uint8_t* d_w_codes, const uint8_t* d_w_sf, int64_t inner, const float* d_g_gate_up,
                                 const float* d_g_h, uint8_t* d_h_codes, uint8_t* d_h_sf, void* d_dbg_y, void* d_dbg_h,
                                 void* d_workspace, size_t workspace_bytes, void* stream) {
    if (d_g_h == nullptr || d_h_codes == nullptr || d_h_sf == nullptr) return NVFP4_ERR_NULL;
    if (inner <= 0 || (inner % 64) != 0 || inner >= (1ll << 29)) return NVFP4_ERR_SHAPE;
    if (!aligned16(d_h_codes) || (reinterpret_cast<uintptr_t>(d_h_sf) & 3u) != 0 ||
        ((reinterpret_cast<uintptr_t>(d_dbg_y) | reinterpret_cast<uintptr_t>(d_dbg_h)) & 31u) != 0)
        return NVFP4_ERR_ALIGN;
    GemmParams fused;
    std::memset(&fused, 0, sizeof(fused));
    fused.g_h = d_g_h;
    fused.h_codes = d_h_codes;
    fused.h_sf = d_h_sf;
    fused.h_katoms = static_cast<int32_t>(inner / 64);
    fused.inner = static_cast<int32_t>(inner);
    fused.dbg_y = d_dbg_y;
    fused.dbg_h = d_dbg_h;
    const nvfp4_segment segs[2] = {{0, inner}, {inner, inner}};        // only their scales are used: columns are interleaved
    return linear_impl(d_a_codes, d_a_sf, d_g_a, M, K, d_w_codes, d_w_sf, 2 * inner, segs, d_g_gate_up, 2, nullptr, 2 * inner, 0u,
                       d_workspace, workspace_bytes, nullptr, 0, stream, 0, &fused);
}

size_t nvfp4_linear_bf16_workspace_bytes(int64_t M, int64_t N, int64_t K, int nseg) {
    (void)N; (void)nseg;
    if (M < 0 || K < 0 || (K % 16) != 0) return 0;
    return fused_min_bytes(M, K);
}

nvfp4_status nvfp4_linear_bf16(const void* d_x, int64_t ldx, const float* d_g_a, int64_t M, int64_t K,
                               const uint8_t* d_w_codes, const uint8_t* d_w_sf, int64_t N,
                               const nvfp4_segment* segs, const float* d_g_seg, int nseg, void* d_y, int64_t ldy,
                               uint32_t flags, void* d_workspace, size_t workspace_bytes, void* stream) {
    return linear_bf16_impl(d_x, ldx, d_g_a, M, K, d_w_codes, d_w_sf, N, segs, d_g_seg, nseg, d_y, ldy, flags,
                            d_workspace, workspace_bytes, stream);
}

// ---------------------------------------------------------------- no-allocation variant
// Scratch for nvfp4_linear_bf16_static.  In host code this name is only a stand-in for the
// symbol: the device address comes from cudaGetSymbolAddress, per device.
static __device__ __align__(256) unsigned char g_static_scratch[NVFP4_STATIC_SCRATCH_BYTES];

namespace {
nvfp4_status static_scratch_address(void** out) {
    static std::mutex mu;
    static std::unordered_map<int, void*> by_device;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return NVFP4_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    auto it = by_device.find(dev);
    if (it != by_device.end()) { *out = it->second; return NVFP4_OK; }
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) {
        cudaGetLastError();
        return NVFP4_ERR_CUDA;
    }
    by_device[dev] = ptr;
    *out = ptr;
    return NVFP4_OK;
}
}  // namespace

nvfp4_status nvfp4_linear_bf16_static(const void* d_x, int64_t ldx, const float* d_g_a, int64_t M, int64_t K,
                                      const uint8_t* d_w_codes, const uint8_t* d_w_sf, int64_t N,
                                      const nvfp4_segment* segs, const float* d_g_seg, int nseg, void* d_y,
                                      int64_t ldy, uint32_t flags, void* stream) {
    if (M < 0 || K <= 0 || (K % 64) != 0) return NVFP4_ERR_SHAPE;
    if (fused_min_bytes(M, K) > NVFP4_STATIC_SCRATCH_BYTES) return NVFP4_ERR_WORKSPACE;   // beyond the fixed array
    void* scratch = nullptr;
    nvfp4_status st = static_scratch_address(&scratch);
    if (st != NVFP4_OK) return st;
    // The array starts as zeros (static storage) and only this library writes it: the status block
    // [0, 256) is cleared by nvfp4_static_status whenever it reports a failure, the split-K part
    // [256, 256 + reserve) is left zero by every call that uses it (and re-zeroed after a timeout),
    // the quantized activations live behind the reserve.  So the NVFP4_WS_ZEROED promise holds.
    return linear_bf16_impl(d_x, ldx, d_g_a, M, K, d_w_codes, d_w_sf, N, segs, d_g_seg, nseg, d_y, ldy,
                            flags | NVFP4_WS_ZEROED, scratch, NVFP4_STATIC_SCRATCH_BYTES, stream);
}

nvfp4_status nvfp4_static_status(void* stream) {
    void* scratch = nullptr;
    nvfp4_status st = static_scratch_address(&scratch);
    if (st != NVFP4_OK) return st;
    st = nvfp4_device_status(scratch, stream);
    if (st != NVFP4_OK) {
        // a kernel that gave up may have left counters or partial sums behind: bring the status block
        // and the split-K part back to zero so that later calls start clean (the stream is idle here)
        if (cudaMemsetAsync(scratch, 0, kStatusBytes + kSplitReserve, as_stream(stream)) != cudaSuccess) return NVFP4_ERR_CUDA;
        if (cudaStreamSynchronize(as_stream(stream)) != cudaSuccess) return NVFP4_ERR_CUDA;
    }
    return st;
}

nvfp4_status nvfp4_device_status(const void* d_workspace, void* stream) {
    if (d_workspace == nullptr) return NVFP4_ERR_NULL;
    uint32_t word = 0;
    if (cudaMemcpyAsync(&word, d_workspace, sizeof(word), cudaMemcpyDeviceToHost, as_stream(stream)) != cudaSuccess)
        return NVFP4_ERR_CUDA;
    if (cudaStreamSynchronize(as_stream(stream)) != cudaSuccess) return NVFP4_ERR_CUDA;
    if (word == 0u) return NVFP4_OK;
    if (word == NVFP4_ERR_TIMEOUT) return NVFP4_ERR_TIMEOUT;
    if (word == NVFP4_ERR_SCALE) return NVFP4_ERR_SCALE;
    return NVFP4_ERR_CUDA;
}

nvfp4_status nvfp4_gdn_lockstep(const float* d_q, const float* d_k, const float* d_v, const float* d_a, const float* d_b,
                                const float* d_q2, const float* d_k2, const float* d_v2, const float* d_a2, const float* d_b2,
                                const float* d_A_log, const float* d_dt_bias, int64_t T, int Hk, int Hv,
                                int64_t impulse_step, float impulse_rel, int64_t sample_every,
                                float* d_rel_state, float* d_rel_out, float* d_final_state, void* stream) {
    if (d_q == nullptr || d_k == nullptr || d_v == nullptr || d_a == nullptr || d_b == nullptr || d_q2 == nullptr ||
        d_k2 == nullptr || d_v2 == nullptr || d_a2 == nullptr || d_b2 == nullptr || d_A_log == nullptr ||
        d_dt_bias == nullptr || d_rel_state == nullptr || d_rel_out == nullptr)
        return NVFP4_ERR_NULL;
    if (T < 0 || Hk < 1 || Hv < 1 || Hv > 65535 || (Hv % Hk) != 0 || sample_every < 1 || !(impulse_rel > -1.0f)) return NVFP4_ERR_SHAPE;
    if (T == 0) return NVFP4_OK;
    DeviceInfo info;
    nvfp4_status st = check_arch(info);
    if (st != NVFP4_OK) return st;
    LockstepParams lp;
    std::memset(&lp, 0, sizeof(lp));
    lp.q[0] = d_q; lp.k[0] = d_k; lp.v[0] = d_v; lp.a[0] = d_a; lp.b[0] = d_b;
    lp.q[1] = d_q2; lp.k[1] = d_k2; lp.v[1] = d_v2; lp.a[1] = d_a2; lp.b[1] = d_b2;
    lp.A_log = d_A_log;
    lp.dt_bias = d_dt_bias;
    lp.T = T;
    lp.Hk = Hk;
    lp.Hv = Hv;
    lp.impulse_step = impulse_step;
    lp.impulse_rel = impulse_rel;
    lp.sample_every = sample_every;
    lp.rel_state = d_rel_state;
    lp.rel_out = d_rel_out;
    lp.final_state = d_final_state;
    const size_t smem = static_cast<size_t>(kGdnDim * (kGdnDim + 1) + kGdnDim) * sizeof(float);
    static std::mutex mu;
    static std::unordered_map<int, bool> configured;
    int dev = 0;
    cudaGetDevice(&dev);
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!configured[dev]) {
            if (cudaFuncSetAttribute(gdn_lockstep_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess)
                return NVFP4_ERR_CUDA;
            configured[dev] = true;
        }
    }
    gdn_lockstep_kernel<<<Hv, 256, smem, as_stream(stream)>>>(lp);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

nvfp4_status nvfp4_last_gemm_clock(const void* d_workspace, double* sm_mhz, double* kernel_us, void* stream) {
    if (d_workspace == nullptr || sm_mhz == nullptr || kernel_us == nullptr) return NVFP4_ERR_NULL;
    unsigned long long w[5] = {0, 0, 0, 0, 0};
    if (cudaMemcpyAsync(w, d_workspace, sizeof(w), cudaMemcpyDeviceToHost, as_stream(stream)) != cudaSuccess) return NVFP4_ERR_CUDA;
    if (cudaStreamSynchronize(as_stream(stream)) != cudaSuccess) return NVFP4_ERR_CUDA;
    const double ns = static_cast<double>(w[4] - w[2]), cycles = static_cast<double>(w[3] - w[1]);
    *kernel_us = ns * 1e-3;
    *sm_mhz = ns > 0.0 ? cycles / ns * 1e3 : 0.0;
    return NVFP4_OK;
}

namespace nvfp4 {
// One CTA waits, with the library's bounded wait, on a barrier that nothing ever completes.
__global__ void bounded_wait_selftest_kernel(uint32_t* status, uint64_t limit_ns) {
    __shared__ uint64_t bar;
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bar, 1);
        abort_flag = 0u;
        ptx::fence_barrier_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const bool completed = ptx::mbar_wait_bounded(&bar, 0u, &abort_flag, limit_ns);
        *status = completed ? static_cast<uint32_t>(NVFP4_OK) : static_cast<uint32_t>(NVFP4_ERR_TIMEOUT);
    }
}
}  // namespace nvfp4

nvfp4_status nvfp4_selftest_bounded_wait(void* d_workspace, size_t workspace_bytes, uint64_t limit_ns, void* stream) {
    if (d_workspace == nullptr) return NVFP4_ERR_NULL;
    if (workspace_bytes < kStatusBytes) return NVFP4_ERR_WORKSPACE;
    if (limit_ns == 0 || limit_ns > 1000000000ull) return NVFP4_ERR_SHAPE;      // at most one second
    DeviceInfo info;
    nvfp4_status st = check_arch(info);
    if (st != NVFP4_OK) return st;
    bounded_wait_selftest_kernel<<<1, 32, 0, as_stream(stream)>>>(reinterpret_cast<uint32_t*>(d_workspace), limit_ns);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

nvfp4_status nvfp4_set_wait_limit_ns(uint64_t limit_ns) {
    g_wait_limit_ns.store(limit_ns, std::memory_order_relaxed);
    return NVFP4_OK;
}

uint64_t nvfp4_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

nvfp4_status nvfp4_set_gemm_variant(int variant) {
    if (variant != 0 && variant != 128 && variant != 256 && variant != 2) return NVFP4_ERR_SHAPE;
    g_variant.store(variant, std::memory_order_relaxed);
    return NVFP4_OK;
}

const char* nvfp4_gemm_variants(void) {
    return "0=auto,128=128x128 tiles (2 accumulators),256=128x256 tiles,2=256x256 tiles on CTA pairs";
}

const char* nvfp4_status_string(nvfp4_status s) {
    switch (s) {
        case NVFP4_OK: return "ok";
        case NVFP4_ERR_NULL: return "null pointer";
        case NVFP4_ERR_SHAPE: return "bad shape or flag";
        case NVFP4_ERR_ALIGN: return "misaligned pointer or leading dimension";
        case NVFP4_ERR_SEGMENTS: return "segment table does not cover [0, N) in order";
        case NVFP4_ERR_WORKSPACE: return "workspace missing or too small";
        case NVFP4_ERR_ARCH: return "device is not compute capability 10.x";
        case NVFP4_ERR_CUDA: return "CUDA call failed";
        case NVFP4_ERR_TIMEOUT: return "a bounded in-kernel wait ran out";
        case NVFP4_ERR_LAYOUT: return "unknown or unsupported scale layout";
        case NVFP4_ERR_SCALE: return "a global scale is not finite and positive";
    }
    return "unknown status";
}

}  // extern "C"
