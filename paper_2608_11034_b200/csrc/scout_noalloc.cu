#include <mutex>

#include "scout_combine.cuh"
#include "scout_scan.cuh"

// ---- signing without any allocation ------------------------------------------
// scout_sign_chunks_noalloc serves callers that must not allocate device memory
// while they run: a health check placed in the middle of a training step, where
// the framework's caching allocator already holds almost all of HBM (a
// cudaMalloc there can fail, and it also stalls the device), or a handler that
// runs right after an out-of-memory error.  It takes no plan: the replicas are R
// contiguous buffers holding one tensor each, and the per-tile partial records
// go to a fixed array that lives in the library's device image.
namespace scout {
namespace {

constexpr uint32_t NOALLOC_MAX_RECORDS = 65536;  // 2 MiB of scratch, held by every GPU that loads the library
constexpr uint32_t NOALLOC_MAX_DEVICES = 64;

// The scratch itself.  In host code this name is only a stand-in for the
// symbol, not an address a kernel can use; the host obtains the device address
// with cudaGetSymbolAddress (below) and passes that to the kernels.
// Eight records (256 bytes) of guard band on either side: they are filled with a pattern at
// set-up and scout_noalloc_guards_ok() checks that no kernel has written to them.
constexpr uint32_t NOALLOC_GUARD_RECORDS = 8;
constexpr int NOALLOC_GUARD_PATTERN = 0xC3;
static __device__ __align__(256) TileRec g_noalloc_scratch[NOALLOC_GUARD_RECORDS + NOALLOC_MAX_RECORDS +
                                                           NOALLOC_GUARD_RECORDS];

struct NoallocArgs {
    const uint8_t *replica[64];
    uint64_t nbytes, chunk_bytes, meta;
    uint64_t n_tiles;          // tiles per replica
    uint32_t tiles_per_chunk;  // tiles of a full chunk
    uint32_t tile_bytes;
    uint32_t R, dtype;
    TileRec *recs;             // device address of g_noalloc_scratch
    scout_sig_t *sigs;
};

// Same scan as sign_tiles_direct, with the tile geometry computed from the tile
// index instead of read from a table (there is no table: nothing was allocated).
__global__ void __launch_bounds__(SIGN_THREADS) sign_tiles_noalloc(const __grid_constant__ NoallocArgs a) {
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t warp = (uint64_t)blockIdx.x * (SIGN_THREADS / 32) + (threadIdx.x >> 5);
    const uint64_t n_warps = (uint64_t)gridDim.x * (SIGN_THREADS / 32);
    const uint64_t n_items = a.n_tiles * a.R;
    for (uint64_t item = warp; item < n_items; item += n_warps) {
        const uint32_t r = (uint32_t)(item / a.n_tiles);
        const uint64_t t = item - (uint64_t)r * a.n_tiles;
        const uint64_t c = t / a.tiles_per_chunk;
        const uint64_t j = t - c * a.tiles_per_chunk;
        const uint64_t chunk_off = c * a.chunk_bytes;
        const uint64_t chunk_n = min(a.chunk_bytes, a.nbytes - chunk_off);
        const uint64_t in_chunk = j * a.tile_bytes;
        const uint32_t n = (uint32_t)min((uint64_t)a.tile_bytes, chunk_n - in_chunk);
        TileRec rec;
        scan_dispatch(a.dtype, a.replica[r] + chunk_off + in_chunk, n, lane, rec);
        if (lane == 0) a.recs[(uint64_t)r * a.n_tiles + t] = rec;
    }
}

// The combine of finalize_chunks for a single tensor whose chunk geometry is arithmetic.
__global__ void __launch_bounds__(FIN_THREADS) finalize_noalloc(const __grid_constant__ NoallocArgs a,
                                                                uint64_t C, uint64_t p_stride) {
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t warp = (uint64_t)blockIdx.x * (FIN_THREADS / 32) + (threadIdx.x >> 5);
    const uint64_t n_warps = (uint64_t)gridDim.x * (FIN_THREADS / 32);
    const uint32_t tile_rows = a.tile_bytes / ROW_BYTES;
    for (uint64_t item = warp; item < C * a.R; item += n_warps) {
        const uint64_t c = item / a.R;
        const uint32_t r = (uint32_t)(item - c * a.R);
        const uint64_t chunk_n = min(a.chunk_bytes, a.nbytes - c * a.chunk_bytes);
        const uint32_t nt = (uint32_t)((chunk_n + a.tile_bytes - 1) / a.tile_bytes);
        const scout_sig_t o = combine_tiles(a.recs + (uint64_t)r * a.n_tiles + c * a.tiles_per_chunk, nt,
                                            chunk_n, c, a.dtype, a.meta, p_stride,
                                            combine_weight(nt, chunk_n, tile_rows, lane), lane);
        if (lane == 0) {
            a.sigs[c * a.R + r] = o;
        }
    }
}

// Device address of the scratch array and SM count, looked up once per device.
// The table is filled under a mutex, so that host threads making their first call
// at the same time do not race on it.
struct NoallocDevice {
    TileRec *scratch;
    int sms;
    bool ready;
};
static NoallocDevice g_noalloc_dev[NOALLOC_MAX_DEVICES];
static std::mutex g_noalloc_mutex;

int noalloc_setup(int device, NoallocDevice *out) {
    if (device < 0 || device >= (int)NOALLOC_MAX_DEVICES) return SCOUT_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> guard(g_noalloc_mutex);
    NoallocDevice &d = g_noalloc_dev[device];
    if (!d.ready) {
        // `device` is the current device here, so the address is this GPU's copy
        void *ptr = nullptr;
        SCOUT_CUDA(cudaGetSymbolAddress(&ptr, g_noalloc_scratch));
        int sms = 0;
        SCOUT_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
        TileRec *base = static_cast<TileRec *>(ptr);
        SCOUT_CUDA(cudaMemset(base, NOALLOC_GUARD_PATTERN, NOALLOC_GUARD_RECORDS * sizeof(TileRec)));
        SCOUT_CUDA(cudaMemset(base + NOALLOC_GUARD_RECORDS + NOALLOC_MAX_RECORDS, NOALLOC_GUARD_PATTERN,
                              NOALLOC_GUARD_RECORDS * sizeof(TileRec)));
        d.scratch = base + NOALLOC_GUARD_RECORDS;
        d.sms = sms;
        d.ready = true;
    }
    *out = d;
    return SCOUT_OK;
}

}  // namespace
}  // namespace scout

extern "C" int scout_noalloc_guards_ok(int *ok) {
    using namespace scout;
    if (!ok) return SCOUT_ERR_INVALID;
    int device = 0;
    SCOUT_CUDA(cudaGetDevice(&device));
    NoallocDevice dev;
    int rc = noalloc_setup(device, &dev);
    if (rc) return rc;
    SCOUT_CUDA(cudaDeviceSynchronize());
    uint8_t host[2 * NOALLOC_GUARD_RECORDS * sizeof(TileRec)];
    const size_t band = NOALLOC_GUARD_RECORDS * sizeof(TileRec);
    SCOUT_CUDA(cudaMemcpy(host, dev.scratch - NOALLOC_GUARD_RECORDS, band, cudaMemcpyDeviceToHost));
    SCOUT_CUDA(cudaMemcpy(host + band, dev.scratch + NOALLOC_MAX_RECORDS, band, cudaMemcpyDeviceToHost));
    *ok = 1;
    for (uint8_t b : host)
        if (b != (uint8_t)NOALLOC_GUARD_PATTERN) *ok = 0;
    return SCOUT_OK;
}

extern "C" int scout_sign_chunks_noalloc(uint32_t R, const void *const *replica_ptrs, uint64_t nbytes,
                                         uint32_t dtype, uint64_t meta_tag, uint64_t chunk_bytes,
                                         scout_sig_t *d_sigs, void *stream) {
    using namespace scout;
    if (R < 2 || !replica_ptrs || !d_sigs || nbytes == 0) return SCOUT_ERR_INVALID;
    if (R > 64) return SCOUT_ERR_UNSUPPORTED;
    if (chunk_bytes == 0 || chunk_bytes % ROW_BYTES != 0 || chunk_bytes > (1ull << 30))
        return SCOUT_ERR_INVALID;
    static const uint32_t elem[7] = {1, 4, 2, 8, 2, 8, 4};
    if (dtype > SCOUT_DT_I32 || nbytes % elem[dtype] != 0) return SCOUT_ERR_INVALID;
    for (uint32_t r = 0; r < R; ++r) {
        if (!replica_ptrs[r]) return SCOUT_ERR_INVALID;
        if ((uintptr_t)replica_ptrs[r] & 15u) return SCOUT_ERR_ALIGN;
    }
    // smallest tile (power of two, 2 KiB .. 64 KiB) whose records fit the fixed scratch
    const uint64_t C = (nbytes + chunk_bytes - 1) / chunk_bytes;
    const uint64_t last_n = nbytes - (C - 1) * chunk_bytes;
    uint32_t tile = 2048;
    uint64_t tpc = 0, n_tiles = 0;
    for (;; tile *= 2) {
        tpc = (chunk_bytes + tile - 1) / tile;
        n_tiles = (C - 1) * tpc + (last_n + tile - 1) / tile;
        if (n_tiles * R <= NOALLOC_MAX_RECORDS) break;
        if (tile == 65536) return SCOUT_ERR_UNSUPPORTED;  // more data than the fixed scratch covers
    }
    int device = 0;
    SCOUT_CUDA(cudaGetDevice(&device));
    NoallocDevice dev_info;
    int rc = noalloc_setup(device, &dev_info);
    if (rc) return rc;
    const NoallocDevice *dev = &dev_info;

    NoallocArgs a;
    for (uint32_t r = 0; r < 64; ++r) a.replica[r] = r < R ? (const uint8_t *)replica_ptrs[r] : nullptr;
    a.nbytes = nbytes;
    a.chunk_bytes = chunk_bytes;
    a.meta = meta_tag;
    a.n_tiles = n_tiles;
    a.tiles_per_chunk = (uint32_t)tpc;
    a.tile_bytes = tile;
    a.R = R;
    a.dtype = dtype;
    a.recs = dev->scratch;
    a.sigs = d_sigs;
    cudaStream_t s = (cudaStream_t)stream;
    const uint64_t items = n_tiles * R;
    uint64_t grid = (items + SIGN_THREADS / 32 - 1) / (SIGN_THREADS / 32);
    if (grid > (uint64_t)dev->sms * 4) grid = (uint64_t)dev->sms * 4;
    sign_tiles_noalloc<<<(unsigned)grid, SIGN_THREADS, 0, s>>>(a);
    SCOUT_CUDA(cudaGetLastError());
    uint64_t fgrid = (C * R + FIN_THREADS / 32 - 1) / (FIN_THREADS / 32);
    if (fgrid > (uint64_t)dev->sms * 8) fgrid = (uint64_t)dev->sms * 8;
    finalize_noalloc<<<(unsigned)fgrid, FIN_THREADS, 0, s>>>(a, C, pow_p(32ull * (tile / ROW_BYTES)));
    SCOUT_CUDA(cudaGetLastError());
    return SCOUT_OK;
}
