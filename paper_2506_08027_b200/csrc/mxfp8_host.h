// Host-side declarations shared by the translation units of the library (not public).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#include "../../include/mxfp8.h"

namespace mxfp8 {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
// element types of the conversion kernels (Table 1) / of the tensor-core path of this library
inline bool valid_elem(int e) { return e == MXFP8_E4M3 || e == MXFP8_E5M2 || e == MXFP8_E2M3 || e == MXFP8_E3M2 || e == MXFP8_E2M1; }
inline bool fp8_elem(int e) { return e == MXFP8_E4M3 || e == MXFP8_E5M2; }

// Raises a kernel's dynamic shared-memory limit once per (kernel instantiation, device): the call
// costs several microseconds of host time and its effect lasts for the life of the context.
// `done` is a bit mask of devices, one static per call site.
template <typename Kernel>
inline cudaError_t ensure_dynamic_smem(Kernel kernel, int bytes, unsigned long long& done)
{
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    const unsigned long long bit = 1ull << (dev & 63);
    if (__atomic_load_n(&done, __ATOMIC_ACQUIRE) & bit) return cudaSuccess;
    err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (err == cudaSuccess) __atomic_fetch_or(&done, bit, __ATOMIC_RELEASE);
    return err;
}

// n / d and n % d for 0 <= n < 2^31, 1 <= d, without a division on the device: a multiply by
// magic = min(floor(2^32 / d), 2^32 - 1) gives the quotient or one less, one correction settles it.
// (The conversion kernel turns a tile index into tile coordinates with it; the host computes the magic.)
inline __host__ __device__ uint32_t div_magic(uint32_t d) { return d <= 1u ? 0xFFFFFFFFu : (uint32_t)(0x100000000ull / d); }
inline __host__ __device__ void divmod(uint32_t n, uint32_t d, uint32_t magic, int& q, int& r)
{
#ifdef __CUDA_ARCH__
    uint32_t qq = __umulhi(n, magic);
#else
    uint32_t qq = (uint32_t)(((uint64_t)n * magic) >> 32);
#endif
    uint32_t rr = n - qq * d;
    if (rr >= d) { rr -= d; ++qq; }
    q = (int)qq; r = (int)rr;
}

// A small integer per (device, stream), handed out on first use and kept: the index of the stream's own words in a
// device-side array (the conversion kernel's tile counter).  Kernels of one stream run one after the other, so words
// that belong to a stream are never used by two kernels at once.  Returns -1 when no index can be given safely: the
// per-thread default stream (one handle, many streams), a stream that is being captured (the captured launch may be
// replayed on any stream later, or next to a second instance of its graph), more streams than slots, a failing
// runtime call.  The caller then takes its path that needs no such words.
class StreamSlots {
public:
    static constexpr int SLOTS = 64;
    int get(cudaStream_t stream)
    {
        if (stream == cudaStreamPerThread) return -1;
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(stream, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone) return -1;
        int device = 0;
        if (cudaGetDevice(&device) != cudaSuccess) return -1;
        const int used = __atomic_load_n(&used_, __ATOMIC_ACQUIRE);
        for (int i = 0; i < used; ++i)
            if (stream_[i] == stream && device_[i] == device) return i;
        while (__atomic_exchange_n(&lock_, 1, __ATOMIC_ACQUIRE)) {}
        int slot = -1;
        for (int i = 0; i < used_; ++i)
            if (stream_[i] == stream && device_[i] == device) slot = i;
        if (slot < 0 && used_ < SLOTS) {
            slot = used_;
            stream_[slot] = stream;
            device_[slot] = device;
            __atomic_store_n(&used_, used_ + 1, __ATOMIC_RELEASE);
        }
        __atomic_store_n(&lock_, 0, __ATOMIC_RELEASE);
        return slot;
    }

private:
    cudaStream_t stream_[SLOTS] = {};
    int device_[SLOTS] = {};
    int used_ = 0;
    int lock_ = 0;
};

// A value per device that costs driver calls to find (multiprocessor count, the address of a __device__ symbol:
// every device holds its own copy of each symbol, at its own address).  get() fills the current device's slot on
// first use, under a lock, and afterwards reads it without one.  `fill(device, value)` returns false on failure,
// which is not cached.  The device index can be given (tests); by default it is the calling thread's current device.
template <typename T>
class PerDeviceCache {
public:
    static constexpr int MAX_DEVICES = 64;
    template <typename Fill>
    bool get(T& out, Fill fill, int device = -1)
    {
        if (device < 0 && cudaGetDevice(&device) != cudaSuccess) return false;
        if (device < 0 || device >= MAX_DEVICES) return false;
        const unsigned long long bit = 1ull << device;
        if (!(__atomic_load_n(&done_, __ATOMIC_ACQUIRE) & bit)) {
            while (__atomic_exchange_n(&lock_, 1, __ATOMIC_ACQUIRE)) {}
            bool ok = true;
            if (!(done_ & bit)) {
                T v{};
                ok = fill(device, v);
                if (ok) {
                    slot_[device] = v;
                    __atomic_fetch_or(&done_, bit, __ATOMIC_RELEASE);
                }
            }
            __atomic_store_n(&lock_, 0, __ATOMIC_RELEASE);
            if (!ok) return false;
        }
        out = slot_[device];
        return true;
    }

private:
    T slot_[MAX_DEVICES] = {};
    unsigned long long done_ = 0;
    int lock_ = 0;
};

// Encoded TMA tensor maps, kept in static storage (nothing is allocated) and keyed by every argument of the encode call.  A map is a pure
// function of those arguments (address, extents, pitches, box, types), so a cached one is valid for as long as
// the caller's buffer is; the cache owns nothing.  Direct-mapped: a colliding key replaces the entry.
// One driver call per map costs about a microsecond, and a launch needs 5 to 15 of them.
struct TensorMapKey {
    const void* base;
    uint64_t dim[3], stride[2];
    uint32_t box[3];
    uint32_t dtype, rank, swizzle, l2;
};
template <typename Map>
class TensorMapCache {
public:
    template <typename Encode>
    bool get(const TensorMapKey& key, Map* out, Encode encode)
    {
        const unsigned char* b = reinterpret_cast<const unsigned char*>(&key);
        uint64_t h = 1469598103934665603ull;
        for (size_t i = 0; i < sizeof(key); ++i) h = (h ^ b[i]) * 1099511628211ull;
        Entry& e = entries_[h % SLOTS];
        while (__atomic_exchange_n(&lock_, 1, __ATOMIC_ACQUIRE)) {}
        const bool hit = e.valid && memcmp(&e.key, &key, sizeof(key)) == 0;
        if (hit) *out = e.map;
        __atomic_store_n(&lock_, 0, __ATOMIC_RELEASE);
        if (hit) return true;
        if (!encode(out)) return false;
        while (__atomic_exchange_n(&lock_, 1, __ATOMIC_ACQUIRE)) {}
        e.key = key;
        e.map = *out;
        e.valid = true;
        __atomic_store_n(&lock_, 0, __ATOMIC_RELEASE);
        return true;
    }

private:
    static constexpr int SLOTS = 256;
    struct Entry { TensorMapKey key; Map map; bool valid; };
    Entry entries_[SLOTS] = {};
    int lock_ = 0;
};
inline TensorMapKey tensor_map_key(const void* base, uint32_t dtype, uint32_t rank, const uint64_t* dims, const uint64_t* strides,
                                   const uint32_t* box, uint32_t swizzle, uint32_t l2)
{
    TensorMapKey k;
    memset(&k, 0, sizeof(k));   // padding bytes take part in the comparison
    k.base = base; k.dtype = dtype; k.rank = rank; k.swizzle = swizzle; k.l2 = l2;
    for (uint32_t i = 0; i < rank; ++i) { k.dim[i] = dims[i]; k.box[i] = box[i]; }
    for (uint32_t i = 0; i + 1 < rank; ++i) k.stride[i] = strides[i];
    return k;
}

// Launch accounting (mxfp8_launch_count).
int64_t launches();
void count_launch(int n);

// Device-pointer implementations behind the C entry points (arguments already validated).
int quantize_device(const void* src, int src_dtype, int64_t rows, int64_t cols, int orientation,
                    int scale_rule, int elem, void* q_row, void* s_row, void* q_col, void* s_col,
                    int sf_layout, cudaStream_t stream);

// TMA fast path of mxfp8_quantize (quantize_tma.cu).
bool quantize_tma_eligible(int src_dtype, int64_t rows, int64_t cols);
int quantize_tma_device(const void* src, int src_dtype, int64_t rows, int64_t cols, int orientation,
                        int scale_rule, int elem, void* q_row, void* s_row, void* q_col, void* s_col,
                        int sf_layout, cudaStream_t stream, bool emulate = false);
// Several tensors of one dtype in one launch (same orientation, rule, element format, scale layout).
struct QuantizeItem {
    const void* src;
    int64_t rows, cols;
    void *q_row, *s_row, *q_col, *s_col;
};
int quantize_tma_batch(const QuantizeItem* items, int count, int src_dtype, int orientation, int scale_rule, int elem,
                       int sf_layout, cudaStream_t stream, bool emulate = false, int act = MXFP8_ACT_NONE,
                       const float* rstd = nullptr, const void* gamma = nullptr, bool gated = false,
                       const float* mean = nullptr, const void* beta = nullptr, const void* second_src = nullptr);
int quantize_read_and_clear_status();

// Device status word (bounded waits report here); defined in gemm.cu.
int read_and_clear_device_status(cudaStream_t stream);

}  // namespace mxfp8
