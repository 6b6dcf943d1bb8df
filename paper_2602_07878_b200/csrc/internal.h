// Host/device declarations shared by the library's translation units (not installed).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/pagedkv.h"

namespace pk {

constexpr int BS = 16;        // tokens per KV block (the only block size supported)
constexpr int MAX_PART = 512; // largest partition: 32 blocks, one block id per producer lane

// int32 words of the plan header at the start of the workspace
enum { HDR_N_ITEMS = 0, HDR_N_UNITS = 1, HDR_P = 2, HDR_COUNTER = 3, HDR_STATUS = 4, HDR_N_MULTI = 5, HDR_N_LONG = 6, HDR_WORDS = 64 };

// bit 16 of record.z: the sequence has a single partition, write bf16 output directly
constexpr int REC_DIRECT = 1 << 16;

struct WsLayout {
    size_t off_seqinfo, off_multi, off_records, off_ml, off_o, total;
    int64_t item_cap;
};
// carve a workspace of `bytes` (or compute `total` for `item_cap` when bytes == 0)
WsLayout ws_layout(int H, int D, int64_t batch, int64_t item_cap, size_t bytes);

// per-thread error slot for PA_ERR_CUDA
void set_cuda_error(int code);
int check_cuda(cudaError_t e);  // returns PA_OK or PA_ERR_CUDA (and records e)
void count_launch(int n = 1);

struct DeviceInfo {
    int device;
    int sm_count;
    int smem_optin;
};
int get_device_info(DeviceInfo* info);

int validate_shape(const pa_shape* s);

// TMA tensor map over one layer's cache: dims (dim, slot, kv head, block), box 64 x 16 x 1 x 1,
// 128-byte swizzle; block ids outside the pool are out of bounds and read as zeros.
int make_cache_map(CUtensorMap* map, const void* base, const pa_shape* s);

constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;  // bound of every in-kernel wait

}  // namespace pk
