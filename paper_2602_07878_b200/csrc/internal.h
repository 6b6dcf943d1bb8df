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

// The workspace starts with a fixed header of HDR_WORDS int32, followed by two plan regions of
// which calls use one in turn: the plan kernel of a call fills the region that the previous
// call did not use, while that call's combine kernel may still be reading its own, and
// publishes the switch (HDR_GEN) only after the previous call has completed.  A region starts
// with a header of its own (same word indices), then holds the per-sequence entries, the list of
// sequences for the combine kernel and the work item records.
enum {
    HDR_N_ITEMS = 0,   // region; mirrored into the fixed header for callers that look
    HDR_N_UNITS = 1,   // region
    HDR_P = 2,         // region; mirrored into the fixed header
    HDR_COUNTER = 3,   // region: next unit to hand out
    HDR_STATUS = 4,    // fixed header: status word of calls that pass no dev_status
    HDR_N_MULTI = 5,   // region
    HDR_N_LONG = 6,    // region
    HDR_GEN = 7,       // fixed header: bit 0 selects the region of the plan in force
    HDR_WORDS = 64
};

// bit 16 of record.z: the sequence has a single partition, write bf16 output directly
constexpr int REC_DIRECT = 1 << 16;

struct WsLayout {
    size_t off_region, region_bytes;              // first plan region, distance to the second
    size_t off_seqinfo, off_multi, off_records;   // inside a region
    size_t off_ml, off_o, total;
    int64_t item_cap;
};

// what a kernel needs to find the plan region in force
struct PlanAddr {
    int* fixed;                 // the fixed header
    unsigned char* region0;     // the first region
    size_t region_bytes;
    size_t off_seqinfo, off_multi, off_records;
};
struct PlanView {
    int* hdr;
    int2* seq_info;
    int* multi;
    int4* records;
};
#ifdef __CUDACC__
__device__ __forceinline__ PlanView plan_view(const PlanAddr& a, int gen) {
    unsigned char* r = a.region0 + (size_t)(gen & 1) * a.region_bytes;
    PlanView v;
    v.hdr = reinterpret_cast<int*>(r);
    v.seq_info = reinterpret_cast<int2*>(r + a.off_seqinfo);
    v.multi = reinterpret_cast<int*>(r + a.off_multi);
    v.records = reinterpret_cast<int4*>(r + a.off_records);
    return v;
}
#endif
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
