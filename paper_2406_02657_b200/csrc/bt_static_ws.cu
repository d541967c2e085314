// bt_block_decode_attn_noalloc: block-decoder decode attention whose split scratch lives in
// a file-scope device array instead of a caller-supplied workspace.
//
// Some hosts of this library cannot hand over a workspace: a serving process whose own pool
// reserved all device memory at start-up has nothing left to cudaMalloc from, and a decode
// loop with a latency budget cannot afford the device-wide synchronisation an allocation
// implies.  For them the scratch is part of the loaded module: every GPU that loads the
// library holds BT_STATIC_WORKSPACE_BYTES of it until the process exits.
//
// The array's name is only a host-side handle here; the kernels need its device address,
// which differs per device, so it is looked up once per device with cudaGetSymbolAddress
// (while that device is current) and remembered.
#include <cuda_runtime.h>

#include <mutex>

#include "../../include/bt.h"
#include "bt_kernels.h"

namespace {

static __device__ __align__(256) unsigned char g_static_ws[BT_STATIC_WORKSPACE_BYTES];

constexpr int kMaxDevices = 64;
void* g_ws_addr[kMaxDevices];  // device address of g_static_ws on each device, 0 = not looked up yet
std::mutex g_ws_mutex;

// Device address of the scratch array on the current device (set-up on first use).
bt_status static_ws_on_current_device(void** addr)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return BT_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return BT_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_ws_mutex);
    if (!g_ws_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_ws) != cudaSuccess || !p) {
            (void)cudaGetLastError();  // the failure is reported here; it must not surface in a later call's launch check
            return BT_ERR_CUDA;
        }
        g_ws_addr[dev] = p;
    }
    *addr = g_ws_addr[dev];
    return BT_OK;
}

}  // namespace

extern "C" bt_status bt_block_decode_attn_noalloc(const bt_config* cfg, const bt_block_cache* cache, int layer,
                                                  const void* q, void* out, uint32_t* dev_status, void* stream)
{
    // every argument is judged first: a call that is refused has enqueued nothing and has not touched the
    // shared scratch, which a call already in flight may be using
    bt_status st = bt::validate_decode_attn_args(cfg, cache, layer, q, out, dev_status);
    if (st != BT_OK) return st;
    if (bt_workspace_bytes(cfg) > (size_t)BT_STATIC_WORKSPACE_BYTES) return BT_ERR_WORKSPACE;
    void* ws = nullptr;
    if (bt_decode_splits(cfg) > 1) {
        st = static_ws_on_current_device(&ws);
        if (st != BT_OK) return st;
        // configs of different shapes share the array, and one config's partial results may lie where
        // another's arrival counters do: the counters are zeroed (a memset node, no allocation) every time
        st = bt_workspace_init(cfg, ws, (size_t)BT_STATIC_WORKSPACE_BYTES, stream);
        if (st != BT_OK) return st;
    }
    return bt_block_decode_attn(cfg, cache, layer, q, out, ws, ws ? (size_t)BT_STATIC_WORKSPACE_BYTES : 0,
                                dev_status, stream);
}
