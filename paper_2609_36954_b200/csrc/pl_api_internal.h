// Handle definitions shared by the C-ABI translation units.
#pragma once
#include <atomic>
#include <cstdint>
#include <mutex>
#include <string>
#include <vector>

#include "purlin.h"

constexpr int kStatusWords = 16;  // pl_devstatus_t words [0..8) + abort word [8]

struct pl_comm_s {
  int R = 0;
  int dtype = 0;
  bool planner = false;
  int device = -1;
  int sm_count = 148;
  int* d_status = nullptr;
  void* status_stream = nullptr;  // non-blocking stream used only to read the status record
  std::mutex mu;
  std::vector<pl_schedule_s*> schedules;
  int n_plans = 0;
  int tuned_push_ctas = 0;  // pl_comm_tune: best grid for pushed copies on the bulk-copy datapath (0 = not measured)
  int tuned_idle_first = 0, tuned_idle_count = 0;  // and the idle SM window measured with it (count 0: plain launch)
  std::string last_error;
  // pl_execute_host_async: an upload and a download stream, and the downloads still in flight
  // with the host and device ranges they touch (hazards are resolved with their events)
  struct Range { const char* lo; const char* hi; };
  struct Download {
    void* done = nullptr;          // cudaEvent_t recorded behind the download's last copy
    std::vector<Range> host_out;   // host ranges the download writes
    std::vector<Range> dev_out;    // device ranges it reads
    bool live = false;
  };
  static constexpr int kHostSlots = 8;
  void* up_stream = nullptr;
  void* down_stream = nullptr;
  void* ev_up[kHostSlots] = {};      // uploads of call n complete
  void* ev_kernel[kHostSlots] = {};  // schedule of call n complete
  void* ev_entry = nullptr;
  Download downloads[kHostSlots];
  uint64_t host_calls = 0;           // async host executes so far
  void* host_stream_last = nullptr;  // the caller's stream of the previous async host execute
  int last_download = -1;            // slot of the most recent download
  uint64_t host_h2d_bytes = 0, host_d2h_bytes = 0;  // bytes the host entry points have copied so far
  std::mutex host_mu;                // serialises the host-pipeline entry points
};

namespace pl {
extern std::atomic<uint64_t> g_launches;
// true when the calling thread's current CUDA device is the communicator's (always for a planner)
bool on_comm_device(pl_comm_s* comm);
}
