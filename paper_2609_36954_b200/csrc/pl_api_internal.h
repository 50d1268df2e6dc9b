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
  std::string last_error;
};

namespace pl {
extern std::atomic<uint64_t> g_launches;
// true when the calling thread's current CUDA device is the communicator's (always for a planner)
bool on_comm_device(pl_comm_s* comm);
}
