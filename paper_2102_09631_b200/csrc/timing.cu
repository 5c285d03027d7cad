// Per-kernel timing for the benchmark: when enabled, every launch of this library is bracketed by
// CUDA events on its own stream; dad_timing_collect() synchronises and sums the elapsed time per tag.
#include <mutex>
#include <string>
#include <vector>

#include "common.cuh"

namespace dad {

std::atomic<bool> g_timing{false};

namespace {
struct Span {
  int tag;
  cudaEvent_t a, b;
};
struct Tag {
  std::string name;
  double ms = 0.0;
  uint64_t launches = 0;
};
std::mutex g_mu;
std::vector<Tag> g_tags;
std::vector<Span> g_open;
std::vector<cudaEvent_t> g_free;

int tag_index(const char* name) {
  for (size_t i = 0; i < g_tags.size(); ++i)
    if (g_tags[i].name == name) return (int)i;
  g_tags.push_back(Tag{name});
  return (int)g_tags.size() - 1;
}
cudaEvent_t get_event() {
  if (!g_free.empty()) {
    cudaEvent_t e = g_free.back();
    g_free.pop_back();
    return e;
  }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}
}  // namespace

void timing_mark(const char* tag, cudaStream_t st, bool begin) {
  std::lock_guard<std::mutex> lk(g_mu);
  if (begin) {
    Span s{tag_index(tag), get_event(), get_event()};
    if (s.a) cudaEventRecord(s.a, st);
    g_open.push_back(s);
  } else if (!g_open.empty()) {
    Span& s = g_open.back();
    if (s.b) cudaEventRecord(s.b, st);
  }
}

}  // namespace dad

using namespace dad;

extern "C" {

void dad_timing_enable(int on) { g_timing.store(on != 0); }

int dad_timing_collect(void) {
  std::lock_guard<std::mutex> lk(g_mu);
  for (Span& s : g_open) {
    if (s.a && s.b && cudaEventSynchronize(s.b) == cudaSuccess) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, s.a, s.b) == cudaSuccess) {
        g_tags[s.tag].ms += ms;
        g_tags[s.tag].launches += 1;
      }
    }
    if (s.a) g_free.push_back(s.a);
    if (s.b) g_free.push_back(s.b);
  }
  g_open.clear();
  return (int)g_tags.size();
}

void dad_timing_reset(void) {
  dad_timing_collect();
  std::lock_guard<std::mutex> lk(g_mu);
  for (Tag& t : g_tags) {
    t.ms = 0.0;
    t.launches = 0;
  }
}

const char* dad_timing_name(int i) {
  std::lock_guard<std::mutex> lk(g_mu);
  return (i >= 0 && (size_t)i < g_tags.size()) ? g_tags[i].name.c_str() : "";
}
double dad_timing_ms(int i) {
  std::lock_guard<std::mutex> lk(g_mu);
  return (i >= 0 && (size_t)i < g_tags.size()) ? g_tags[i].ms : 0.0;
}
uint64_t dad_timing_launches(int i) {
  std::lock_guard<std::mutex> lk(g_mu);
  return (i >= 0 && (size_t)i < g_tags.size()) ? g_tags[i].launches : 0;
}

}  // extern "C"
