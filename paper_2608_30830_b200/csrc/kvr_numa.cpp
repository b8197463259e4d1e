// Where a GPU hangs in the host: its NUMA node and that node's CPUs, read from sysfs text files.
// Host DRAM bandwidth is shared between the GPUs of a node; an arena that lives on the GPU's own NUMA node keeps
// the suspend / resume traffic off the inter-socket link.  No CUDA in this file.
#include "kvr_numa.hpp"

#include <cctype>
#include <cstdio>
#include <cstdlib>
#include <string>

#include "../../include/kvr.h"

namespace kvr {

namespace {

bool read_line(const std::string &path, std::string *out) {
  FILE *f = fopen(path.c_str(), "r");
  if (!f) return false;
  char buf[4096];
  const bool ok = fgets(buf, sizeof buf, f) != nullptr;
  fclose(f);
  if (!ok) return false;
  *out = buf;
  while (!out->empty() && isspace((unsigned char)out->back())) out->pop_back();
  return true;
}

}  // namespace

// "0-15,32-47" -> 0..15, 32..47.  Malformed text gives an empty list.
std::vector<int> parse_cpulist(const std::string &text) {
  std::vector<int> cpus;
  size_t i = 0;
  while (i < text.size()) {
    char *end = nullptr;
    const long lo = strtol(text.c_str() + i, &end, 10);
    if (end == text.c_str() + i || lo < 0) return {};
    long hi = lo;
    i = (size_t)(end - text.c_str());
    if (i < text.size() && text[i] == '-') {
      hi = strtol(text.c_str() + i + 1, &end, 10);
      if (end == text.c_str() + i + 1 || hi < lo) return {};
      i = (size_t)(end - text.c_str());
    }
    if (hi - lo > 65536) return {};
    for (long c = lo; c <= hi; ++c) cpus.push_back((int)c);
    if (i < text.size()) {
      if (text[i] != ',') return {};
      ++i;
    }
  }
  return cpus;
}

int numa_lookup(const char *sysfs_root, const char *pci_bus_id, std::vector<int> *cpus) {
  if (cpus) cpus->clear();
  if (!pci_bus_id || !*pci_bus_id) return -1;
  const std::string root = (sysfs_root && *sysfs_root) ? sysfs_root : "/sys";
  std::string bdf = pci_bus_id;
  for (auto &c : bdf) c = (char)tolower((unsigned char)c);      // CUDA prints hex digits in upper case, sysfs in lower
  std::string text;
  if (!read_line(root + "/bus/pci/devices/" + bdf + "/numa_node", &text)) return -1;
  char *end = nullptr;
  const long node = strtol(text.c_str(), &end, 10);
  if (end == text.c_str() || node < 0) return -1;               // "-1": the platform does not say
  if (cpus && read_line(root + "/devices/system/node/node" + std::to_string(node) + "/cpulist", &text))
    *cpus = parse_cpulist(text);
  return (int)node;
}

}  // namespace kvr

extern "C" int32_t kvr_numa_lookup(const char *sysfs_root, const char *pci_bus_id, int32_t *node, int32_t *cpus, int32_t cap) {
  std::vector<int> list;
  const int n = kvr::numa_lookup(sysfs_root, pci_bus_id, &list);
  if (node) *node = n;
  if (n < 0) return 0;
  if (cpus) for (size_t i = 0; i < list.size() && (int32_t)i < cap; ++i) cpus[i] = list[i];
  return (int32_t)list.size();
}
