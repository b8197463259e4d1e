// NUMA placement helpers (sysfs parsing).  No CUDA in this file.
#pragma once
#include <string>
#include <vector>

namespace kvr {

std::vector<int> parse_cpulist(const std::string &text);
// NUMA node of the PCI device (-1: unknown) and, if asked for, that node's CPUs.  sysfs_root NULL = "/sys".
int numa_lookup(const char *sysfs_root, const char *pci_bus_id, std::vector<int> *cpus);

}  // namespace kvr
