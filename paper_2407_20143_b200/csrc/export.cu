// Export of a set of tensors as one Safetensors image in device memory.
//
// The paper's system can export checkpoints in the Safetensors format for compatibility with
// the Hugging Face ecosystem (Sec. 7, related work on checkpoint representation).  The file
// format itself is public: 8 bytes little-endian header length N, N bytes of JSON mapping every
// tensor name to {"dtype", "shape", "data_offsets": [begin, end)} (offsets relative to the end of
// the header, tensors back to back in offset order), then the tensor bytes.  Here the header
// is built on the host and the byte buffer is a bcp_pack of the tensors without padding.
#include <cstdio>
#include <cstring>
#include <string>
#include <vector>

#include "kernels.cuh"
#include "plan.hpp"

using namespace bcp;

namespace {

const struct {
  const char* name;
  uint32_t itemsize;
} kDtypes[] = {{"BOOL", 1}, {"U8", 1}, {"I8", 1}, {"F8_E5M2", 1}, {"F8_E4M3", 1}, {"I16", 2}, {"U16", 2}, {"F16", 2},
               {"BF16", 2}, {"I32", 4}, {"U32", 4}, {"F32", 4}, {"F64", 8}, {"I64", 8}, {"U64", 8}};

uint32_t dtype_size(const char* d) {
  for (const auto& k : kDtypes)
    if (strcmp(k.name, d) == 0) return k.itemsize;
  return 0;
}

void json_string(const char* s, std::string* out) {
  out->push_back('"');
  for (const unsigned char* p = reinterpret_cast<const unsigned char*>(s); *p; ++p) {
    if (*p == '"' || *p == '\\') {
      out->push_back('\\');
      out->push_back(char(*p));
    } else if (*p < 0x20) {
      char buf[8];
      snprintf(buf, sizeof buf, "\\u%04x", *p);
      out->append(buf);
    } else {
      out->push_back(char(*p));
    }
  }
  out->push_back('"');
}

int build_header(const bcp_export_entry* e, size_t n, std::string* header, std::vector<bcp_pack_meta>* metas, uint64_t* file_bytes) {
  if (n && !e) return fail(BCP_ERR_INVALID, "safetensors export: entries is NULL");
  std::string js = "{";
  uint64_t pos = 0;
  metas->resize(n);
  for (size_t i = 0; i < n; ++i) {
    if (!e[i].name || !e[i].dtype || !*e[i].name) return fail(BCP_ERR_INVALID, "safetensors export: entry %zu has no name or dtype", i);
    if (strcmp(e[i].name, "__metadata__") == 0) return fail(BCP_ERR_INVALID, "safetensors export: \"__metadata__\" is reserved");
    for (size_t j = 0; j < i; ++j)
      if (strcmp(e[i].name, e[j].name) == 0) return fail(BCP_ERR_INVALID, "safetensors export: duplicate tensor name %s", e[i].name);
    const uint32_t isz = dtype_size(e[i].dtype);
    if (!isz) return fail(BCP_ERR_INVALID, "safetensors export: unknown dtype %s for %s", e[i].dtype, e[i].name);
    if (e[i].ndim > BCP_MAX_NDIM) return fail(BCP_ERR_INVALID, "safetensors export: %s has ndim %u", e[i].name, e[i].ndim);
    uint64_t numel = 1;
    for (uint32_t k = 0; k < e[i].ndim; ++k) {
      if (e[i].shape[k] < 0) return fail(BCP_ERR_INVALID, "safetensors export: %s has a negative extent", e[i].name);
      numel *= uint64_t(e[i].shape[k]);
    }
    const uint64_t bytes = numel * isz;
    if (i) js.push_back(',');
    json_string(e[i].name, &js);
    js += ":{\"dtype\":\"";
    js += e[i].dtype;
    js += "\",\"shape\":[";
    for (uint32_t k = 0; k < e[i].ndim; ++k) {
      if (k) js.push_back(',');
      js += std::to_string((long long)e[i].shape[k]);
    }
    js += "],\"data_offsets\":[" + std::to_string((unsigned long long)pos) + "," + std::to_string((unsigned long long)(pos + bytes)) + "]}";
    (*metas)[i].byte_offset = pos;
    (*metas)[i].byte_length = bytes;
    pos += bytes;
  }
  js.push_back('}');
  while ((8 + js.size()) % 8) js.push_back(' ');  // the byte buffer starts on an 8-byte boundary
  const uint64_t hlen = js.size();
  header->assign(8, '\0');
  for (int k = 0; k < 8; ++k) (*header)[k] = char((hlen >> (8 * k)) & 0xFF);
  header->append(js);
  for (bcp_pack_meta& m : *metas) m.byte_offset += header->size();
  *file_bytes = header->size() + pos;
  return BCP_OK;
}

}  // namespace

extern "C" {

int bcp_safetensors_layout(const bcp_export_entry* entries, size_t n, void* header_out, size_t header_cap, size_t* header_bytes,
                           bcp_pack_meta* out_metas, uint64_t* file_bytes) {
  if (!header_bytes || !file_bytes || (n && !out_metas)) return fail(BCP_ERR_INVALID, "bcp_safetensors_layout: NULL argument");
  std::string header;
  std::vector<bcp_pack_meta> metas;
  uint64_t total = 0;
  try {
    if (int rc = build_header(entries, n, &header, &metas, &total)) return rc;
  } catch (const std::bad_alloc&) {
    return fail(BCP_ERR_NOMEM, "out of host memory");
  }
  *header_bytes = header.size();
  *file_bytes = total;
  for (size_t i = 0; i < n; ++i) out_metas[i] = metas[i];
  if (!header_out || header_cap < header.size())
    return fail(BCP_ERR_CAPACITY, "bcp_safetensors_layout: header needs %zu bytes, room for %zu", header.size(), header_out ? header_cap : size_t(0));
  memcpy(header_out, header.data(), header.size());
  return BCP_OK;
}

int bcp_safetensors_export(const bcp_export_entry* entries, const void* const* tensors, size_t n, void* file, uint64_t file_cap,
                           uint64_t* file_bytes, void* stream_) {
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  if (!file_bytes || (n && !tensors)) return fail(BCP_ERR_INVALID, "bcp_safetensors_export: NULL argument");
  std::string header;
  std::vector<bcp_pack_meta> metas;
  uint64_t total = 0;
  try {
    if (int rc = build_header(entries, n, &header, &metas, &total)) return rc;
  } catch (const std::bad_alloc&) {
    return fail(BCP_ERR_NOMEM, "out of host memory");
  }
  *file_bytes = total;
  if (!file || file_cap < total)
    return fail(BCP_ERR_CAPACITY, "bcp_safetensors_export: image needs %llu bytes, room for %llu", (unsigned long long)total,
                (unsigned long long)(file ? file_cap : 0));
  // tensor bytes first (the pack also zeroes the header region), then the header over it
  if (int rc = bcp_pack(tensors, metas.data(), n, file, total, stream)) return rc;
  const cudaError_t e = cudaMemcpyAsync(file, header.data(), header.size(), cudaMemcpyHostToDevice, stream);
  if (e != cudaSuccess) return fail(BCP_ERR_CUDA, "cudaMemcpyAsync(header): %s", cudaGetErrorString(e));
  return BCP_OK;
}

}  // extern "C"
