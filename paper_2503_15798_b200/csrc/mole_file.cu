// Table files: the re-parameterised tables of Eq. 6-7 on a storage device below host memory (Sec. 3.3 and
// Sec. 4.2 of arXiv 2503.15798 keep them "offloaded"; they are far larger than the model).  One file holds
// the tables of all L layers, plain elements or the packed records of a quantised table, behind a 4 KB
// header; whole layers are read into (pinned) host memory for the offload mode, and single rows can be
// read by id for a tier that leaves the file on disk.  Host code only: POSIX file calls, no CUDA.
#include <errno.h>
#include <fcntl.h>
#include <stdio.h>
#include <string.h>
#include <sys/stat.h>
#include <unistd.h>

#include "mole_common.cuh"

namespace mole {

constexpr char kMagic[8] = {'M', 'O', 'L', 'E', 'L', 'U', 'T', '1'};
constexpr uint64_t kDataOffset = 4096;

struct FileHeader {  // little endian, 4096 bytes on disk (zero padded)
    char magic[8];
    uint32_t version, lut_format, dtype, lut_block;
    uint64_t L, V, N, d, row_bytes, data_offset;
};

static int read_header(int fd, FileHeader *h)
{
    unsigned char buf[sizeof(FileHeader)];
    if (pread(fd, buf, sizeof buf, 0) != static_cast<ssize_t>(sizeof buf)) return MOLE_ERR_IO;
    memcpy(h, buf, sizeof *h);
    if (memcmp(h->magic, kMagic, 8) != 0 || h->version != 1) return MOLE_ERR_IO;
    if (h->L < 1 || h->V < 1 || h->N < 1 || h->d < 1 || h->row_bytes < 16 || (h->row_bytes & 15) || h->data_offset < sizeof(FileHeader))
        return MOLE_ERR_IO;
    return MOLE_OK;
}

static int pread_all(int fd, void *dst, uint64_t bytes, uint64_t offset)
{
    unsigned char *p = static_cast<unsigned char *>(dst);
    while (bytes > 0) {
        const size_t want = bytes > (1u << 30) ? (1u << 30) : static_cast<size_t>(bytes);
        const ssize_t got = pread(fd, p, want, static_cast<off_t>(offset));
        if (got < 0 && errno == EINTR) continue;
        if (got <= 0) return MOLE_ERR_IO;  // error, or the file is shorter than its header says
        p += got;
        offset += static_cast<uint64_t>(got);
        bytes -= static_cast<uint64_t>(got);
    }
    return MOLE_OK;
}

static int pwrite_all(int fd, const void *src, uint64_t bytes, uint64_t offset)
{
    const unsigned char *p = static_cast<const unsigned char *>(src);
    while (bytes > 0) {
        const size_t want = bytes > (1u << 30) ? (1u << 30) : static_cast<size_t>(bytes);
        const ssize_t put = pwrite(fd, p, want, static_cast<off_t>(offset));
        if (put < 0 && errno == EINTR) continue;
        if (put <= 0) return MOLE_ERR_IO;
        p += put;
        offset += static_cast<uint64_t>(put);
        bytes -= static_cast<uint64_t>(put);
    }
    return MOLE_OK;
}

}  // namespace mole

using namespace mole;

extern "C" {

int mole_table_file_write(const char *path, const void *tables_host, int64_t layer_stride_bytes, int L, int V, int N, int d,
                          int dtype, int lut_format, int lut_block)
{
    if (!path || !tables_host || L < 1 || V < 1 || N < 1 || N > 64 || d < 1) return MOLE_ERR_INVALID_ARG;
    if (dtype != MOLE_DTYPE_BF16 && dtype != MOLE_DTYPE_F32) return MOLE_ERR_INVALID_ARG;
    int64_t row_bytes = 0;
    if (lut_format == MOLE_LUT_PLAIN) {
        row_bytes = static_cast<int64_t>(N) * d * elem_bytes(dtype);
        if (row_bytes & 15) return MOLE_ERR_UNSUPPORTED_SHAPE;
    } else {
        int rc = mole_quant_record_bytes(N, d, lut_format, lut_block, &row_bytes);
        if (rc != MOLE_OK) return rc;
    }
    if (layer_stride_bytes < row_bytes * V) return MOLE_ERR_INVALID_ARG;
    const int fd = open(path, O_WRONLY | O_CREAT | O_TRUNC, 0644);
    if (fd < 0) return MOLE_ERR_IO;
    unsigned char head[kDataOffset];
    memset(head, 0, sizeof head);
    FileHeader h;
    memset(&h, 0, sizeof h);
    memcpy(h.magic, kMagic, 8);
    h.version = 1;
    h.lut_format = static_cast<uint32_t>(lut_format);
    h.dtype = static_cast<uint32_t>(dtype);
    h.lut_block = static_cast<uint32_t>(lut_format == MOLE_LUT_PLAIN ? 0 : lut_block);
    h.L = L, h.V = V, h.N = N, h.d = d;
    h.row_bytes = static_cast<uint64_t>(row_bytes);
    h.data_offset = kDataOffset;
    memcpy(head, &h, sizeof h);
    int rc = pwrite_all(fd, head, sizeof head, 0);
    const uint64_t layer_bytes = static_cast<uint64_t>(row_bytes) * V;
    for (int l = 0; l < L && rc == MOLE_OK; ++l)
        rc = pwrite_all(fd, static_cast<const unsigned char *>(tables_host) + static_cast<int64_t>(l) * layer_stride_bytes, layer_bytes,
                        kDataOffset + static_cast<uint64_t>(l) * layer_bytes);
    if (close(fd) != 0 && rc == MOLE_OK) rc = MOLE_ERR_IO;
    return rc;
}

int mole_table_file_info(const char *path, mole_table_info *info)
{
    if (!path || !info) return MOLE_ERR_INVALID_ARG;
    const int fd = open(path, O_RDONLY);
    if (fd < 0) return MOLE_ERR_IO;
    FileHeader h;
    int rc = read_header(fd, &h);
    if (rc == MOLE_OK) {
        struct stat st;
        if (fstat(fd, &st) != 0 || static_cast<uint64_t>(st.st_size) < h.data_offset + h.L * h.V * h.row_bytes) rc = MOLE_ERR_IO;  // truncated
    }
    close(fd);
    if (rc != MOLE_OK) return rc;
    info->L = static_cast<int64_t>(h.L);
    info->V = static_cast<int64_t>(h.V);
    info->N = static_cast<int32_t>(h.N);
    info->d = static_cast<int32_t>(h.d);
    info->dtype = static_cast<int32_t>(h.dtype);
    info->lut_format = static_cast<int32_t>(h.lut_format);
    info->lut_block = static_cast<int32_t>(h.lut_block);
    info->reserved = 0;
    info->row_bytes = static_cast<int64_t>(h.row_bytes);
    return MOLE_OK;
}

int mole_table_file_read(const char *path, void *dst_host, int64_t dst_layer_stride_bytes, int layer0, int n_layers)
{
    if (!path || !dst_host || layer0 < 0 || n_layers < 1) return MOLE_ERR_INVALID_ARG;
    const int fd = open(path, O_RDONLY);
    if (fd < 0) return MOLE_ERR_IO;
    FileHeader h;
    int rc = read_header(fd, &h);
    const uint64_t layer_bytes = rc == MOLE_OK ? h.row_bytes * h.V : 0;
    if (rc == MOLE_OK && (static_cast<uint64_t>(layer0) + n_layers > h.L || static_cast<uint64_t>(dst_layer_stride_bytes) < layer_bytes))
        rc = MOLE_ERR_INVALID_ARG;
    for (int l = 0; l < n_layers && rc == MOLE_OK; ++l)
        rc = pread_all(fd, static_cast<unsigned char *>(dst_host) + static_cast<int64_t>(l) * dst_layer_stride_bytes, layer_bytes,
                       h.data_offset + static_cast<uint64_t>(layer0 + l) * layer_bytes);
    close(fd);
    return rc;
}

int mole_table_file_read_rows(const char *path, int layer, const int32_t *ids_host, int n, void *dst_host)
{
    if (!path || layer < 0 || n < 0 || (n > 0 && (!ids_host || !dst_host))) return MOLE_ERR_INVALID_ARG;
    const int fd = open(path, O_RDONLY);
    if (fd < 0) return MOLE_ERR_IO;
    FileHeader h;
    int rc = read_header(fd, &h);
    if (rc == MOLE_OK && static_cast<uint64_t>(layer) >= h.L) rc = MOLE_ERR_INVALID_ARG;
    for (int i = 0; i < n && rc == MOLE_OK; ++i) {
        if (ids_host[i] < 0 || static_cast<uint64_t>(ids_host[i]) >= h.V) {
            rc = MOLE_ERR_INVALID_ARG;
            break;
        }
        rc = pread_all(fd, static_cast<unsigned char *>(dst_host) + static_cast<uint64_t>(i) * h.row_bytes, h.row_bytes,
                       h.data_offset + (static_cast<uint64_t>(layer) * h.V + static_cast<uint64_t>(ids_host[i])) * h.row_bytes);
    }
    close(fd);
    return rc;
}

}  // extern "C"
