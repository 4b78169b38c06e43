// Header of a device blob (internal to the library).
#ifndef SQNN_BLOB_H_
#define SQNN_BLOB_H_
#include "sqnn.h"

#define SQNN_BLOB_MAGIC        "SQNNBLB2"
#define SQNN_BLOB_VERSION      2u
#define SQNN_BLOB_HEADER_BYTES 512u

typedef struct sqnn_blob_header {
    char     magic[8];
    uint32_t version;
    uint32_t header_bytes;
    sqnn_desc desc;
} sqnn_blob_header;

#ifdef __cplusplus
static_assert(sizeof(sqnn_blob_header) <= SQNN_BLOB_HEADER_BYTES, "header does not fit");
#endif
#endif
