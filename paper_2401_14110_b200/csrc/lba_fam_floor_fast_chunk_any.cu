#define LBA_QM lba::QM_FLOOR_FAST
#define LBA_ORD lba::ORD_CHUNK_ANY
#include "lba_family.inc"
