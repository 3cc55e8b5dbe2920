#define LBA_QM lba::QM_RNE_WIDE
#define LBA_ORD lba::ORD_CHUNK_SLAB
#include "lba_family.inc"
