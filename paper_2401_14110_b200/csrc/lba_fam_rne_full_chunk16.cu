#define LBA_QM lba::QM_RNE_FULL
#define LBA_ORD lba::ORD_CHUNK16
#include "lba_family.inc"
