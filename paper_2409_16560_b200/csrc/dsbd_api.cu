// Small host-only entry points of the DSBD library.
#include "dsbd.h"

extern "C" const char *dsbd_status_string(int code) {
    switch (code) {
        case DSBD_OK: return "ok";
        case DSBD_ERR_INVALID_ARG: return "invalid argument";
        case DSBD_ERR_UNSUPPORTED: return "unsupported shape, dtype or alignment";
        case DSBD_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case DSBD_ERR_CUDA: return "CUDA launch failed";
        case DSBD_DEV_BAD_TOKEN: return "device: draft token outside the vocabulary";
        case DSBD_DEV_EXHAUSTED: return "device: distribution without mass";
        case DSBD_DEV_CAPACITY: return "device: output range too small";
        case DSBD_DEV_BAD_FOREST: return "device: malformed forest";
        case DSBD_DEV_TIMEOUT: return "device: bounded wait gave up";
        case DSBD_DEV_BAD_PARAM: return "device: per-request width out of range";
        default: return "unknown status";
    }
}
