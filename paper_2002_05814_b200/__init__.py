"""hpl: chunk-pipelined reduce and broadcast over an object store on one B200 (sm_100a).

The product is the C-ABI library ``libhpl.so`` (declared in ``include/hpl.h``); this package
is its thin ctypes binding.  Importing the package does not load the library; the first use
does, and fails loudly if it has not been built (``python -m paper_2002_05814_b200.build``).
"""
from .hpl import (  # noqa: F401
    HplError, Context, Config, load_library, lib_path, reduce_noalloc, choose_degree, ipc_export, ipc_import, ipc_close,
    HPL_F32, HPL_BF16, HPL_SUM, HPL_MIN, HPL_MAX,
    HPL_OK, HPL_ERR_INVALID, HPL_ERR_NOT_FOUND, HPL_ERR_EXISTS, HPL_ERR_TIMEOUT,
    HPL_ERR_INSUFFICIENT, HPL_ERR_FAILED_WORKER, HPL_ERR_CUDA, HPL_ERR_NOMEM,
    Event, EventList, HPL_EV_CREATE, HPL_EV_PUT, HPL_EV_PUT_HOST, HPL_EV_REDUCE, HPL_EV_BROADCAST, HPL_EV_JOIN,
    HPL_EV_FAIL, HPL_EV_REJOIN, HPL_EV_PROGRESS, HPL_EV_GET, HPL_EV_DELETE, HPL_EV_SYNC, HPL_EV_MARK,
)
