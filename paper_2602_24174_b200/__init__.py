"""B200 (sm_100a) implementation of one batched n-gram speculative-decoding step
(draft from corpus + context n-grams, verify k+1 positions in one forward, greedy accept).

The work is done by ``libtasc.so`` (CUDA, C ABI declared in ``include/tasc.h``); ``binding``
marshals torch CUDA tensors into it.  There is no CPU or PyTorch fallback: using the binding
without the built library raises ImportError.
"""

# File name of the CUDA library inside this package that `binding` loads.
LIBRARY_FILE = "libtasc.so"


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
