"""B200-native full-batch gradient-descent logistic regression (CUDA, sm_100a).

``datagen`` (seeded inputs) imports without the compiled library; the binding in ``api`` loads the
C-ABI shared library on first use and raises if it is missing -- there is no CPU fallback.
"""
__all__ = ["datagen", "api", "lr_loss_grad", "lr_fit", "lr_predict", "Context", "LrError"]


def __getattr__(name):
    if name in ("lr_loss_grad", "lr_fit", "lr_predict", "Context", "LrError"):
        from . import api
        return getattr(api, name)
    raise AttributeError(name)
