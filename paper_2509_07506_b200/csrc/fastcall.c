/*
 * _astra_fastcall -- a CPython extension that re-issues prepared calls of the astra.h ABI.
 *
 * The Python binding reaches libastra.so through ctypes, whose per-call cost (about 1 us: argument
 * conversion and the foreign-function transition) is as large as the device time of the decode-sized
 * shapes of the paper's Table 4.  A prepared call has already validated and converted its arguments
 * once; this module keeps them in a C struct and `launch(prepared, stream)` passes them straight to
 * the entry point.  It only marshals: every argument check of the C ABI still runs inside the entry
 * point on every launch, and nothing is computed here.
 *
 * The module does not link against libastra.so.  The binding hands it the addresses of the entry
 * points it has already resolved (`bind`), so there is one copy of the library in the process and
 * the staleness check made when the library was loaded covers these calls too.
 */
#define PY_SSIZE_T_CLEAN
#include <Python.h>
#include <stdint.h>
#include <string.h>

#include "astra.h"

#ifndef ASTRA_BUILD_ID
#define ASTRA_BUILD_ID "unidentified"
#endif
/* hash of the sources this module was compiled from; the build script finds it in the file */
__attribute__((used, visibility("default"))) const char astra_fastcall_build_marker[] =
    "astra-build-id:" ASTRA_BUILD_ID;

enum {
    KIND_RMSNORM = 0,
    KIND_SILU = 1,
    KIND_MERGE = 2,
    KIND_ALLREDUCE_RMSNORM = 3,
    KIND_COUNT = 4
};

#define MAX_PARTS 16

typedef astra_status_t (*rmsnorm_fn)(void *, void *, const void *, int64_t, int64_t, float, astra_dtype_t, void *);
typedef astra_status_t (*silu_fn)(void *, const void *, int64_t, int64_t, astra_dtype_t, void *);
typedef astra_status_t (*merge_fn)(void *, float *, const void *, const float *, const void *, const float *,
                                   int64_t, int64_t, int64_t, astra_dtype_t, void *);
typedef astra_status_t (*allreduce_fn)(void *, void *, const void *const *, int32_t, const void *, int64_t,
                                       int64_t, float, astra_dtype_t, void *);

static void *entry_points[KIND_COUNT];

typedef struct {
    PyObject_HEAD
    int kind;
    int dtype;
    int n_parts;
    float eps;
    void *ptr[6];               /* the call's pointer arguments, in the order of its declaration */
    int64_t ext[3];             /* the call's extents, in the order of its declaration */
    const void *parts[MAX_PARTS];
} Prepared;

static PyTypeObject PreparedType = {
    PyVarObject_HEAD_INIT(NULL, 0)
    .tp_name = "_astra_fastcall.Prepared",
    .tp_basicsize = sizeof(Prepared),
    .tp_flags = Py_TPFLAGS_DEFAULT,
    .tp_doc = "arguments of one astra call, ready to be launched",
};

static int as_address(PyObject *o, void **out) {
    if (o == Py_None) {
        *out = NULL;
        return 0;
    }
    *out = PyLong_AsVoidPtr(o);
    return (*out == NULL && PyErr_Occurred()) ? -1 : 0;
}

/* bind(kind, address): the entry point that calls of this kind go to */
static PyObject *fc_bind(PyObject *self, PyObject *args) {
    int kind;
    PyObject *addr;
    if (!PyArg_ParseTuple(args, "iO", &kind, &addr)) return NULL;
    if (kind < 0 || kind >= KIND_COUNT) {
        PyErr_SetString(PyExc_ValueError, "unknown kind of call");
        return NULL;
    }
    void *p;
    if (as_address(addr, &p) < 0) return NULL;
    entry_points[kind] = p;
    Py_RETURN_NONE;
}

/* prepare(kind, pointers, extents, eps, dtype, parts) -> Prepared
 * pointers: the call's pointer arguments (ints or None) in declaration order; extents: its int64
 * extents in declaration order; parts: the partial hidden states of the all-reduce form (else ()). */
static PyObject *fc_prepare(PyObject *self, PyObject *args) {
    int kind, dtype;
    double eps;
    PyObject *pointers, *extents, *parts;
    if (!PyArg_ParseTuple(args, "iO!O!diO!", &kind, &PyTuple_Type, &pointers, &PyTuple_Type, &extents, &eps,
                          &dtype, &PyTuple_Type, &parts))
        return NULL;
    static const int n_pointers[KIND_COUNT] = {3, 2, 6, 3};
    static const int n_extents[KIND_COUNT] = {2, 2, 3, 2};
    if (kind < 0 || kind >= KIND_COUNT) {
        PyErr_SetString(PyExc_ValueError, "unknown kind of call");
        return NULL;
    }
    if (entry_points[kind] == NULL) {
        PyErr_SetString(PyExc_RuntimeError, "no entry point bound for this kind of call");
        return NULL;
    }
    if (PyTuple_GET_SIZE(pointers) != n_pointers[kind] || PyTuple_GET_SIZE(extents) != n_extents[kind]) {
        PyErr_SetString(PyExc_ValueError, "wrong number of pointers or extents for this kind of call");
        return NULL;
    }
    const Py_ssize_t np = PyTuple_GET_SIZE(parts);
    if ((kind == KIND_ALLREDUCE_RMSNORM) ? (np < 1 || np > MAX_PARTS) : (np != 0)) {
        PyErr_SetString(PyExc_ValueError, "wrong number of partial hidden states");
        return NULL;
    }
    Prepared *p = PyObject_New(Prepared, &PreparedType);
    if (p == NULL) return NULL;
    p->kind = kind;
    p->dtype = dtype;
    p->eps = (float)eps;
    p->n_parts = (int)np;
    memset(p->ptr, 0, sizeof p->ptr);
    memset(p->ext, 0, sizeof p->ext);
    memset(p->parts, 0, sizeof p->parts);
    for (int i = 0; i < n_pointers[kind]; ++i)
        if (as_address(PyTuple_GET_ITEM(pointers, i), &p->ptr[i]) < 0) goto fail;
    for (int i = 0; i < n_extents[kind]; ++i) {
        p->ext[i] = PyLong_AsLongLong(PyTuple_GET_ITEM(extents, i));
        if (p->ext[i] == -1 && PyErr_Occurred()) goto fail;
    }
    for (Py_ssize_t i = 0; i < np; ++i) {
        void *a;
        if (as_address(PyTuple_GET_ITEM(parts, i), &a) < 0) goto fail;
        p->parts[i] = a;
    }
    return (PyObject *)p;
fail:
    Py_DECREF(p);
    return NULL;
}

/* launch(prepared, stream_handle) -> status code of the entry point */
static PyObject *fc_launch(PyObject *self, PyObject *const *args, Py_ssize_t nargs) {
    if (nargs != 2 || !Py_IS_TYPE(args[0], &PreparedType)) {
        PyErr_SetString(PyExc_TypeError, "launch(prepared, stream_handle)");
        return NULL;
    }
    const Prepared *p = (const Prepared *)args[0];
    void *stream = PyLong_AsVoidPtr(args[1]);
    if (stream == NULL && PyErr_Occurred()) return NULL;
    const astra_dtype_t dt = (astra_dtype_t)p->dtype;
    void *fn = entry_points[p->kind];
    if (fn == NULL) {  /* unbound again since the call was prepared */
        PyErr_SetString(PyExc_RuntimeError, "no entry point bound for this kind of call");
        return NULL;
    }
    astra_status_t st;
    switch (p->kind) {
        case KIND_RMSNORM:
            st = ((rmsnorm_fn)fn)(p->ptr[0], p->ptr[1], p->ptr[2], p->ext[0], p->ext[1], p->eps, dt, stream);
            break;
        case KIND_SILU:
            st = ((silu_fn)fn)(p->ptr[0], p->ptr[1], p->ext[0], p->ext[1], dt, stream);
            break;
        case KIND_MERGE:
            st = ((merge_fn)fn)(p->ptr[0], (float *)p->ptr[1], p->ptr[2], (const float *)p->ptr[3], p->ptr[4],
                                (const float *)p->ptr[5], p->ext[0], p->ext[1], p->ext[2], dt, stream);
            break;
        default:
            st = ((allreduce_fn)fn)(p->ptr[0], p->ptr[1], p->parts, p->n_parts, p->ptr[2], p->ext[0], p->ext[1],
                                    p->eps, dt, stream);
            break;
    }
    return PyLong_FromLong((long)st);
}

static PyObject *fc_build_id(PyObject *self, PyObject *noargs) {
    return PyUnicode_FromString(astra_fastcall_build_marker + sizeof("astra-build-id:") - 1);
}

static PyMethodDef methods[] = {
    {"bind", fc_bind, METH_VARARGS, "bind(kind, address): set the entry point of one kind of call"},
    {"prepare", fc_prepare, METH_VARARGS, "prepare(kind, pointers, extents, eps, dtype, parts) -> Prepared"},
    {"launch", (PyCFunction)(void (*)(void))fc_launch, METH_FASTCALL, "launch(prepared, stream_handle) -> status"},
    {"build_id", fc_build_id, METH_NOARGS, "hash of the sources this module was compiled from"},
    {NULL, NULL, 0, NULL},
};

static struct PyModuleDef module = {PyModuleDef_HEAD_INIT, "_astra_fastcall",
                                    "re-issue prepared calls of the astra C ABI without ctypes", -1, methods};

PyMODINIT_FUNC PyInit__astra_fastcall(void) {
    if (PyType_Ready(&PreparedType) < 0) return NULL;
    PyObject *m = PyModule_Create(&module);
    if (m == NULL) return NULL;
    Py_INCREF(&PreparedType);
    if (PyModule_AddObject(m, "Prepared", (PyObject *)&PreparedType) < 0) {
        Py_DECREF(&PreparedType);
        Py_DECREF(m);
        return NULL;
    }
    PyModule_AddIntConstant(m, "KIND_RMSNORM", KIND_RMSNORM);
    PyModule_AddIntConstant(m, "KIND_SILU", KIND_SILU);
    PyModule_AddIntConstant(m, "KIND_MERGE", KIND_MERGE);
    PyModule_AddIntConstant(m, "KIND_ALLREDUCE_RMSNORM", KIND_ALLREDUCE_RMSNORM);
    return m;
}
